// Prefill of one MoE layer from bit-sliced AMAT weights: many tokens at once, so the expert FFN is a
// genuine dense contraction (Section 3 of the paper: prefill loads every expert of a layer).  Section 6.3 notes
// that prefill wants high-bit computation; the per-expert precision flag here is this library's generalisation
// (an expert can also be run from its MSB slice alone), which the mixed-precision prefill benchmark uses.
//
// Steps, all on the device:
//   1. count the tokens of every routed expert, lay the experts' token rows out one after the other
//      (each expert padded to a multiple of 128 rows), list the 128-row tiles;
//   2. gather x (bf16) into that order as fp16 (exact for every bf16 value in fp16's normal range);
//   3. grouped GEMM 1: per tile  H = silu(X Wg^T) * (X Wu^T)  (fp16 out);
//   4. grouped GEMM 2: per tile  Yrow = H Wd^T  (fp32 out, one row per (token, expert) pair);
//   5. combine: y[t] = sum_j w[t,j] Yrow[pos(t,j)] + shared experts, in list order (deterministic).
// In both GEMMs the weight tile is dequantised on the fly from the nibble planes - s * (q - zp) from both
// slices, 16 s * (q_msb - (zp >> 4)) from the MSB slice alone - straight into tensor memory and multiplied on
// the 5th-generation tensor cores (tcgen05.mma, fp16 x fp16 -> fp32).  A dequantised weight needs about 20
// significant bits, fp16 holds 11: every weight is therefore kept as the exact sum of two fp16 numbers and
// multiplied in two MMAs.
#include <cuda.h>  // CUtensorMap (types only; the encoder is fetched through the runtime)
#include <cuda_fp16.h>

#include "common.cuh"

namespace slicemoe {

constexpr int kPfTileM = 128;  // token rows per tile
constexpr int kPfTileB = 128;  // weight rows per tile: 64 gate + 64 up columns of h (GEMM 1), 128 columns of y (GEMM 2)
constexpr int kPfChunkK = 64;  // contraction columns per pipeline step (one plane block)

// ---- workspace layout (host and device agree through this one function) --------------------------------
struct PfLayout {
  size_t counts, cursor, offsets, tile_expert, tile_row0, item_start, ntiles, row_token, posmap, gate, xs, h, yrow, total;
  int rmax, max_tiles, nexp_all;
};
__host__ __device__ inline size_t pf_align(size_t v) { return (v + 255) & ~(size_t)255; }
__host__ __device__ inline PfLayout pf_layout(int T, int E, int k, int n_shared, int hidden, int inter, int shared_inter) {
  PfLayout L;
  L.nexp_all = E + n_shared;
  // routed rows: T*k plus at most 127 rows of padding per expert; shared: T rows each, padded
  const int tpad = (T + kPfTileM - 1) / kPfTileM * kPfTileM;
  L.rmax = (T * k + E * (kPfTileM - 1) + kPfTileM - 1) / kPfTileM * kPfTileM + n_shared * tpad;
  L.max_tiles = L.rmax / kPfTileM;
  const int wide = inter > shared_inter ? inter : shared_inter;
  size_t o = 0;
  L.counts = o;       o = pf_align(o + sizeof(int) * L.nexp_all);
  L.cursor = o;       o = pf_align(o + sizeof(int) * L.nexp_all);
  L.offsets = o;      o = pf_align(o + sizeof(int) * (L.nexp_all + 1));
  L.tile_expert = o;  o = pf_align(o + sizeof(int) * L.max_tiles);
  L.tile_row0 = o;    o = pf_align(o + sizeof(int) * L.max_tiles);
  L.item_start = o;   o = pf_align(o + sizeof(int) * (L.max_tiles + 1));
  L.ntiles = o;       o = pf_align(o + sizeof(int) * 4);
  L.row_token = o;    o = pf_align(o + sizeof(int) * L.rmax);
  L.posmap = o;       o = pf_align(o + sizeof(int) * (size_t)T * (k + n_shared));
  L.gate = o;         o = pf_align(o + sizeof(float) * T);
  L.xs = o;           o = pf_align(o + sizeof(__half) * (size_t)L.rmax * hidden);
  L.h = o;            o = pf_align(o + sizeof(__half) * (size_t)L.rmax * wide);
  L.yrow = o;         o = pf_align(o + sizeof(float) * (size_t)L.rmax * hidden);
  L.total = o;
  return L;
}

// ---- step 1: token rows per expert -----------------------------------------------------------------------
__global__ void pf_count_kernel(const int32_t* __restrict__ ids, int n, int E, int* __restrict__ counts,
                                unsigned* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int e = ids[i];
  if (e < 0 || e >= E) {
    atomicOr(status, (unsigned)SLICEMOE_STATUS_BAD_EXPERT_ID);
    return;
  }
  atomicAdd(&counts[e], 1);
}

// One warp: padded offsets of every expert (routed, then shared with T rows each) and the tile list.  Lane l takes
// the experts l, l + 32, ...; warp scans turn the experts' tile and item counts into each tile's place in the lists.
__global__ void pf_scan_kernel(const int* __restrict__ counts, int E, int n_shared, int T, int inter, int shared_inter,
                               int* __restrict__ offsets, int* __restrict__ tile_expert, int* __restrict__ tile_row0,
                               int* __restrict__ item_start, int* __restrict__ ntiles) {
  const int lane = threadIdx.x & 31;
  if (threadIdx.x >= 32) return;
  const int n = E + n_shared;
  int nt = 0, items = 0, nt_routed = 0;  // tiles / first-GEMM work items / routed experts' tiles so far
  for (int e0 = 0; e0 < n; e0 += 32) {
    const int e = e0 + lane;
    const int c = e < n ? (e < E ? counts[e] : T) : 0;
    const int tiles = (c + kPfTileM - 1) / kPfTileM;
    const int per = (e < E ? inter : shared_inter) / 64;  // first GEMM: 64 columns of h per work item
    int tin = tiles, iin = tiles * per;                    // inclusive scans
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, tin, off), b = __shfl_up_sync(0xffffffffu, iin, off);
      if (lane >= off) {
        tin += a;
        iin += b;
      }
    }
    const int routed = __reduce_add_sync(0xffffffffu, e < E ? tiles : 0);
    if (e < n) {
      const int first = nt + tin - tiles;  // the expert's first tile; rows are padded to whole tiles
      offsets[e] = first * kPfTileM;
      for (int r = 0; r < tiles; ++r) {
        tile_expert[first + r] = e;
        tile_row0[first + r] = (first + r) * kPfTileM;
        item_start[first + r] = items + iin - tiles * per + r * per;
      }
    }
    nt += __shfl_sync(0xffffffffu, tin, 31);
    items += __shfl_sync(0xffffffffu, iin, 31);
    nt_routed += routed;
  }
  if (lane == 0) {
    offsets[n] = nt * kPfTileM;
    item_start[nt] = items;
    ntiles[0] = nt;
    ntiles[1] = nt * kPfTileM;
    ntiles[2] = items;
    ntiles[3] = n_shared > 0 ? nt_routed : nt;  // tiles of routed experts: they come first and have inter / 64 items each
  }
}

// Every (token, slot) pair takes a row of its expert; shared experts take row t.  Which row a pair gets
// depends on the order of the atomics, the values computed for it do not.
__global__ void pf_scatter_kernel(const int32_t* __restrict__ ids, int T, int k, int E, int n_shared,
                                  const int* __restrict__ offsets, int* __restrict__ cursor, int* __restrict__ row_token,
                                  int* __restrict__ posmap) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int slots = k + n_shared;
  if (i >= T * slots) return;
  const int t = i / slots, j = i % slots;
  int pos = -1;
  if (j < k) {
    const int e = ids[t * k + j];
    if (e >= 0 && e < E) pos = offsets[e] + atomicAdd(&cursor[e], 1);
  } else {
    pos = offsets[E + (j - k)] + t;
  }
  posmap[i] = pos;
  if (pos >= 0) row_token[pos] = t;
}

// ---- step 2: gather x into expert order, bf16 -> fp16; padding rows are zero ----------------------------
// With a gated shared expert the rows of the first shared expert - one per token - also give the token's gate
// sigmoid(gate_vec . x): the row is being read anyway.  `shared_row0` points at the first shared expert's offset.
__global__ void pf_gather_kernel(const uint16_t* __restrict__ x, int hidden, const int* __restrict__ row_token,
                                 const int* __restrict__ ntiles, __half* __restrict__ xs,
                                 const float* __restrict__ gate_vec, const int* __restrict__ shared_row0, int T,
                                 float* __restrict__ gate) {
  const int row = blockIdx.x;
  if (row >= ntiles[1]) return;
  const int t = row_token[row];
  __half2* dst = reinterpret_cast<__half2*>(xs + (size_t)row * hidden);
  if (t < 0) {
    for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) dst[i] = __floats2half2_rn(0.f, 0.f);
    return;
  }
  const bool gated = gate_vec != nullptr && row >= shared_row0[0] && row < shared_row0[0] + T;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(x + (size_t)t * hidden);
  float dot = 0.f;
  for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) {
    const uint32_t raw = src[i];
    const float lo = __uint_as_float(raw << 16), hi = __uint_as_float(raw & 0xffff0000u);
    dst[i] = __floats2half2_rn(lo, hi);
    if (gated) {
      const float2 gv = *reinterpret_cast<const float2*>(gate_vec + 2 * i);
      dot = fmaf(gv.x, lo, dot);
      dot = fmaf(gv.y, hi, dot);
    }
  }
  if (gated) {  // block sum in a fixed order: lanes by butterfly, then the warps one after the other
    __shared__ float part[32];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = dot;
    __syncthreads();
    if (threadIdx.x == 0) {
      float sum = 0.f;
      for (int w = 0; w < (int)(blockDim.x >> 5); ++w) sum += part[w];
      gate[t] = 1.f / (1.f + expf(-sum));
    }
  }
}

// ---- steps 3 and 4: the grouped GEMM on the 5th-generation tensor cores ---------------------------------
// One persistent CTA per SM walks work items (128 weight rows x 128 token rows) and computes the transposed
// product D[weight row, token].  Per 64-column step of the contraction:
//   - the load warp brings the token tile (rows of x or h, fp16) into shared memory with one TMA tiled copy,
//     128-byte swizzle: the B operand;
//   - the dequantisation warps (sets of four, taking the steps in turn) build from the nibble planes and
//     zero-points the integer d = q - zp (or 16 (q_msb - (zp >> 4))), exact in fp16, and multiply it by the
//     group's scale normalised by a power of two per weight row: the product is kept as p + e with p the
//     rounded fp16 product and e = fma(d, f, -p) the exact remainder, and both halves go straight into tensor
//     memory with tcgen05.st: the A operands, one weight row per lane.  Weights never pass through shared
//     memory as fp16;
//   - the MMA warp issues eight tcgen05.mma (M 128, N 128, K 16): leading parts and remainders against the
//     same tokens, all accumulating into one of two fp32 accumulators in tensor memory.
// When an item's contraction is complete its accumulator is handed to eight epilogue warps, which read it with
// tcgen05.ld and multiply each row by its power of two; meanwhile the next item accumulates in the other
// buffer.  No weight is ever rounded: p + e equals s 2^n (q - zp) exactly.  Every wait is bounded; a wait that
// runs out sets SLICEMOE_STATUS_WAIT_TIMEOUT and the CTA winds down (tensor memory is freed on every path).
constexpr int kUSets = 2;           // dequantisation sets of four warps; the steps go round them
constexpr int kUWarpTma = 8 + 4 * kUSets, kUWarpMma = kUWarpTma + 1;
constexpr int kUThreads = 32 * (kUWarpMma + 1);  // warps 0-7 epilogue, then the dequantisation sets, loads, MMA issue
constexpr int kUStages = 4;
constexpr int kUTileBytes = kPfTileM * kPfChunkK * 2;  // 16,384: the token tile of a step
constexpr int kUScaleSlots = 4;     // ring of per-item row scales: dequantisation is less than 4 items ahead of the epilogue
constexpr int kUScaleBytes = kUScaleSlots * kPfTileB * 4;
constexpr int kURawDepth = 3;       // steps of raw plane words each dequantisation warp keeps in flight (cp.async)
constexpr int kURawBytes = 4 * kUSets * kURawDepth * 2048;  // per warp and step: 2 blocks x 512 bytes MSB, the same of LSB
constexpr int kUXchBytes = 4 * 64 * 32 * 4;        // silu(gate) on its way from the gate warps to the up warps
constexpr int kUSmemBytes =
    kUStages * kUTileBytes + kURawBytes + kUXchBytes + kUScaleBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kUAccCols = 256;      // two accumulators of 128 fp32 columns (tokens)
constexpr int kUWCols = 64;         // a step's weights: 64 fp16 per row, twice (leading part, remainder)
constexpr int kUTmemCols = 512;     // accumulators + kUStages weight stages, rounded up to a power of two
constexpr long long kUWaitCycles = 2000000000ll;

struct PfGemmParams {
  const slicemoe_expert* experts;  // routed
  const slicemoe_expert* shared;
  const uint8_t* expert_prec;      // per routed expert: 1 = both slices, 0 = MSB slice only
  const int* tile_expert;
  const int* tile_row0;
  const int* item_start;           // phase 1: first work item of every tile (prefix sum of its n-tiles)
  const int* ntiles;               // [0] tiles, [1] rows, [2] phase-1 work items
  __half* h;                       // phase 1 output, phase 2 A operand [rows, ldh]
  float* yrow;                     // phase 2 output [rows, hidden]
  unsigned* status;
  int E, hidden, inter, shared_inter, ldh;
  int shift;  // b_high - b_low
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
// Bounded wait for the phase of the given parity; false when the limit ran out or another role gave up.
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok)
               : "r"(smem_u32(b)), "r"(parity)
               : "memory");
  return ok != 0;
}
__device__ __noinline__ bool mbar_wait_slow(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try(b, parity)) return true;
    if (*abort_flag || clock64() - t0 > kUWaitCycles) return false;
  }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(b, parity)) return true;  // the common case costs one instruction
  return mbar_wait_slow(b, parity, abort_flag);
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_but() {  // all but the N most recent groups have landed
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);  // start address / 16
  d |= (uint64_t)1 << 16;                   // leading byte offset (unused with swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset / 16
  d |= (uint64_t)1 << 46;                   // descriptor version
  d |= (uint64_t)2 << 61;                   // 128-byte swizzle
  return d;
}
// Instruction descriptor: fp16 x fp16 -> fp32, both operands K-major, M 128, N 128.
constexpr uint32_t kUmmaIdesc = (1u << 4) | ((uint32_t)(kPfTileB >> 3) << 17) | ((uint32_t)(kPfTileM >> 4) << 24);

// D (tensor memory) (+)= A (tensor memory: lane = row, 32-bit column = two consecutive k) x B (shared memory).
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b), "r"(kUmmaIdesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Byte offset of element (row, k) in a swizzled [128][64] fp16 tile (k a multiple of 4 here).
__device__ __forceinline__ uint32_t swz128(int row, int k) {
  return (uint32_t)(row * 128 + ((((k >> 3) ^ (row & 7)) << 4) | ((k & 7) << 1)));
}

// What a work item is: which tile of token rows, which 128 weight rows of which expert.
struct UItem {
  const slicemoe_expert* ex;
  int row0, nt, K;
  bool prec;     // both slices (else the MSB slice alone)
  bool missing;  // both slices were asked for but the LSB planes are absent
};
template <int PHASE>
__device__ __forceinline__ int u_item_count(const PfGemmParams& p) {
  return PHASE == 1 ? p.ntiles[2] : p.ntiles[0] * (p.hidden / 128);
}
template <int PHASE>
__device__ __forceinline__ UItem u_item(const PfGemmParams& p, int item) {
  int tile, nt;
  if (PHASE == 1) {
    // routed tiles first, inter / 64 items each, then the shared experts' tiles with shared_inter / 64 items each
    const int per_r = p.inter / 64, routed_items = p.ntiles[3] * per_r;
    if (item < routed_items) {
      tile = item / per_r;
      nt = item - tile * per_r;
    } else {
      const int per_s = p.shared_inter / 64, rest = item - routed_items;
      tile = p.ntiles[3] + rest / per_s;
      nt = rest - (rest / per_s) * per_s;
    }
  } else {
    const int per = p.hidden / 128;
    tile = item / per;
    nt = item - tile * per;
  }
  UItem it;
  const int e = p.tile_expert[tile];
  const bool is_shared = e >= p.E;
  it.ex = is_shared ? p.shared + (e - p.E) : p.experts + e;
  it.row0 = p.tile_row0[tile];
  it.nt = nt;
  it.K = PHASE == 1 ? p.hidden : (is_shared ? p.shared_inter : p.inter);
  it.prec = is_shared ? true : (p.expert_prec[e] != 0);
  const bool has_lsb = PHASE == 1 ? (it.ex->gate.lsb && it.ex->up.lsb) : (it.ex->down.lsb != nullptr);
  it.missing = it.prec && !has_lsb;
  if (it.missing) it.prec = false;
  return it;
}
// Weight row block (16 rows) that row block rbk (0..7) of an item's 128 weight rows holds.  First GEMM: rows
// [0,64) are gate rows of h columns [64 nt, 64 nt + 64), rows [64,128) the up rows of the same columns.
template <int PHASE>
__device__ __forceinline__ const slicemoe_mat& u_block_mat(const UItem& it, int rbk, int* rb) {
  if (PHASE == 1) {
    *rb = it.nt * 4 + (rbk & 3);
    return rbk < 4 ? it.ex->gate : it.ex->up;
  }
  *rb = it.nt * 8 + rbk;
  return it.ex->down;
}

template <int G, int PHASE>
__global__ void __launch_bounds__(kUThreads, 1) pf_umma_kernel(const PfGemmParams p, const __grid_constant__ CUtensorMap tm_tok) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  extern __shared__ uint8_t u_smem_raw[];
  uint8_t* smem = u_smem_raw + ((1024 - (smem_u32(u_smem_raw) & 1023)) & 1023);
  uint8_t* raw_ring = smem + kUStages * kUTileBytes;
  float(*xch)[64][32] = reinterpret_cast<float(*)[64][32]>(raw_ring + kURawBytes);  // [pair][token][row]
  float(*row_scale)[kPfTileB] = reinterpret_cast<float(*)[kPfTileB]>(raw_ring + kURawBytes + kUXchBytes);  // [item % 4][row]
  uint64_t* bars = reinterpret_cast<uint64_t*>(raw_ring + kURawBytes + kUXchBytes + kUScaleBytes);
  uint64_t* full = bars;                    // [stage]: tokens landed (TMA) and weights stored (8 warps)
  uint64_t* empty = bars + kUStages;        // [stage]: the MMAs that read the stage have completed
  uint64_t* acc_full = bars + 2 * kUStages;       // [2]: an item's sums are complete in the accumulator
  uint64_t* acc_empty = bars + 2 * kUStages + 2;  // [2]: the epilogue warps have read it
  uint64_t* xch_full = bars + 2 * kUStages + 4;   // [4]: silu(gate) of a warp pair is in shared memory
  uint64_t* xch_empty = bars + 2 * kUStages + 8;  // [4]: it has been consumed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kUStages + 12);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  // the warp index by way of a shuffle: the compiler then knows that it is uniform across the warp, and keeps
  // the role branches and what they compute (addresses, descriptors, counters) on the uniform datapath
  const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kUStages; ++s) {
      mbar_init(&full[s], 5);  // the set's four dequantisation warps and the load warp
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 8);
    }
    for (int a = 0; a < 4; ++a) {
      mbar_init(&xch_full[a], 1);
      mbar_init(&xch_empty[a], 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kUWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kUTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_items = u_item_count<PHASE>(p);
  bool alive = true;

  if (warp == kUWarpTma) {
    // ---- token tiles: one TMA copy per step ----
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      // the next item's description is fetched while this item's copies go out
      UItem w{};
      if ((int)blockIdx.x < n_items) w = u_item<PHASE>(p, blockIdx.x);
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        UItem wn = w;
        if (item + (int)gridDim.x < n_items) wn = u_item<PHASE>(p, item + gridDim.x);
        const int nk = w.K / kPfChunkK;
        for (int kc = 0; kc < nk; ++kc) {
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { alive = false; break; }
          mbar_expect_tx(&full[s], kUTileBytes);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                  smem_u32(smem + s * kUTileBytes)),
              "l"(&tm_tok), "r"(smem_u32(&full[s])), "r"(kc * kPfChunkK), "r"(w.row0)
              : "memory");
          if (++s == kUStages) { s = 0; ph ^= 1; }
        }
        w = wn;
      }
    }
  } else if (warp == kUWarpMma) {
    // ---- MMA issue: D[weight row, token] += W[weight row, k] (tensor memory) x X[token, k] (shared memory) ----
    // The whole warp walks the loop (waits included) so that its bookkeeping stays uniform; lane 0 issues.
    uint32_t st = 0, ph = 0, ni = 0;  // stage, its parity, items issued so far
    uint64_t* last_empty = nullptr;
    uint32_t last_ph = 0;
    const uint64_t bd0 = umma_desc(smem_u32(smem));
    UItem w{};
      if ((int)blockIdx.x < n_items) w = u_item<PHASE>(p, blockIdx.x);
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++ni) {
      UItem wn = w;
      if (item + (int)gridDim.x < n_items) wn = u_item<PHASE>(p, item + gridDim.x);
      const int nk = w.K / kPfChunkK;
      const uint32_t ab = ni & 1;
      // the accumulator must have been read out (the item before the previous one used it)
      if (!__all_sync(0xffffffffu, mbar_wait(&acc_empty[ab], ((ni >> 1) & 1) ^ 1, abort_flag))) { alive = false; break; }
      tc_fence_after();
      for (int kc = 0; kc < nk; ++kc) {
        if (!__all_sync(0xffffffffu, mbar_wait(&full[st], ph, abort_flag))) { alive = false; break; }
        tc_fence_after();
        const uint64_t bd = bd0 + (uint64_t)(st * (kUTileBytes >> 4));
        const uint32_t a_tmem = tmem + kUAccCols + st * kUWCols;
        if (lane == 0) {
#pragma unroll
          for (int ks = 0; ks < kPfChunkK / 16; ++ks) {
            // leading part and remainder of the weights against the same tokens
            umma_f16_ts(tmem + ab * kPfTileM, a_tmem + 8 * ks, bd + 2 * ks, (kc | ks) ? 1u : 0u);
            umma_f16_ts(tmem + ab * kPfTileM, a_tmem + 32 + 8 * ks, bd + 2 * ks, 1u);
          }
          umma_commit(&empty[st]);
        }
        __syncwarp();
        last_empty = &empty[st];
        last_ph = ph;
        if (++st == kUStages) { st = 0; ph ^= 1; }
      }
      if (!alive) break;
      if (lane == 0) umma_commit(&acc_full[ab]);
      __syncwarp();
      w = wn;
    }
    // the last commit must have arrived before shared memory goes away
    if (alive && last_empty && !__all_sync(0xffffffffu, mbar_wait(last_empty, last_ph, abort_flag))) alive = false;
  } else if (warp >= 8) {
    // ---- dequantisation: sets of four warps take the 64-column steps in turn; thread (q, lane) of a set owns
    // weight row 32 q + lane and stores the row's 64 values of the step, as leading parts and remainders,
    // into the stage's tensor-memory columns ----
    const int q = warp & 3, set = (warp - 8) >> 2;
    const int blk = lane >> 4, g = lane & 7, sh = ((lane >> 3) & 1) * 4;  // row = 16 (2 q + blk) + g + 8 (sh / 4)
    constexpr int kGpc = G == 32 ? 2 : 1;  // quantisation groups in a step
    // Raw plane words run kURawDepth of the warp's steps ahead of their use, across work items.  Per step the
    // warp needs two 16-row blocks of 512 bytes per plane; lane l copies the 16 bytes of plane lane l of both
    // blocks with cp.async into the warp's ring (16-byte pieces XOR-swizzled against bank conflicts), and
    // after a warp barrier every lane reads the four pieces of its row.
    uint8_t* raw = raw_ring + (warp - 8) * (kURawDepth * 2048);
    const int wr_piece = (lane ^ (lane >> 3)) * 16;  // plane lane l = 4 g' + c: low two bits XOR (g' >> 1)
    // Step c of the CTA (counted over all its items) belongs to set c mod kUSets and to stage c mod kUStages.
    auto first_kc = [&](uint32_t base) { return (int)((set + kUSets - base % kUSets) % kUSets); };
    uint32_t i_base = 0;  // steps of the items before the one the copies are in
    int i_item = blockIdx.x, i_kc = set, i_nk = 0;
    const uint8_t *i_mp = nullptr, *i_lp = nullptr;
    bool i_prec = false;
    auto i_open = [&]() {
      if (i_item >= n_items) return;
      const UItem w = u_item<PHASE>(p, i_item);
      int rb;
      const slicemoe_mat& m = u_block_mat<PHASE>(w, 2 * q, &rb);  // blocks 2 q and 2 q + 1 are neighbours in one matrix
      i_nk = w.K / kPfChunkK;
      i_prec = w.prec;
      i_mp = reinterpret_cast<const uint8_t*>(m.msb) + (size_t)rb * i_nk * 512 + lane * 16;
      i_lp = w.prec ? reinterpret_cast<const uint8_t*>(m.lsb) + (size_t)rb * i_nk * 512 + lane * 16 : i_mp;
    };
    auto i_issue = [&](int slot) {
      if (i_item < n_items) {
        uint8_t* dst = raw + slot * 2048 + wr_piece;
        const size_t o = (size_t)i_kc * 512, o1 = o + (size_t)i_nk * 512;
        cp_async16(dst, i_mp + o);
        cp_async16(dst + 512, i_mp + o1);
        if (i_prec) {
          cp_async16(dst + 1024, i_lp + o);
          cp_async16(dst + 1536, i_lp + o1);
        }
        i_kc += kUSets;
        if (i_kc >= i_nk) {
          i_base += i_nk;
          i_item += gridDim.x;
          i_kc = first_kc(i_base);
          i_open();
        }
      }
      cp_async_commit();
    };
    i_open();
    for (int j = 0; j < kURawDepth; ++j) i_issue(j);
    uint32_t base = 0, slot = 0, ni = 0;  // steps of the items so far; ring slot of the raw words; items so far
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++ni) {
      const UItem w = u_item<PHASE>(p, item);
      int rb;
      const slicemoe_mat& m = u_block_mat<PHASE>(w, 2 * q + blk, &rb);
      if (w.missing && warp == 8 && lane == 0) atomicOr(p.status, (unsigned)SLICEMOE_STATUS_MISSING_LSB);
      const int nk = w.K / kPfChunkK, ngroups = w.K >> LG;
      const size_t meta = (size_t)rb * ngroups * 16 + g + 2 * sh;  // the row's entry of group 0
      const uint8_t* zp = m.zp + meta;
      const uint16_t* sc = m.scale + meta;
      // The row's weights are normalised by a power of two, 2^(emax - 15) with emax the largest exponent field
      // among the row's fp16 scales: every factor f = s 2^(15 - emax) is below 2, so |(q - zp) f| < 512 sits in
      // the middle of fp16's range for the leading part and its remainder alike.  The epilogue multiplies the
      // row's sums by 2^(emax - 15).
      unsigned emax = 0;
      for (int grp = 0; grp < ngroups; ++grp) emax = max(emax, ((unsigned)__ldg(sc + grp * 16) >> 10) & 31u);
      const float rnorm = exp2f(15.f - (float)emax);
      if (set == 0) row_scale[ni % kUScaleSlots][32 * q + lane] = exp2f((float)emax - 15.f);
      // zero-points and scales of the groups of the warp's next step
      const int kc0 = first_kc(base);
      int z_next[kGpc];
      uint16_t s_next[kGpc];
#pragma unroll
      for (int i = 0; i < kGpc; ++i) {
        const int grp = ((kc0 * kPfChunkK) >> LG) + i;
        z_next[i] = __ldg(zp + grp * 16);
        s_next[i] = __ldg(sc + grp * 16);
      }
      for (int kc = kc0; kc < nk; kc += kUSets) {
        const uint32_t st = (base + kc) % kUStages, ph = ((base + kc) / kUStages) & 1;
        cp_async_wait_but<kURawDepth - 1>();
        __syncwarp();
        const uint8_t* src = raw + slot * 2048 + blk * 512 + g * 64;
        const int rsw = (g >> 1) * 16;  // piece c sits at 16 (c ^ (g >> 1))
        uint32_t mws[16], lws[16];      // [4 c + w]: word w of plane lane 4 g + c: k = 16 w + 4 c + j
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint4 mv = *reinterpret_cast<const uint4*>(src + ((16 * c) ^ rsw));
          mws[4 * c] = mv.x; mws[4 * c + 1] = mv.y; mws[4 * c + 2] = mv.z; mws[4 * c + 3] = mv.w;
          uint4 lv = make_uint4(0, 0, 0, 0);
          if (w.prec) lv = *reinterpret_cast<const uint4*>(src + 1024 + ((16 * c) ^ rsw));
          lws[4 * c] = lv.x; lws[4 * c + 1] = lv.y; lws[4 * c + 2] = lv.z; lws[4 * c + 3] = lv.w;
        }
        __half2 off[kGpc], fac[kGpc];
#pragma unroll
        for (int i = 0; i < kGpc; ++i) {
          off[i] = __half2half2(__int2half_rn(1024 + (w.prec ? z_next[i] : ((z_next[i] >> p.shift) << p.shift))));
          fac[i] = __half2half2(__float2half_rn(__half2float(__ushort_as_half(s_next[i])) * rnorm));  // exact: a power of two
        }
        if (kc + kUSets < nk) {
#pragma unroll
          for (int i = 0; i < kGpc; ++i) {
            const int grp = (((kc + kUSets) * kPfChunkK) >> LG) + i;
            z_next[i] = __ldg(zp + grp * 16);
            s_next[i] = __ldg(sc + grp * 16);
          }
        }
        if (!__all_sync(0xffffffffu, mbar_wait(&empty[st], ph ^ 1, abort_flag))) { alive = false; break; }
        tc_fence_after();
        const uint32_t ta = tmem + ((uint32_t)(32 * q) << 16) + kUAccCols + st * kUWCols;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t rh[16], rl[16];  // column 8 (w & 1) + 2 c + jj holds k = 16 w + 4 c + 2 jj, + 1 for w = 2 half, 2 half + 1
#pragma unroll
          for (int wi = 0; wi < 2; ++wi) {
            const int wd = 2 * half + wi;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const uint32_t m0 = mws[4 * c + wd] >> sh, l0 = lws[4 * c + wd] >> sh;
              // both slices: the whole code; MSB slice alone: 2^shift x its code (the factor of the low-bit
              // dequantisation, exact in fp16).  shift = 4 for 8-bit codes; narrower slices sit in the low bits
              // of their nibbles, so a code never exceeds a byte
              const uint32_t qv = ((m0 & 0x0f0f0f0fu) << p.shift) | (l0 & 0x0f0f0f0fu);
              // bytes -> fp16 1024 + code, minus (1024 + zero-point): the integer d = q - zp, exact
              uint32_t h01 = __byte_perm(qv, 0x64646464u, 0x4140), h23 = __byte_perm(qv, 0x64646464u, 0x4342);
              const __half2 o = off[kGpc == 2 ? (wd >> 1) : 0], f = fac[kGpc == 2 ? (wd >> 1) : 0];
              const __half2 d01 = __hsub2(*reinterpret_cast<__half2*>(&h01), o);
              const __half2 d23 = __hsub2(*reinterpret_cast<__half2*>(&h23), o);
              // d f as an unevaluated sum of two fp16: the rounded product and, by one fused multiply-add, what
              // the rounding dropped (at most 10 significant bits, so it is exact)
              const __half2 p01 = __hmul2(d01, f), p23 = __hmul2(d23, f);
              const __half2 e01 = __hfma2(d01, f, __hneg2(p01)), e23 = __hfma2(d23, f, __hneg2(p23));
              rh[8 * wi + 2 * c] = *reinterpret_cast<const uint32_t*>(&p01);
              rh[8 * wi + 2 * c + 1] = *reinterpret_cast<const uint32_t*>(&p23);
              rl[8 * wi + 2 * c] = *reinterpret_cast<const uint32_t*>(&e01);
              rl[8 * wi + 2 * c + 1] = *reinterpret_cast<const uint32_t*>(&e23);
            }
          }
          tmem_st16(ta + 16 * half, rh);
          tmem_st16(ta + 32 + 16 * half, rl);
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[st]);
        i_issue(slot);  // after the step's words were consumed by every lane: the slot is free
        if (++slot == kURawDepth) slot = 0;
      }
      base += nk;
    }
    cp_async_wait_but<0>();
  } else {
    // ---- epilogue: warp (q, hh) owns weight rows [32 q, 32 q + 32) x tokens [64 hh, 64 hh + 64) ----
    const int q = warp & 3, hh = warp >> 2;
    uint32_t n_done = 0;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++n_done) {
      const UItem w = u_item<PHASE>(p, item);
      const uint32_t ab = n_done & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[ab], (n_done >> 1) & 1, abort_flag))) { alive = false; break; }
      tc_fence_after();
      const float rs = row_scale[n_done % kUScaleSlots][32 * q + lane];  // 2^(emax - 15) of the lane's weight row
      const uint32_t ta = tmem + ((uint32_t)(32 * q) << 16) + ab * kPfTileM + 64 * hh;
      float tot[64];
      {
        uint32_t r0[16], r1[16];
        tmem_ld16(ta, r0);
        tmem_ld16(ta + 16, r1);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) tot[j] = rs * __uint_as_float(r0[j]);
#pragma unroll
        for (int j = 0; j < 16; ++j) tot[16 + j] = rs * __uint_as_float(r1[j]);
        tmem_ld16(ta + 32, r0);
        tmem_ld16(ta + 48, r1);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[ab]);  // the accumulator is free for the item after the next
#pragma unroll
        for (int j = 0; j < 16; ++j) tot[32 + j] = rs * __uint_as_float(r0[j]);
#pragma unroll
        for (int j = 0; j < 16; ++j) tot[48 + j] = rs * __uint_as_float(r1[j]);
      }
      if (!alive) break;
      const int tok0 = w.row0 + 64 * hh;
      if (PHASE == 1) {
        // rows [0,64) hold gate, rows [64,128) up: warp (q, hh) with q < 2 hands silu(gate) to warp (q + 2, hh)
        // through shared memory; that warp multiplies and writes h
        const int pair = 2 * hh + (q & 1);
        if (q < 2) {
          if (!__all_sync(0xffffffffu, mbar_wait(&xch_empty[pair], (n_done & 1) ^ 1, abort_flag))) { alive = false; break; }
#pragma unroll
          for (int j = 0; j < 64; ++j) xch[pair][j][lane] = tot[j] / (1.f + __expf(-tot[j]));
          __syncwarp();
          if (lane == 0) mbar_arrive(&xch_full[pair]);
        } else {
          if (!__all_sync(0xffffffffu, mbar_wait(&xch_full[pair], n_done & 1, abort_flag))) { alive = false; break; }
          __half* dst = p.h + (size_t)tok0 * p.ldh + 64 * w.nt + 32 * (q & 1) + lane;
#pragma unroll
          for (int j = 0; j < 64; ++j) dst[(size_t)j * p.ldh] = __float2half_rn(xch[pair][j][lane] * tot[j]);
          __syncwarp();
          if (lane == 0) mbar_arrive(&xch_empty[pair]);
        }
      } else {
        float* dst = p.yrow + (size_t)tok0 * p.hidden + 128 * w.nt + 32 * q + lane;
#pragma unroll
        for (int j = 0; j < 64; ++j) dst[(size_t)j * p.hidden] = tot[j];
      }
    }
  }
  if (!alive) {
    *abort_flag = 1;
    if (lane == 0) atomicOr(p.status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kUWarpMma) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kUTmemCols) : "memory");
  }
}

// ---- step 5: weighted combine in list order ---------------------------------------------------------------
__global__ void pf_combine_kernel(const float* __restrict__ yrow, const int* __restrict__ posmap,
                                  const float* __restrict__ weights, const float* __restrict__ gate, int T, int k,
                                  int n_shared, int hidden, float* __restrict__ y) {
  const int t = blockIdx.x;
  const int slots = k + n_shared;
  for (int col = threadIdx.x * 4; col < hidden; col += blockDim.x * 4) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < slots; ++j) {
      const int pos = posmap[t * slots + j];
      if (pos < 0) continue;
      const float w = j < k ? weights[t * k + j] : (gate ? gate[t] : 1.f);
      const float4 v = *reinterpret_cast<const float4*>(yrow + (size_t)pos * hidden + col);
      a.x = fmaf(w, v.x, a.x);
      a.y = fmaf(w, v.y, a.y);
      a.z = fmaf(w, v.z, a.z);
      a.w = fmaf(w, v.w, a.w);
    }
    *reinterpret_cast<float4*>(y + (size_t)t * hidden + col) = a;
  }
}

typedef CUresult (*PfEncodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of a row-major fp16 matrix [rows, cols] for 128-row x 64-column tiles with 128-byte swizzle.
static int pf_tensor_map(CUtensorMap* tm, const __half* base, int rows, int cols) {
  static PfEncodeTiled encode = nullptr;
  if (!encode) {
    cudaDriverEntryPointQueryResult q;
    void* fn = nullptr;
    SM_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return SLICEMOE_E_UNSUPPORTED;
    encode = reinterpret_cast<PfEncodeTiled>(fn);
  }
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * sizeof(__half)};
  const cuuint32_t box[2] = {(cuuint32_t)kPfChunkK, (cuuint32_t)kPfTileM};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(base), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SLICEMOE_OK : SLICEMOE_E_INVALID_ARG;
}

template <int G>
static int pf_launch_gemms(const PfGemmParams& p, const __half* xs, int rmax, cudaStream_t st) {
  static bool attr_set[64];
  static int sm_count[64];
  int dev = 0;
  SM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SLICEMOE_E_UNSUPPORTED;
  if (!attr_set[dev]) {
    SM_CUDA_TRY(cudaFuncSetAttribute(pf_umma_kernel<G, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUSmemBytes));
    SM_CUDA_TRY(cudaFuncSetAttribute(pf_umma_kernel<G, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUSmemBytes));
    SM_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    attr_set[dev] = true;
  }
  CUtensorMap tm_x, tm_h;
  int rc = pf_tensor_map(&tm_x, xs, rmax, p.hidden);
  if (rc != SLICEMOE_OK) return rc;
  rc = pf_tensor_map(&tm_h, p.h, rmax, p.ldh);
  if (rc != SLICEMOE_OK) return rc;
  // one persistent CTA per SM (shared memory admits one); each walks its share of the work items
  pf_umma_kernel<G, 1><<<sm_count[dev], kUThreads, kUSmemBytes, st>>>(p, tm_x);
  SM_LAUNCH_CHECK();
  pf_umma_kernel<G, 2><<<sm_count[dev], kUThreads, kUSmemBytes, st>>>(p, tm_h);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

static int pf_check(const slicemoe_shape* s, int T) {
  if (!s || T <= 0) return SLICEMOE_E_INVALID_ARG;
  if (!valid_widths(s->b_high, s->b_low)) return SLICEMOE_E_UNSUPPORTED;
  if (!valid_group(s->group)) return SLICEMOE_E_UNSUPPORTED;
  if (s->hidden <= 0 || s->inter <= 0 || s->n_experts <= 0 || s->top_k < 1) return SLICEMOE_E_INVALID_ARG;
  if (s->top_k > s->n_experts || s->top_k > SLICEMOE_MAX_TOP_K) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared < 0 || s->n_shared > SLICEMOE_MAX_SHARED) return SLICEMOE_E_INVALID_ARG;
  if ((s->hidden % 128) || (s->inter % 128)) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && (s->shared_inter <= 0 || (s->shared_inter % 128))) return SLICEMOE_E_INVALID_ARG;
  if ((long long)T * (s->top_k + s->n_shared) > (1ll << 28)) return SLICEMOE_E_UNSUPPORTED;
  return SLICEMOE_OK;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" size_t slicemoe_prefill_workspace_bytes(const slicemoe_shape* s, int T) {
  if (pf_check(s, T) != SLICEMOE_OK) return 0;
  return pf_layout(T, s->n_experts, s->top_k, s->n_shared, s->hidden, s->inter, s->n_shared ? s->shared_inter : 0).total;
}

extern "C" int slicemoe_prefill_layer(const slicemoe_shape* s, const slicemoe_expert* experts,
                                      const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                                      const int32_t* ids, const float* weights, const uint8_t* expert_prec, float* y,
                                      void* workspace, size_t workspace_bytes, int* status_out_device, void* stream) {
  int rc = pf_check(s, T);
  if (rc != SLICEMOE_OK) return rc;
  if (!experts || !x || !ids || !weights || !expert_prec || !y || !workspace || !status_out_device)
    return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && !shared) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && s->shared_sigmoid_gate && !shared_gate_vec) return SLICEMOE_E_INVALID_ARG;
  const int nsh = s->n_shared, E = s->n_experts, k = s->top_k;
  const int shared_inter = nsh ? s->shared_inter : 0;
  const PfLayout L = pf_layout(T, E, k, nsh, s->hidden, s->inter, shared_inter);
  if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SLICEMOE_E_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 3) || (reinterpret_cast<uintptr_t>(y) & 15)) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && s->shared_sigmoid_gate && (reinterpret_cast<uintptr_t>(shared_gate_vec) & 7))
    return SLICEMOE_E_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  int* counts = reinterpret_cast<int*>(ws + L.counts);
  int* cursor = reinterpret_cast<int*>(ws + L.cursor);
  int* offsets = reinterpret_cast<int*>(ws + L.offsets);
  int* tile_expert = reinterpret_cast<int*>(ws + L.tile_expert);
  int* tile_row0 = reinterpret_cast<int*>(ws + L.tile_row0);
  int* item_start = reinterpret_cast<int*>(ws + L.item_start);
  int* ntiles = reinterpret_cast<int*>(ws + L.ntiles);
  int* row_token = reinterpret_cast<int*>(ws + L.row_token);
  int* posmap = reinterpret_cast<int*>(ws + L.posmap);
  float* gate = reinterpret_cast<float*>(ws + L.gate);
  __half* xs = reinterpret_cast<__half*>(ws + L.xs);
  __half* h = reinterpret_cast<__half*>(ws + L.h);
  float* yrow = reinterpret_cast<float*>(ws + L.yrow);

  // counters start at zero, unused rows are marked -1
  SM_CUDA_TRY(cudaMemsetAsync(ws + L.counts, 0, L.offsets - L.counts, st));
  SM_CUDA_TRY(cudaMemsetAsync(row_token, 0xff, sizeof(int) * (size_t)L.rmax, st));
  SM_CUDA_TRY(cudaMemsetAsync(status_out_device, 0, sizeof(int), st));
  const int npairs = T * k;
  pf_count_kernel<<<(npairs + 255) / 256, 256, 0, st>>>(ids, npairs, E, counts, reinterpret_cast<unsigned*>(status_out_device));
  SM_LAUNCH_CHECK();
  pf_scan_kernel<<<1, 32, 0, st>>>(counts, E, nsh, T, s->inter, shared_inter, offsets, tile_expert, tile_row0, item_start, ntiles);
  SM_LAUNCH_CHECK();
  const int nslots = T * (k + nsh);
  pf_scatter_kernel<<<(nslots + 255) / 256, 256, 0, st>>>(ids, T, k, E, nsh, offsets, cursor, row_token, posmap);
  SM_LAUNCH_CHECK();
  const bool gated = nsh > 0 && s->shared_sigmoid_gate;
  pf_gather_kernel<<<L.rmax, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), s->hidden, row_token, ntiles, xs,
                                           gated ? shared_gate_vec : nullptr, offsets + E, T, gate);
  SM_LAUNCH_CHECK();
  PfGemmParams p;
  p.experts = experts;
  p.shared = shared;
  p.expert_prec = expert_prec;
  p.tile_expert = tile_expert;
  p.tile_row0 = tile_row0;
  p.item_start = item_start;
  p.ntiles = ntiles;
  p.h = h;
  p.yrow = yrow;
  p.status = reinterpret_cast<unsigned*>(status_out_device);
  p.E = E;
  p.hidden = s->hidden;
  p.inter = s->inter;
  p.shared_inter = shared_inter;
  p.ldh = s->inter > shared_inter ? s->inter : shared_inter;
  p.shift = s->b_high - s->b_low;
  if (s->group == 128) {
    rc = pf_launch_gemms<128>(p, xs, L.rmax, st);
  } else if (s->group == 64) {
    rc = pf_launch_gemms<64>(p, xs, L.rmax, st);
  } else {
    rc = pf_launch_gemms<32>(p, xs, L.rmax, st);
  }
  if (rc != SLICEMOE_OK) return rc;
  pf_combine_kernel<<<T, 256, 0, st>>>(yrow, posmap, weights, gated ? gate : nullptr, T, k, nsh, s->hidden, y);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}
