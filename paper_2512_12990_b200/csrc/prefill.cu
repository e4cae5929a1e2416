// Prefill of one MoE layer from bit-sliced AMAT weights: many tokens at once, so the expert FFN is a
// genuine dense contraction (Section 3 of the paper: prefill loads every expert of a layer; Section 5.3:
// prefill runs at the precision each expert's cached slices allow).
//
// Steps, all on the device:
//   1. count the tokens of every routed expert, lay the experts' token rows out one after the other
//      (each expert padded to a multiple of 128 rows), list the 128-row tiles;
//   2. gather x (bf16) into that order as fp16 (exact for every bf16 value in fp16's normal range);
//   3. grouped GEMM 1: per tile  H = silu(X Wg^T) * (X Wu^T)  (fp16 out);
//   4. grouped GEMM 2: per tile  Yrow = H Wd^T  (fp32 out, one row per (token, expert) pair);
//   5. combine: y[t] = sum_j w[t,j] Yrow[pos(t,j)] + shared experts, in list order (deterministic).
// In both GEMMs the weight tile is dequantised on the fly from the nibble planes into fp16 in shared
// memory - s * (q - zp) from both slices, 16 s * (q_msb - (zp >> 4)) from the MSB slice alone - and fed
// to the tensor cores (mma.sync m16n8k16, fp16 x fp16 -> fp32).  fp16 rather than bf16: a dequantised
// weight needs 11 significant bits to stay inside the parity tolerance, bf16 has 8.
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

// One CTA: padded offsets of every expert (routed, then shared with T rows each) and the tile list.
__global__ void pf_scan_kernel(const int* __restrict__ counts, int E, int n_shared, int T, int inter, int shared_inter,
                               int* __restrict__ offsets, int* __restrict__ tile_expert, int* __restrict__ tile_row0,
                               int* __restrict__ item_start, int* __restrict__ ntiles) {
  if (threadIdx.x != 0) return;
  int off = 0, nt = 0, items = 0;
  for (int e = 0; e < E + n_shared; ++e) {
    const int c = e < E ? counts[e] : T;
    offsets[e] = off;
    for (int r = 0; r < c; r += kPfTileM) {
      tile_expert[nt] = e;
      tile_row0[nt] = off + r;
      item_start[nt] = items;
      items += (e < E ? inter : shared_inter) / 64;  // first GEMM: 64 columns of h per work item
      ++nt;
    }
    off += (c + kPfTileM - 1) / kPfTileM * kPfTileM;
  }
  offsets[E + n_shared] = off;
  item_start[nt] = items;
  ntiles[0] = nt;
  ntiles[1] = off;
  ntiles[2] = items;
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
__global__ void pf_gather_kernel(const uint16_t* __restrict__ x, int hidden, const int* __restrict__ row_token,
                                 const int* __restrict__ ntiles, __half* __restrict__ xs) {
  const int row = blockIdx.x;
  if (row >= ntiles[1]) return;
  const int t = row_token[row];
  __half2* dst = reinterpret_cast<__half2*>(xs + (size_t)row * hidden);
  if (t < 0) {
    for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) dst[i] = __floats2half2_rn(0.f, 0.f);
    return;
  }
  const uint32_t* src = reinterpret_cast<const uint32_t*>(x + (size_t)t * hidden);
  for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) {
    const uint32_t raw = src[i];
    dst[i] = __floats2half2_rn(__uint_as_float(raw << 16), __uint_as_float(raw & 0xffff0000u));
  }
}

// ---- steps 3 and 4: the grouped GEMM on the 5th-generation tensor cores ---------------------------------
// One persistent CTA per SM walks work items (128 token rows x 128 weight rows).  Per 64-column step of the
// contraction:
//   - the load warp brings the A tile (token rows of x or h, fp16) in with one TMA tiled copy, 128-byte swizzle;
//   - eight dequantisation warps (one per 16-row block of the weight tile) read the nibble planes and the
//     zero-points and write the INTEGER q - zp (or q_msb - (zp >> 4)), which fp16 holds exactly, into the B tile
//     in the same swizzled K-major layout;
//   - one thread issues four tcgen05.mma (M 128, N 128, K 16) that accumulate in tensor memory.
// At the end of every quantisation group the accumulator (one of two, 128 columns each) is handed to eight
// epilogue warps, which read it with tcgen05.ld, scale column n by the group's fp16 scale of weight row n in
// fp32 and add it to the running result in registers; meanwhile the next group accumulates in the other
// buffer.  No weight is ever rounded.  Every wait is bounded; a wait that runs out sets
// SLICEMOE_STATUS_WAIT_TIMEOUT and the CTA winds down (tensor memory is freed on every path).
constexpr int kUThreads = 576;      // warps 0-7 epilogue, 8-15 dequantisation, 16 loads, 17 MMA issue
constexpr int kUStages = 6;
constexpr int kUTileBytes = kPfTileM * kPfChunkK * 2;  // 16,384: one operand tile of a step
constexpr int kUStageBytes = 2 * kUTileBytes;
constexpr int kUScaleSlots = 16;    // ring of per-group scale rows: dequantisation runs at most 15 groups ahead of the epilogue
constexpr int kUScaleBytes = kUScaleSlots * kPfTileB * 4;
constexpr int kUSmemBytes = kUStages * kUStageBytes + kUScaleBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kUTmemCols = 256;     // two accumulators of 128 fp32 columns
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
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(b)), "r"(parity)
                 : "memory");
    if (ok) return true;
    if (*abort_flag || clock64() - t0 > kUWaitCycles) return false;
  }
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

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(kUmmaIdesc), "r"(acc)
      : "memory");
}
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
    int lo = 0, hi = p.ntiles[0];  // last tile whose first item is <= item
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (p.item_start[mid] <= item) lo = mid; else hi = mid;
    }
    tile = lo;
    nt = item - p.item_start[lo];
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
// Weight row block (16 rows) that row block rbk (0..7) of an item's B tile holds.  Phase 1 interleaves gate and
// up so that each half of the accumulator columns holds 32 gate columns of h and the matching 32 up columns:
// B rows [0,32) gate, [32,64) up, [64,96) gate, [96,128) up.
template <int PHASE>
__device__ __forceinline__ const slicemoe_mat& u_block_mat(const UItem& it, int rbk, int* rb) {
  if (PHASE == 1) {
    const int half = rbk >> 2, sub = rbk & 3;
    *rb = it.nt * 4 + 2 * half + (sub & 1);
    return sub < 2 ? it.ex->gate : it.ex->up;
  }
  *rb = it.nt * 8 + rbk;
  return it.ex->down;
}

template <int G, int PHASE>
__global__ void __launch_bounds__(kUThreads, 1) pf_umma_kernel(const PfGemmParams p, const __grid_constant__ CUtensorMap tm_a) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  constexpr int kStepsPerGroup = G / 16;  // k16 MMA steps per quantisation group
  extern __shared__ uint8_t u_smem_raw[];
  uint8_t* smem = u_smem_raw + ((1024 - (smem_u32(u_smem_raw) & 1023)) & 1023);
  float(*sc_ring)[kPfTileB] = reinterpret_cast<float(*)[kPfTileB]>(smem + kUStages * kUStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kUStages * kUStageBytes + kUScaleBytes);
  uint64_t* full = bars;                    // [stage]: A landed (TMA) and B written (8 warps)
  uint64_t* empty = bars + kUStages;        // [stage]: the MMAs that read the stage have completed
  uint64_t* acc_full = bars + 2 * kUStages;       // [2]: a group's sums are complete in the accumulator
  uint64_t* acc_empty = bars + 2 * kUStages + 2;  // [2]: the epilogue warps have read it
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kUStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kUStages; ++s) {
      mbar_init(&full[s], 9);
      mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&acc_full[a], 1);
      mbar_init(&acc_empty[a], 8);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 17) {
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

  if (warp == 16) {
    // ---- A tiles: one TMA copy per step ----
    if (lane == 0) {
      uint32_t it = 0;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        const UItem w = u_item<PHASE>(p, item);
        const int nk = w.K / kPfChunkK;
        for (int kc = 0; kc < nk; ++kc, ++it) {
          const int s = it % kUStages;
          if (!mbar_wait(&empty[s], ((it / kUStages) & 1) ^ 1, abort_flag)) { alive = false; break; }
          mbar_expect_tx(&full[s], kUTileBytes);
          asm volatile(
              "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                  smem_u32(smem + s * kUStageBytes)),
              "l"(&tm_a), "r"(smem_u32(&full[s])), "r"(kc * kPfChunkK), "r"(w.row0)
              : "memory");
        }
      }
    }
  } else if (warp == 17) {
    // ---- MMA issue ----
    if (lane == 0) {
      uint32_t it = 0, gc = 0;  // steps and quantisation groups issued so far
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        const UItem w = u_item<PHASE>(p, item);
        const int nk = w.K / kPfChunkK;
        int step = 0;
        for (int kc = 0; kc < nk && alive; ++kc, ++it) {
          const int s = it % kUStages;
          if (!mbar_wait(&full[s], (it / kUStages) & 1, abort_flag)) { alive = false; break; }
          tc_fence_after();
          const uint64_t ad = umma_desc(smem_u32(smem + s * kUStageBytes));
          const uint64_t bd = umma_desc(smem_u32(smem + s * kUStageBytes + kUTileBytes));
#pragma unroll
          for (int ks = 0; ks < kPfChunkK / 16; ++ks, ++step) {
            const int in_group = step % kStepsPerGroup;
            const uint32_t ab = gc & 1;
            if (in_group == 0) {
              // first step of a group: the accumulator must have been read out
              if (!mbar_wait(&acc_empty[ab], ((gc >> 1) & 1) ^ 1, abort_flag)) { alive = false; break; }
              tc_fence_after();
            }
            umma_f16(tmem + ab * kPfTileB, ad + 2 * ks, bd + 2 * ks, in_group ? 1u : 0u);
            if (in_group == kStepsPerGroup - 1) {
              umma_commit(&acc_full[ab]);
              ++gc;
            }
          }
          umma_commit(&empty[s]);
        }
      }
      // the last commit must have arrived before shared memory goes away
      if (alive && it > 0) {
        const uint32_t last = it - 1;
        if (!mbar_wait(&empty[last % kUStages], (last / kUStages) & 1, abort_flag)) alive = false;
      }
    }
  } else if (warp >= 8) {
    // ---- dequantisation: warp d fills B rows [16 d, 16 d + 16) of every step ----
    const int d = warp - 8, g = lane >> 2, c = lane & 3;
    uint32_t it = 0, gc = 0;  // steps and quantisation groups produced so far
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const UItem w = u_item<PHASE>(p, item);
      int rb;
      const slicemoe_mat& m = u_block_mat<PHASE>(w, d, &rb);
      if (w.missing && d == 0 && lane == 0) atomicOr(p.status, (unsigned)SLICEMOE_STATUS_MISSING_LSB);
      const int nk = w.K / kPfChunkK;
      const uint4* mp = reinterpret_cast<const uint4*>(m.msb) + (size_t)rb * nk * 32 + lane;
      const uint4* lp = w.prec ? reinterpret_cast<const uint4*>(m.lsb) + (size_t)rb * nk * 32 + lane : mp;
      const uint8_t* zp = m.zp + (size_t)rb * (w.K >> LG) * 16 + g;
      const uint16_t* sc = m.scale + (size_t)rb * (w.K >> LG) * 16 + (lane & 15);
      uint4 mw = __ldg(mp), lw = w.prec ? __ldg(lp) : make_uint4(0, 0, 0, 0);
      __half2 off[2];
      for (int kc = 0; kc < nk; ++kc, ++it) {
        uint4 mw_n = mw, lw_n = lw;
        if (kc + 1 < nk) {
          mw_n = __ldg(mp + (size_t)(kc + 1) * 32);
          if (w.prec) lw_n = __ldg(lp + (size_t)(kc + 1) * 32);
        }
        if (kc + 12 < nk && (lane & 7) == 0) {
          asm volatile("prefetch.global.L2 [%0];" ::"l"(mp + (size_t)(kc + 12) * 32));
          if (w.prec) asm volatile("prefetch.global.L2 [%0];" ::"l"(lp + (size_t)(kc + 12) * 32));
        }
        const int s = it % kUStages;
        uint8_t* bs = smem + s * kUStageBytes + kUTileBytes;
        if (!__all_sync(0xffffffffu, mbar_wait(&empty[s], ((it / kUStages) & 1) ^ 1, abort_flag))) { alive = false; break; }
        const uint32_t mws[4] = {mw.x, mw.y, mw.z, mw.w}, lws[4] = {lw.x, lw.y, lw.z, lw.w};
#pragma unroll
        for (int wd = 0; wd < 4; ++wd) {
          const int k = 16 * wd + 4 * c;
          if (G >= 64 ? (wd == 0 && ((kc * kPfChunkK) & (G - 1)) == 0) : ((wd & 1) == 0)) {
            // a new quantisation group starts: zero-points of rows g and g + 8
            const int grp = (kc * kPfChunkK + 16 * wd) >> LG;
#pragma unroll
            for (int hi = 0; hi < 2; ++hi) {
              const int z = __ldg(zp + grp * 16 + 8 * hi);
              off[hi] = __half2half2(__int2half_rn(1024 + (w.prec ? z : (z & 0xf0))));
            }
            // the group's scales of the warp's 16 rows, for the epilogue (published by the arrive below)
            if (lane < 16) sc_ring[gc % kUScaleSlots][16 * d + lane] = __half2float(__ushort_as_half(__ldg(sc + grp * 16)));
            ++gc;
          }
          const uint32_t m0 = mws[wd], l0 = lws[wd];
          // both slices: the 8-bit code; MSB slice alone: 16 x its 4-bit code (the factor 16 of the low-bit
          // dequantisation, exact in fp16)
          const uint32_t qlo = ((m0 & 0x0f0f0f0fu) << 4) | (l0 & 0x0f0f0f0fu);
          const uint32_t qhi = (m0 & 0xf0f0f0f0u) | ((l0 >> 4) & 0x0f0f0f0fu);
#pragma unroll
          for (int hi = 0; hi < 2; ++hi) {
            const uint32_t q = hi ? qhi : qlo;
            // bytes -> fp16 1024 + code, minus (1024 + zero-point): the integer q - zp (or 16 (q_msb - (zp >> 4))), exact
            uint32_t h01 = __byte_perm(q, 0x64646464u, 0x4140), h23 = __byte_perm(q, 0x64646464u, 0x4342);
            const __half2 w01 = __hsub2(*reinterpret_cast<__half2*>(&h01), off[hi]);
            const __half2 w23 = __hsub2(*reinterpret_cast<__half2*>(&h23), off[hi]);
            uint2 o;
            o.x = *reinterpret_cast<const uint32_t*>(&w01);
            o.y = *reinterpret_cast<const uint32_t*>(&w23);
            *reinterpret_cast<uint2*>(bs + swz128(16 * d + g + 8 * hi, k)) = o;
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        mw = mw_n;
        lw = lw_n;
      }
    }
  } else {
    // ---- epilogue: warp (q, hh) owns accumulator lanes [32 q, 32 q + 32) x columns [64 hh, 64 hh + 64) ----
    const int q = warp & 3, hh = warp >> 2;
    uint32_t gc = 0;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const UItem w = u_item<PHASE>(p, item);
      const int ngroups = w.K >> LG;
      float tot[64];
#pragma unroll
      for (int j = 0; j < 64; ++j) tot[j] = 0.f;
      for (int grp = 0; grp < ngroups; ++grp, ++gc) {
        const uint32_t ab = gc & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[ab], (gc >> 1) & 1, abort_flag))) { alive = false; break; }
        tc_fence_after();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t r[16];
          tmem_ld16(tmem + ((uint32_t)(32 * q) << 16) + ab * kPfTileB + 64 * hh + 16 * cc, r);
          const float4* sp = reinterpret_cast<const float4*>(&sc_ring[gc % kUScaleSlots][64 * hh + 16 * cc]);
          float sf[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) *reinterpret_cast<float4*>(&sf[4 * j]) = sp[j];
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) tot[16 * cc + j] = fmaf(sf[j], __uint_as_float(r[j]), tot[16 * cc + j]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[ab]);
      }
      if (!alive) break;
      const int row = w.row0 + 32 * q + lane;
      if (PHASE == 1) {
        // columns 0-31 of the warp's half are gate, 32-63 the matching up columns
        uint32_t hv[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float g0 = tot[2 * j], g1 = tot[2 * j + 1], u0 = tot[32 + 2 * j], u1 = tot[32 + 2 * j + 1];
          const __half2 hp = __floats2half2_rn(g0 / (1.f + __expf(-g0)) * u0, g1 / (1.f + __expf(-g1)) * u1);
          hv[j] = *reinterpret_cast<const uint32_t*>(&hp);
        }
        uint4* dst = reinterpret_cast<uint4*>(p.h + (size_t)row * p.ldh + 64 * w.nt + 32 * hh);
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j] = make_uint4(hv[4 * j], hv[4 * j + 1], hv[4 * j + 2], hv[4 * j + 3]);
      } else {
        float4* dst = reinterpret_cast<float4*>(p.yrow + (size_t)row * p.hidden + 128 * w.nt + 64 * hh);
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = make_float4(tot[4 * j], tot[4 * j + 1], tot[4 * j + 2], tot[4 * j + 3]);
      }
    }
  }
  if (!alive) {
    *abort_flag = 1;
    if (lane == 0) atomicOr(p.status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 17) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kUTmemCols) : "memory");
  }
}

// ---- step 5: weighted combine in list order ---------------------------------------------------------------
__global__ void pf_gate_kernel(const uint16_t* __restrict__ x, const float* __restrict__ gate_vec, int T, int hidden,
                               float* __restrict__ gate) {
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= T) return;
  float dot = 0.f;
  for (int i = lane; i < hidden; i += 32)
    dot = fmaf(gate_vec[i], __uint_as_float((uint32_t)x[(size_t)t * hidden + i] << 16), dot);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
  if (lane == 0) gate[t] = 1.f / (1.f + expf(-dot));
}

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
  if (s->b_high != 8 || s->b_low != 4) return SLICEMOE_E_UNSUPPORTED;
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
  pf_gather_kernel<<<L.rmax, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), s->hidden, row_token, ntiles, xs);
  SM_LAUNCH_CHECK();
  const bool gated = nsh > 0 && s->shared_sigmoid_gate;
  if (gated) {
    pf_gate_kernel<<<(T + 7) / 8, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), shared_gate_vec, T, s->hidden, gate);
    SM_LAUNCH_CHECK();
  }
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
