// Batch-1 decode of one MoE layer from bit-sliced AMAT weights (Section 4.1 of the paper: an expert
// runs from MSB+LSB slices at full precision or from the MSB slice alone), as ONE persistent kernel.
//
// The work is a pure weight stream: every plane byte is used once, so the bound is HBM bandwidth and
// everything else is arranged so that the stream never stops.
//   * One CTA per SM: 16 consumer warps, one epilogue warp, one producer warp (4 lanes, one per bulk
//     copy of a chunk).  The producer streams chunks - 16 rows x <=2048 columns: the MSB plane tile,
//     the LSB plane tile when the expert runs at 8 bits (<=16 KB each, one contiguous run thanks to the
//     tiled layout), scales and zero-points - into a ring of eight 16 KB units with cp.async.bulk +
//     mbarriers.  It never waits for the gate/up -> down dependency, so down-projection tiles are
//     already in flight (up to the whole ring) while the grid exchanges h.
//   * Integer arithmetic on the tensor pipe.  The activation vector (x, later h) is converted once,
//     per 128-element block, to fixed point relative to the block's largest magnitude and split into
//     three balanced base-256 digits (int8).  The digits sit in separate columns of the B operand of
//     mma.sync m16n8k32 (u8 x s8 -> s32); the A operand is the raw nibble plane: the layout stores
//     the two row halves of a fragment in the low and high nibbles of each byte, so `w & 0x0f0f0f0f`
//     and `w & 0xf0f0f0f0` are the whole unpack (the second half comes out 16 times too large, which
//     the per-row fold divides away).  Sums are exact in int32; MSB and LSB planes combine as
//     16 * Cm + Cl.  Scale and zero-point are applied once per (row, group):
//        sum_k x_k s (q_k - zp) = s (sum_k q_k x_k - zp sum_{k in group} x_k).
//     The plain ALUs could not unpack + convert + FMA two weights per byte at HBM rate; this costs
//     about seven instructions per 512 weights.
//   * Phase 1 (gate/up + SwiGLU): tasks are (expert slot, 16-row block), split over the CTAs by
//     bytes.  The epilogue warp adds the warps' partial rows, applies SwiGLU and writes h (fp32) to
//     the workspace; one bounded grid barrier publishes it.
//   * Phase 2 (down + weighted combine): a task is a 16-row block of the OUTPUT over ALL slots, so
//     the top-k combine stays inside the CTA: no atomics, no cross-CTA reduction, fixed summation
//     order (results are bit-reproducible).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace slicemoe {

constexpr int kConsumerWarps = 16;
constexpr int kEpilogueWarp = kConsumerWarps;
constexpr int kProducerWarp = kConsumerWarps + 1;
constexpr int kThreads = 32 * (kConsumerWarps + 2);
constexpr int kUnits = 8;                                 // ring units; a chunk takes one per plane
constexpr int kChunkK = 128 * kConsumerWarps;             // K columns per chunk: one 128-column block per warp
constexpr int kPlaneUnitBytes = 16 * kChunkK / 2;         // 16384
constexpr int kScaleUnitBytes = 16 * (kChunkK / 32) * 2;  // 2048 (group 32 is the worst case)
constexpr int kZpUnitBytes = 16 * (kChunkK / 32);         // 1024
constexpr int kUnitBytes = kPlaneUnitBytes + kScaleUnitBytes + kZpUnitBytes;  // 19456
constexpr int kMaxSlots = SLICEMOE_MAX_TOP_K + SLICEMOE_MAX_SHARED;
constexpr int kMaxHidden = 4096;
constexpr int kHCap = 12288;  // sum of intermediate widths over all slots of a layer
constexpr unsigned long long kWaitCycles = 4000000000ull;  // ~2 s: every device-side wait is bounded

// ---- workspace --------------------------------------------------------------------------------
struct WsHeader {
  unsigned bar_arrive;  // grid barrier: CTAs that finished the gate/up phase
  unsigned depart;      // CTAs that finished the kernel (the last one re-zeroes the header)
  unsigned status;      // SLICEMOE_STATUS_* bits
  unsigned pad;
};
constexpr size_t kWsHOff = 2048;                              // float h[kHCap]
constexpr size_t kWsStageOff = kWsHOff + sizeof(float) * kHCap;
// host-step staging: x bf16[kMaxHidden] | logits f32[512] | ids i32[16] | w f32[16] | prec u8[16] | y f32[kMaxHidden]
constexpr size_t kWsStX = kWsStageOff;
constexpr size_t kWsStLogits = kWsStX + 2 * kMaxHidden;
constexpr size_t kWsStIds = kWsStLogits + 4 * 512;
constexpr size_t kWsStW = kWsStIds + 64;
constexpr size_t kWsStPrec = kWsStW + 64;
constexpr size_t kWsStY = kWsStPrec + 64;
constexpr size_t kWsBytes = kWsStY + 4 * kMaxHidden;
static_assert(sizeof(WsHeader) <= kWsHOff, "workspace header");

// ---- kernel parameters -------------------------------------------------------------------------
struct DecodeParams {
  const slicemoe_expert* experts;
  const slicemoe_expert* shared;
  const float* gate_vec;
  const uint16_t* x;
  const int32_t* ids;
  const uint8_t* prec;
  const float* weights;
  float* y;
  WsHeader* ws;
  float* ws_h;
  int n_experts, n_shared, k;
  int hidden, inter, shared_inter, group;
  int sigmoid_gate;
};

struct Slot {
  const uint8_t* msb[3];  // gate, up, down
  const uint8_t* lsb[3];
  const uint16_t* sc[3];
  const uint8_t* zp[3];
  const slicemoe_expert* src;  // where the pointers above come from
  int inter;
  int prec;
  float coef;
  int hoff;   // offset of this slot's h in the workspace / in the digit buffer
  int gated;  // 1: the combine weight is sigmoid(gate_vec . x)
  int pad_;
};

// One chunk as the consumers see it (16 bytes, written by the producer):
//   x: flags | nblocks << 8 | rot << 16 | slot << 24
//   y: byte offset in shared memory of the activation digits of the chunk's first column
//   z: byte offset in shared memory of the chunk's first (group, digit-pair) weighted digit sum
//   w: byte offset in shared memory of the chunk's first per-128-block inverse scale
enum : uint32_t {
  kFlagLastOfMatrix = 4,  // last chunk of the matrix row block
  kFlagLastOfTask = 8,    // last matrix of the task: hand the partial rows to the epilogue warp
  kFlagEnd = 16,          // sentinel, no data
  kFlagPrec8 = 32,        // two units: MSB plane, then LSB plane (sums combine as 16 Cm + Cl)
  kFlagPhase2 = 64,
};

struct Plan {
  int first_slot, first_idx, count1;  // phase 1: contiguous run of (slot, row block) tasks
  int count2;                         // phase 2: output row blocks blockIdx.x, + gridDim.x, ...
  int nslots;
  int htotal;  // sum of the slots' intermediate widths
  float gate;  // sigmoid(gate_vec . x) when the shared experts are gated
  int pad_;
};

struct SmemLayout {
  // offsets into dynamic shared memory
  static constexpr int ring = 0;
  static constexpr int hdig = ring + kUnits * kUnitBytes;    // int8 [kHCap/32][3 digits][32]
  static constexpr int xdig = hdig + kHCap * 3;              // int8 [kMaxHidden/32][3][32]
  static constexpr int hsumw = xdig + kMaxHidden * 3;        // float [kHCap/32][2]: weighted digit sums per group
  static constexpr int xsumw = hsumw + (kHCap / 32) * 8;     // float [kMaxHidden/32][2]
  static constexpr int hinv = xsumw + (kMaxHidden / 32) * 8;  // float [kHCap/128]: 2^-e of each 128-block of h
  static constexpr int xinv = hinv + (kHCap / 128) * 4;       // float [kMaxHidden/128]
  static constexpr int partial = xinv + (kMaxHidden / 128) * 4;  // float [2][warps][16][2]
  static constexpr int slots = partial + 2 * kConsumerWarps * 16 * 2 * 4;
  static constexpr int desc = slots + kMaxSlots * (int)sizeof(Slot);  // uint4 [kUnits]
  static constexpr int plan = desc + kUnits * 16;
  static constexpr int bars = (plan + (int)sizeof(Plan) + 15) & ~15;  // uint64 barriers
  static constexpr int nbars = 2 * kUnits + 6;
  static constexpr int dead = bars + nbars * 8;
  static constexpr int total = dead + 16;
};
static_assert(SmemLayout::total <= 227 * 1024, "shared memory budget");
static_assert(sizeof(Slot) % 8 == 0, "slot alignment");
static_assert(SmemLayout::slots % 8 == 0 && SmemLayout::hdig % 16 == 0 && SmemLayout::xdig % 16 == 0 &&
                  SmemLayout::desc % 16 == 0 && SmemLayout::plan % 8 == 0,
              "alignment");

// Ring barriers: full[c % kUnits] for chunk number c (armed with the chunk's bytes), empty[u] for unit u
// (one arrive per consumer warp).  Barrier indices after the 2 * kUnits ring barriers:
enum { kBarPFull0 = 0, kBarPFull1, kBarPEmpty0, kBarPEmpty1, kBarHxGo, kBarHsReady };

// ---- PTX helpers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's dead flag) when the limit is hit or another
// role of this CTA already gave up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* dead, unsigned* status) {
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*dead) return false;
    if ((unsigned long long)(clock64() - t0) > kWaitCycles) {
      *dead = 1;
      atomicOr(status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* dead, unsigned* status) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, dead, status);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// ---- fixed-point activations ---------------------------------------------------------------------
// Byte offset, inside a digit buffer, of digit t of the four values k..k+3 (k % 4 == 0): steps of 32
// columns, 3 digit rows of 32 bytes, and inside a row the order in which the B fragment of m16n8k32 wants
// them: (k % 16) / 4 selects the lane quad position, (k % 32) / 16 the register.
__device__ __forceinline__ int digit_offset(int k, int t) {
  return (k >> 5) * 96 + t * 32 + ((k >> 2) & 3) * 8 + ((k >> 4) & 1) * 4;
}

// One warp converts one 128-element block (lane L holds elements 4L..4L+3 of the block, whose first
// element has index k0 in its vector): fixed point X = rint(v * 2^e) with 2^e * max|v| < 2^22, split into
// balanced base-256 digits d0 + 256 d1 + 65536 d2 (each in int8 range), stored in B-fragment order; the
// weighted digit sums of every group of G elements (the zero-point term of the fold) and the block's 2^-e.
template <int G>
__device__ __forceinline__ void block_to_digits(const float (&v)[4], int k0, int lane, uint8_t* dig, float* sumw,
                                                float* inv) {
  unsigned mb = 0u;  // bit pattern of max |v|: non-negative floats order like their bit patterns
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const unsigned a = __float_as_uint(v[j]) & 0x7fffffffu;
    if (a <= 0x7f800000u) mb = max(mb, a);  // a NaN input gives an undefined result, never a fault
  }
  mb = __reduce_max_sync(0xffffffffu, mb);
  const int ex = (int)(mb >> 23) - 127;  // floor(log2 max) for normal numbers
  const int e = max(-100, min(100, 21 - ex));
  const float scale = __uint_as_float((unsigned)(127 + e) << 23);
  uint32_t dw[3] = {0u, 0u, 0u};
  int ds[3] = {0, 0, 0};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int X = __float2int_rn(v[j] * scale);
    X = max(-4194304, min(4194304, X));
    const int d0 = ((X + 128) & 255) - 128;
    X = (X - d0) >> 8;
    const int d1 = ((X + 128) & 255) - 128;
    const int d2 = (X - d1) >> 8;
    dw[0] |= (uint32_t)(d0 & 255) << (8 * j);
    dw[1] |= (uint32_t)(d1 & 255) << (8 * j);
    dw[2] |= (uint32_t)(d2 & 255) << (8 * j);
    ds[0] += d0;
    ds[1] += d1;
    ds[2] += d2;
  }
  const int k = k0 + 4 * lane;
#pragma unroll
  for (int t = 0; t < 3; ++t) *reinterpret_cast<uint32_t*>(dig + digit_offset(k, t)) = dw[t];
  constexpr int lanes_per_group = G / 4;  // 8, 16 or 32 consecutive lanes cover one group
  const unsigned gmask = lanes_per_group == 32 ? 0xffffffffu
                                               : ((1u << lanes_per_group) - 1u) << (lane & ~(lanes_per_group - 1));
  ds[0] = __reduce_add_sync(gmask, ds[0]);
  ds[1] = __reduce_add_sync(gmask, ds[1]);
  ds[2] = __reduce_add_sync(gmask, ds[2]);
  if ((lane & (lanes_per_group - 1)) == 0) {
    sumw[(k / G) * 2 + 0] = (float)ds[0] + 256.f * (float)ds[1];
    sumw[(k / G) * 2 + 1] = 65536.f * (float)ds[2];
  }
  if (lane == 0) inv[k0 >> 7] = __uint_as_float((unsigned)(127 - e) << 23);
}

// ---- task enumeration (identical in every role) ---------------------------------------------------
__device__ __forceinline__ int nchunks_of(int K) { return (K + kChunkK - 1) / kChunkK; }
// ring units of one phase-1 task (gate + up of a 16-row block) of a slot
__device__ __forceinline__ int slot_spt1(const Slot& s, int hidden) { return 2 * (s.prec ? 2 : 1) * nchunks_of(hidden); }

// ---- consumers -----------------------------------------------------------------------------------
// Phase change: wait until the epilogue warp has seen the whole grid's h in the workspace, then turn it
// into digits (all consumer warps, one 128-block at a time).  Returns false if a wait ran out.
template <int G>
__device__ bool fetch_h(const DecodeParams& p, uint8_t* smem, int warp, int lane, int htotal, volatile int* dead,
                        unsigned* status, uint32_t xbars) {
  const uint32_t hx_go = xbars + 8 * kBarHxGo, hs_ready = xbars + 8 * kBarHsReady;
  if (!mbar_wait(hx_go, 0, dead, status)) return false;
  if (*dead) return false;
  const int nblk = htotal >> 7;
  constexpr int kMaxIt = (kHCap / 128 + kConsumerWarps - 1) / kConsumerWarps;
  float4 v[kMaxIt];
#pragma unroll
  for (int it = 0; it < kMaxIt; ++it) {
    const int blk = it * kConsumerWarps + warp;
    if (blk < nblk) v[it] = __ldcg(reinterpret_cast<const float4*>(p.ws_h) + blk * 32 + lane);
  }
#pragma unroll
  for (int it = 0; it < kMaxIt; ++it) {
    const int blk = it * kConsumerWarps + warp;
    if (blk < nblk) {
      const float q[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
      block_to_digits<G>(q, blk * 128, lane, smem + SmemLayout::hdig, reinterpret_cast<float*>(smem + SmemLayout::hsumw),
                         reinterpret_cast<float*>(smem + SmemLayout::hinv));
    }
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(hs_ready);
  return mbar_wait(hs_ready, 0, dead, status);
}

template <int G>
__device__ void consumer_loop(const DecodeParams& p, uint8_t* smem, int warp, int lane) {
  constexpr int SG = 128 / G;
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const uint4* descs = reinterpret_cast<const uint4*>(smem + SmemLayout::desc);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  float* partial = reinterpret_cast<float*>(smem + SmemLayout::partial);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars, empty0 = bars + 8 * kUnits, xbars = bars + 16 * kUnits;
  const uint32_t pfull0 = xbars + 8 * kBarPFull0, pempty0 = xbars + 8 * kBarPEmpty0;
  unsigned* status = &p.ws->status;

  // The lane folds row r of the 16-row block for the digit columns it holds: lanes with c in {0, 1} take
  // the accumulators of row g, lanes with c in {2, 3} those of row g + 8 (which are 16 times too large
  // because their nibbles were left in the high half of the byte); even c holds digits 0 and 1, odd c
  // digit 2 (and the unused fourth column).
  const int c = lane & 3, g8 = lane >> 2;
  const int r = g8 + 8 * (c >> 1);
  const int cq = c & 1;
  const float rowfix = (c >> 1) ? 0.0625f : 1.f;
  const float w0 = (cq ? 65536.f : 1.f) * rowfix, w1 = (cq ? 0.f : 256.f) * rowfix;
  // B column n = g8 takes digit n % 4; the fourth is unused, so those lanes re-read digit 0 and are ignored
  const int boff = ((g8 & 3) == 3 ? 0 : (g8 & 3)) * 32 + c * 8;
  int acc[SG][4];
  float rowacc = 0.f, part0 = 0.f, part1 = 0.f;
  bool fetched = false;
  int taskcount = 0;
  int unit = 0;  // running unit counter

  for (int cn = 0;; ++cn) {  // chunk number
    if (!mbar_wait(full0 + 8 * (cn % kUnits), (cn / kUnits) & 1, dead, status)) return;
    const uint4 d = descs[cn % kUnits];
    const uint32_t flags = d.x & 0xffu;
    if (flags & kFlagEnd) break;
    if ((flags & kFlagPhase2) && !fetched) {
      if (!fetch_h<G>(p, smem, warp, lane, plan.htotal, dead, status, xbars)) return;
      fetched = true;
    }
    const bool p8 = (flags & kFlagPrec8) != 0;
    const int u0 = unit % kUnits, u1 = (unit + 1) % kUnits;
    // the 128-column block of this chunk handled by this warp
    int b = warp - (int)((d.x >> 16) & 0xffu);
    if (b < 0) b += kConsumerWarps;
    if (b < (int)((d.x >> 8) & 0xffu)) {
#pragma unroll
      for (int sg = 0; sg < SG; ++sg)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[sg][q] = 0;
      const uint8_t* bp = smem + d.y + b * 384 + boff;
      const uint2 bv0 = *reinterpret_cast<const uint2*>(bp);
      const uint2 bv1 = *reinterpret_cast<const uint2*>(bp + 96);
      const uint2 bv2 = *reinterpret_cast<const uint2*>(bp + 192);
      const uint2 bv3 = *reinterpret_cast<const uint2*>(bp + 288);
      const uint8_t* ap = smem + SmemLayout::ring + u0 * kUnitBytes + b * 1024 + lane * 16;
      {
        const uint4 wlo = *reinterpret_cast<const uint4*>(ap);
        const uint4 whi = *reinterpret_cast<const uint4*>(ap + 512);
        mma_u8s8(acc[0], wlo.x & 0x0f0f0f0fu, wlo.x & 0xf0f0f0f0u, wlo.y & 0x0f0f0f0fu, wlo.y & 0xf0f0f0f0u, bv0.x, bv0.y);
        mma_u8s8(acc[32 / G], wlo.z & 0x0f0f0f0fu, wlo.z & 0xf0f0f0f0u, wlo.w & 0x0f0f0f0fu, wlo.w & 0xf0f0f0f0u, bv1.x,
                 bv1.y);
        mma_u8s8(acc[64 / G], whi.x & 0x0f0f0f0fu, whi.x & 0xf0f0f0f0u, whi.y & 0x0f0f0f0fu, whi.y & 0xf0f0f0f0u, bv2.x,
                 bv2.y);
        mma_u8s8(acc[96 / G], whi.z & 0x0f0f0f0fu, whi.z & 0xf0f0f0f0u, whi.w & 0x0f0f0f0fu, whi.w & 0xf0f0f0f0u, bv3.x,
                 bv3.y);
      }
      if (p8) {
        const uint8_t* ap2 = smem + SmemLayout::ring + u1 * kUnitBytes + b * 1024 + lane * 16;
        const uint4 wlo = *reinterpret_cast<const uint4*>(ap2);
        const uint4 whi = *reinterpret_cast<const uint4*>(ap2 + 512);
#pragma unroll
        for (int sg = 0; sg < SG; ++sg)
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[sg][q] <<= 4;
        mma_u8s8(acc[0], wlo.x & 0x0f0f0f0fu, wlo.x & 0xf0f0f0f0u, wlo.y & 0x0f0f0f0fu, wlo.y & 0xf0f0f0f0u, bv0.x, bv0.y);
        mma_u8s8(acc[32 / G], wlo.z & 0x0f0f0f0fu, wlo.z & 0xf0f0f0f0u, wlo.w & 0x0f0f0f0fu, wlo.w & 0xf0f0f0f0u, bv1.x,
                 bv1.y);
        mma_u8s8(acc[64 / G], whi.x & 0x0f0f0f0fu, whi.x & 0xf0f0f0f0u, whi.y & 0x0f0f0f0fu, whi.y & 0xf0f0f0f0u, bv2.x,
                 bv2.y);
        mma_u8s8(acc[96 / G], whi.z & 0x0f0f0f0fu, whi.z & 0xf0f0f0f0u, whi.w & 0x0f0f0f0fu, whi.w & 0xf0f0f0f0u, bv3.x,
                 bv3.y);
      }
      // fold: scales / zero-points travel in the first unit of the chunk
      {
        const uint8_t* meta = smem + SmemLayout::ring + u0 * kUnitBytes + kPlaneUnitBytes;
        const uint16_t* ms = reinterpret_cast<const uint16_t*>(meta) + (b * SG) * 16 + r;
        const uint8_t* mz = meta + kScaleUnitBytes + (b * SG) * 16 + r;
        const float* sumw = reinterpret_cast<const float*>(smem + d.z) + (b * SG) * 2 + cq;
        const float binv = *(reinterpret_cast<const float*>(smem + d.w) + b);
        const float sfix = p8 ? binv : 16.f * binv;
        const int zsh = p8 ? 0 : 4;
#pragma unroll
        for (int sg = 0; sg < SG; ++sg) {
          const int ca = (c >> 1) ? acc[sg][2] : acc[sg][0];
          const int cb = (c >> 1) ? acc[sg][3] : acc[sg][1];
          const float t = fmaf((float)cb, w1, (float)ca * w0);
          const float sc = __half2float(__ushort_as_half(ms[sg * 16])) * sfix;
          const float z = (float)((int)mz[sg * 16] >> zsh);
          // both slices: s (16 Cm + Cl - zp X); MSB only: 16 s (Cm - (zp >> 4) X)
          rowacc = fmaf(sc, fmaf(-z, sumw[sg * 2], t), rowacc);
        }
      }
    }
    __syncwarp();
    if (lane == 0) {
      mbar_arrive(empty0 + 8 * u0);
      if (p8) mbar_arrive(empty0 + 8 * u1);
    }
    unit += p8 ? 2 : 1;
    if (flags & kFlagLastOfMatrix) {
      rowacc += __shfl_xor_sync(0xffffffffu, rowacc, 1);  // digits 0,1 (even c) + digit 2 (odd c)
      if (!(flags & kFlagPhase2)) {
        if (!(flags & kFlagLastOfTask)) part0 = rowacc;  // gate
        else part1 = rowacc;                             // up
      } else {
        const Slot& sl = slots[d.x >> 24];
        part1 = fmaf(sl.gated ? plan.gate : sl.coef, rowacc, part1);  // weighted combine, in slot order
      }
      rowacc = 0.f;
      if (flags & kFlagLastOfTask) {
        // hand this warp's share of the K split to the epilogue warp
        const int buf = taskcount & 1;
        if (!mbar_wait(pempty0 + 8 * buf, ((taskcount >> 1) & 1) ^ 1, dead, status)) return;
        if (cq == 0) *reinterpret_cast<float2*>(partial + ((buf * kConsumerWarps + warp) * 16 + r) * 2) = make_float2(part0, part1);
        __syncwarp();
        if (lane == 0) mbar_arrive(pfull0 + 8 * buf);
        ++taskcount;
        part0 = part1 = 0.f;
      }
    }
  }
}

// ---- epilogue warp ---------------------------------------------------------------------------------
__device__ void epilogue_loop(const DecodeParams& p, uint8_t* smem, int lane) {
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  const float* partial = reinterpret_cast<const float*>(smem + SmemLayout::partial);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t xbars = bars + 16 * kUnits;
  const uint32_t pfull0 = xbars + 8 * kBarPFull0, pempty0 = xbars + 8 * kBarPEmpty0, hx_go = xbars + 8 * kBarHxGo;
  unsigned* status = &p.ws->status;
  const int total = plan.count1 + plan.count2;
  int slot = plan.first_slot, idx = plan.first_idx;
  for (int tc = 0;; ++tc) {
    if (tc == plan.count1) {
      // ---- the single grid-wide dependency: every CTA has written its rows of h ----
      __syncwarp();
      if (lane == 0) {
        __threadfence();
        atomicAdd(&p.ws->bar_arrive, 1u);
      }
      __syncwarp();
      if (plan.count2 > 0) {
        // the whole warp polls, converged: no lane spins on something another lane must provide
        const long long t0 = clock64();
        while (ld_acquire_u32(&p.ws->bar_arrive) < gridDim.x) {
          if (*dead) break;
          if ((unsigned long long)(clock64() - t0) > kWaitCycles) {
            *dead = 1;
            atomicOr(status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
            break;
          }
        }
        __threadfence();
        __syncwarp();
        if (*dead) return;
        if (lane == 0) mbar_arrive(hx_go);
      }
    }
    if (tc == total) break;
    const int buf = tc & 1;
    if (!mbar_wait(pfull0 + 8 * buf, (tc >> 1) & 1, dead, status)) return;
    float a = 0.f, b = 0.f;
    if (lane < 16) {
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float2 v = *reinterpret_cast<const float2*>(partial + ((buf * kConsumerWarps + w) * 16 + lane) * 2);
        a += v.x;
        b += v.y;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(pempty0 + 8 * buf);
    if (tc < plan.count1) {
      if (lane < 16) p.ws_h[slots[slot].hoff + idx * 16 + lane] = a / (1.f + expf(-a)) * b;  // silu(gate) * up
      if (++idx >= slots[slot].inter / 16) {
        idx = 0;
        ++slot;
      }
    } else if (lane < 16) {
      p.y[(blockIdx.x + (tc - plan.count1) * gridDim.x) * 16 + lane] = b;
    }
  }
}

// ---- producer --------------------------------------------------------------------------------------
struct ProducerState {
  int cn;    // chunk number: selects the full barrier and the descriptor slot
  int unit;  // running unit counter: a chunk takes one unit per plane
};

// Streams the chunks of one (slot, matrix, row block) into the ring.  Run by lanes 0..3 of the producer
// warp together: lane 0 copies the MSB plane tile, lane 1 the LSB tile (8-bit slots), lane 2 the scales,
// lane 3 the zero-points.  Returns false if a wait ran out.  act_* are the shared-memory byte offsets of
// the activation digits / digit sums / block scales that go with the matrix' first column.
template <int G>
__device__ __forceinline__ bool produce_matrix(uint8_t* smem, ProducerState& ps, int lane, const Slot& s, int slot,
                                               int mat, int K, int rb, uint32_t base_flags, bool last_matrix,
                                               uint32_t act_dig, uint32_t act_sum, uint32_t act_inv, volatile int* dead,
                                               unsigned* status) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  uint4* descs = reinterpret_cast<uint4*>(smem + SmemLayout::desc);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars, empty0 = bars + 8 * kUnits;
  const uint32_t ring = smem_u32(smem + SmemLayout::ring);
  const bool p8 = s.prec != 0;
  // this lane's source: base for the row block, bytes per column block of kChunkK, destination inside the unit
  const unsigned plane_off = (unsigned)rb * (unsigned)(K >> 6) * 512u;
  const unsigned meta_off = (unsigned)rb * (unsigned)(K >> LG) * 16u;  // entries
  const uint8_t* src;
  uint32_t per_k_shift_bytes;  // bytes per 128 columns
  uint32_t dst_in_unit;
  if (lane == 0) {
    src = s.msb[mat] + plane_off;
    per_k_shift_bytes = 1024u;
    dst_in_unit = 0u;
  } else if (lane == 1) {
    src = s.lsb[mat] + plane_off;
    per_k_shift_bytes = 1024u;
    dst_in_unit = (uint32_t)kUnitBytes;  // the chunk's second unit
  } else if (lane == 2) {
    src = reinterpret_cast<const uint8_t*>(s.sc[mat] + meta_off);
    per_k_shift_bytes = (128u >> LG) * 32u;
    dst_in_unit = (uint32_t)kPlaneUnitBytes;
  } else {
    src = s.zp[mat] + meta_off;
    per_k_shift_bytes = (128u >> LG) * 16u;
    dst_in_unit = (uint32_t)(kPlaneUnitBytes + kScaleUnitBytes);
  }
  const bool active = lane != 1 || p8;
  const uint32_t flags0 = base_flags | (p8 ? kFlagPrec8 : 0u);
  for (int k0 = 0; k0 < K; k0 += kChunkK) {
    const int kc = min(kChunkK, K - k0);
    const int u0 = ps.unit % kUnits, u1 = (ps.unit + 1) % kUnits;
    if (!mbar_wait(empty0 + 8 * u0, ((ps.unit / kUnits) & 1) ^ 1, dead, status)) return false;
    if (p8 && !mbar_wait(empty0 + 8 * u1, (((ps.unit + 1) / kUnits) & 1) ^ 1, dead, status)) return false;
    const uint32_t bar = full0 + 8 * (ps.cn % kUnits);
    if (lane == 0) {
      uint32_t flags = flags0;
      if (k0 + kChunkK >= K) flags |= kFlagLastOfMatrix | (last_matrix ? kFlagLastOfTask : 0u);
      descs[ps.cn % kUnits] = make_uint4(flags | ((uint32_t)(kc >> 7) << 8) |
                                             ((uint32_t)(ps.cn % kConsumerWarps) << 16) | ((uint32_t)slot << 24),
                                         act_dig + (uint32_t)k0 * 3u, act_sum + (uint32_t)(k0 >> LG) * 8u,
                                         act_inv + (uint32_t)(k0 >> 7) * 4u);
      const uint32_t nblk = (uint32_t)(kc >> 7);
      mbar_arrive_expect_tx(bar, nblk * ((p8 ? 2048u : 1024u) + (128u >> LG) * 48u));
    }
    __syncwarp(0xfu);
    if (active) {
      // a second-unit destination wraps around the ring with the unit index
      const uint32_t dst = ring + (lane == 1 ? (uint32_t)u1 * kUnitBytes : (uint32_t)u0 * kUnitBytes + dst_in_unit);
      bulk_g2s(dst, src + (size_t)(k0 >> 7) * per_k_shift_bytes, (uint32_t)(kc >> 7) * per_k_shift_bytes, bar);
    }
    ps.unit += p8 ? 2 : 1;
    ++ps.cn;
  }
  return true;
}

template <int G>
__device__ void producer_loop(const DecodeParams& p, uint8_t* smem, int lane) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  uint4* descs = reinterpret_cast<uint4*>(smem + SmemLayout::desc);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars;
  unsigned* status = &p.ws->status;
  ProducerState ps;
  ps.cn = 0;
  ps.unit = 0;
  bool ok = true;
  // phase 1: gate and up of (slot, row block) tasks
  {
    int slot = plan.first_slot, idx = plan.first_idx;
    for (int n = 0; n < plan.count1 && ok; ++n) {
      const Slot& s = slots[slot];
      ok = produce_matrix<G>(smem, ps, lane, s, slot, 0, p.hidden, idx, 0u, false, SmemLayout::xdig, SmemLayout::xsumw,
                             SmemLayout::xinv, dead, status) &&
           produce_matrix<G>(smem, ps, lane, s, slot, 1, p.hidden, idx, 0u, true, SmemLayout::xdig, SmemLayout::xsumw,
                             SmemLayout::xinv, dead, status);
      if (++idx >= s.inter / 16) {
        idx = 0;
        ++slot;
      }
    }
  }
  // phase 2: down rows of every slot for the output row blocks of this CTA
  for (int n = 0; n < plan.count2 && ok; ++n) {
    const int rb = blockIdx.x + n * gridDim.x;
    for (int slot = 0; slot < plan.nslots && ok; ++slot) {
      const Slot& s = slots[slot];
      ok = produce_matrix<G>(smem, ps, lane, s, slot, 2, s.inter, rb, kFlagPhase2, slot == plan.nslots - 1,
                             SmemLayout::hdig + (uint32_t)s.hoff * 3u, SmemLayout::hsumw + (uint32_t)(s.hoff >> LG) * 8u,
                             SmemLayout::hinv + (uint32_t)(s.hoff >> 7) * 4u, dead, status);
    }
  }
  // The sentinel takes a descriptor slot but no unit.  Waiting for the next unit to be free, as a real
  // chunk would, is what guarantees that chunk cn - kUnits (the slot's previous user) has been consumed.
  if (ok && mbar_wait(bars + 8 * kUnits + 8 * (ps.unit % kUnits), ((ps.unit / kUnits) & 1) ^ 1, dead, status)) {
    if (lane == 0) {
      descs[ps.cn % kUnits] = make_uint4(kFlagEnd, 0u, 0u, 0u);
      mbar_arrive(full0 + 8 * (ps.cn % kUnits));
    }
    ++ps.cn;
  }
  // Never leave the CTA with bulk copies still landing in its shared memory: wait (bounded) for the
  // last kUnits armed barriers.  In the normal path they have all completed long ago.
  for (int j = max(0, ps.cn - kUnits); j < ps.cn; ++j) {
    const uint32_t bar = full0 + 8 * (j % kUnits);
    const long long t0 = clock64();
    while (!mbar_try(bar, (j / kUnits) & 1)) {
      if (*dead || (unsigned long long)(clock64() - t0) > kWaitCycles) break;
    }
  }
}

// ---- prologue pieces ---------------------------------------------------------------------------------
// Warp 0: the routing list -> slot table -> plane pointers -> the static partition.
// Slot order: shared experts, then the routed experts that run at 8 bits, then those that run at 4 bits,
// each group in list order.  With the larger tasks first, windows of a multiple of the larger task size cut
// the phase-1 unit sequence at task boundaries, so every CTA gets the same number of units.
__device__ void build_plan(const DecodeParams& p, uint8_t* smem, int lane) {
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);
  // routed experts: lane j reads entry j of the list; out-of-range ids are dropped and reported
  int e = -1, pr = 0;
  float w = 0.f;
  if (lane < p.k) {
    e = p.ids[lane];
    pr = p.prec[lane];
    w = p.weights[lane];
  }
  const bool valid = lane < p.k && e >= 0 && e < p.n_experts;
  const unsigned vmask = __ballot_sync(0xffffffffu, valid);
  const unsigned bigmask = __ballot_sync(0xffffffffu, valid && pr != 0);
  if (lane < p.k && !valid) atomicOr(&p.ws->status, (unsigned)SLICEMOE_STATUS_BAD_EXPERT_ID);
  const int nrouted = __popc(vmask), nbig = __popc(bigmask);
  const int nslots = nrouted + p.n_shared;
  const unsigned below = (1u << lane) - 1u;
  if (valid) {
    const int pos = pr != 0 ? __popc(bigmask & below) : nbig + __popc(vmask & ~bigmask & below);
    Slot& s = slots[p.n_shared + pos];
    s.src = p.experts + e;
    s.inter = p.inter;
    s.prec = pr != 0;
    s.coef = w;
    s.gated = 0;
    s.hoff = p.n_shared * p.shared_inter + pos * p.inter;
  }
  if (lane < p.n_shared) {
    Slot& s = slots[lane];
    s.src = p.shared + lane;
    s.inter = p.shared_inter;
    s.prec = 1;
    s.coef = 1.f;
    s.gated = p.sigmoid_gate;
    s.hoff = lane * p.shared_inter;
  }
  __syncwarp();
  // plane pointers: one 8-byte load per (slot, matrix, field)
  for (int i = lane; i < nslots * 12; i += 32) {
    const int s = i / 12, q = i % 12, m = q >> 2, f = q & 3;
    const slicemoe_mat* mat = reinterpret_cast<const slicemoe_mat*>(slots[s].src) + m;
    const void* ptr = *(reinterpret_cast<const void* const*>(mat) + f);
    if (f == 0) slots[s].msb[m] = reinterpret_cast<const uint8_t*>(ptr);
    else if (f == 1) slots[s].lsb[m] = reinterpret_cast<const uint8_t*>(ptr);
    else if (f == 2) slots[s].sc[m] = reinterpret_cast<const uint16_t*>(ptr);
    else slots[s].zp[m] = reinterpret_cast<const uint8_t*>(ptr);
  }
  __syncwarp();
  // lane j owns slot j: a slot without LSB planes runs MSB-only; units and tasks per slot
  int nt = 0, sp = 0;
  if (lane < nslots) {
    Slot& s = slots[lane];
    if (!(s.lsb[0] && s.lsb[1] && s.lsb[2])) s.prec = 0;
    nt = s.inter / 16;
    sp = slot_spt1(s, p.hidden);
  }
  unsigned cs = (unsigned)(nt * sp), ct = (unsigned)nt;  // inclusive scans over the slots
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned a = __shfl_up_sync(0xffffffffu, cs, off), b = __shfl_up_sync(0xffffffffu, ct, off);
    if (lane >= off) {
      cs += a;
      ct += b;
    }
  }
  const unsigned S = __shfl_sync(0xffffffffu, cs, 31);
  const unsigned NT = __shfl_sync(0xffffffffu, ct, 31);
  const unsigned spmax = max(1u, __reduce_max_sync(0xffffffffu, (unsigned)sp));
  // phase 1: CTA c takes the tasks whose first unit lies in [c T, (c + 1) T), T = the equal share rounded
  // up to a multiple of the larger task size
  const unsigned T = ((S + gridDim.x - 1) / gridDim.x + spmax - 1) / spmax * spmax;
  const unsigned lo = blockIdx.x * T, hi = lo + T;
  const unsigned off_s = cs - (unsigned)(nt * sp), off_t = ct - (unsigned)nt;  // exclusive
  unsigned ord_lo = NT, ord_hi = NT;
  int slot_lo = nslots, idx_lo = 0;
  if (lane < nslots && nt > 0) {
    if (lo >= off_s && lo < cs) {
      const unsigned i = (lo - off_s + sp - 1) / sp;  // may equal nt: then it is the next slot's first task
      ord_lo = off_t + i;
      slot_lo = lane;
      idx_lo = (int)i;
    }
    if (hi >= off_s && hi < cs) ord_hi = off_t + (hi - off_s + sp - 1) / sp;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {  // at most one lane holds each answer
    const unsigned o = __shfl_xor_sync(0xffffffffu, ord_lo, off);
    const int sl2 = __shfl_xor_sync(0xffffffffu, slot_lo, off), ix2 = __shfl_xor_sync(0xffffffffu, idx_lo, off);
    if (sl2 < slot_lo) {
      ord_lo = o;
      slot_lo = sl2;
      idx_lo = ix2;
    }
    ord_hi = min(ord_hi, __shfl_xor_sync(0xffffffffu, ord_hi, off));
  }
  if (lane == 0) {
    if (slot_lo < nslots && idx_lo >= slots[slot_lo].inter / 16) {  // the bound fell on the slot's end
      idx_lo = 0;
      ++slot_lo;
    }
    plan->first_slot = slot_lo;
    plan->first_idx = idx_lo;
    plan->count1 = (int)(ord_hi - ord_lo);
    const int nrb = p.hidden / 16;
    plan->count2 = (nslots > 0 && (int)blockIdx.x < nrb) ? (nrb - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    plan->nslots = nslots;
    plan->htotal = nrouted * p.inter + p.n_shared * p.shared_inter;
  }
}

// ---- the kernel ------------------------------------------------------------------------------------
template <int G>
__global__ void __launch_bounds__(kThreads, 1) decode_layer_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);

  // Prologue, all roles in parallel and one barrier at the end: warp 0 builds the slot table and the
  // partition (two dependent global reads: the routing list, then the experts' plane pointers); the other
  // warps turn x into digits, one 128-element block per warp; the last warp sets up the barriers and the
  // shared-expert gate.
  if (warp == 0) {
    build_plan(p, smem, lane);
  } else if (warp == kProducerWarp) {
    if (lane == 0) {
      *reinterpret_cast<int*>(smem + SmemLayout::dead) = 0;
      const uint32_t bars = smem_u32(smem + SmemLayout::bars);
      for (int s = 0; s < kUnits; ++s) {
        mbar_init(bars + 8 * s, 1);                           // full: lane 0's expect_tx arrive
        mbar_init(bars + 8 * kUnits + 8 * s, kConsumerWarps);  // empty: one arrive per consumer warp
      }
      const uint32_t xbars = bars + 16 * kUnits;
      mbar_init(xbars + 8 * kBarPFull0, kConsumerWarps);
      mbar_init(xbars + 8 * kBarPFull1, kConsumerWarps);
      mbar_init(xbars + 8 * kBarPEmpty0, 1);
      mbar_init(xbars + 8 * kBarPEmpty1, 1);
      mbar_init(xbars + 8 * kBarHxGo, 1);
      mbar_init(xbars + 8 * kBarHsReady, kConsumerWarps);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (p.sigmoid_gate && p.n_shared > 0) {
      // Qwen-style shared-expert gate: sigmoid(v . x)
      float dot = 0.f;
      for (int i = lane; i < p.hidden / 2; i += 32) {
        const uint32_t raw = *reinterpret_cast<const uint32_t*>(p.x + 2 * i);
        const float2 gv = __ldg(reinterpret_cast<const float2*>(p.gate_vec) + i);
        dot = fmaf(gv.x, __uint_as_float(raw << 16), dot);
        dot = fmaf(gv.y, __uint_as_float(raw & 0xffff0000u), dot);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
      if (lane == 0) plan->gate = 1.f / (1.f + expf(-dot));
    }
  } else {
    for (int blk = warp - 1; blk < p.hidden / 128; blk += kConsumerWarps) {
      const uint2 raw = *reinterpret_cast<const uint2*>(p.x + blk * 128 + 4 * lane);
      const float v[4] = {__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                          __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u)};
      block_to_digits<G>(v, blk * 128, lane, smem + SmemLayout::xdig, reinterpret_cast<float*>(smem + SmemLayout::xsumw),
                         reinterpret_cast<float*>(smem + SmemLayout::xinv));
    }
  }
  __syncthreads();
  if (plan->nslots == 0 && blockIdx.x == 0)
    for (int i = tid; i < p.hidden; i += kThreads) p.y[i] = 0.f;

  if (warp < kConsumerWarps) {
    consumer_loop<G>(p, smem, warp, lane);
  } else if (warp == kEpilogueWarp) {
    epilogue_loop(p, smem, lane);
  } else if (lane < 4) {
    producer_loop<G>(p, smem, lane);
  }
  __syncthreads();
  if (tid == 0) {
    const unsigned old = atomicAdd(&p.ws->depart, 1u);
    if (old == gridDim.x - 1) {  // everyone is past the barrier: make the header reusable
      p.ws->bar_arrive = 0;
      p.ws->depart = 0;
      __threadfence();
    }
  }
}

// ---- host side --------------------------------------------------------------------------------------
static int g_num_sms[64];
static bool g_attr_set[64][3];

static int device_setup(int* dev_out, int* sms_out) {
  int dev = 0;
  SM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SLICEMOE_E_UNSUPPORTED;
  if (g_num_sms[dev] == 0) {
    int sms = 0;
    SM_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    g_num_sms[dev] = sms;
  }
  *dev_out = dev;
  *sms_out = g_num_sms[dev];
  return SLICEMOE_OK;
}

template <int G>
static int launch_decode(const DecodeParams& p, int dev, int sms, int gi, cudaStream_t st) {
  if (!g_attr_set[dev][gi]) {
    SM_CUDA_TRY(cudaFuncSetAttribute(decode_layer_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     SmemLayout::total));
    g_attr_set[dev][gi] = true;
  }
  decode_layer_kernel<G><<<sms, kThreads, SmemLayout::total, st>>>(p);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

static int check_shape(const slicemoe_shape* s) {
  if (!s) return SLICEMOE_E_INVALID_ARG;
  if (s->b_high != 8 || s->b_low != 4) return SLICEMOE_E_UNSUPPORTED;
  if (!valid_group(s->group)) return SLICEMOE_E_UNSUPPORTED;
  if (s->hidden <= 0 || s->inter <= 0 || s->n_experts <= 0 || s->top_k < 1) return SLICEMOE_E_INVALID_ARG;
  if (s->top_k > s->n_experts || s->top_k > SLICEMOE_MAX_TOP_K) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared < 0 || s->n_shared > SLICEMOE_MAX_SHARED) return SLICEMOE_E_INVALID_ARG;
  if ((s->hidden % 128) || (s->inter % 128)) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && (s->shared_inter <= 0 || (s->shared_inter % 128))) return SLICEMOE_E_INVALID_ARG;
  if (s->hidden > kMaxHidden) return SLICEMOE_E_UNSUPPORTED;
  return SLICEMOE_OK;
}

static int run_layer(const slicemoe_shape* shape, const slicemoe_expert* experts, const slicemoe_expert* shared,
                     int n_shared, const float* gate_vec, const void* x, int T, const int32_t* ids,
                     const uint8_t* prec, const float* weights, float* y, void* workspace, size_t workspace_bytes,
                     void* stream) {
  int rc = check_shape(shape);
  if (rc != SLICEMOE_OK) return rc;
  if (!experts || !x || !ids || !prec || !weights || !y || !workspace || T <= 0) return SLICEMOE_E_INVALID_ARG;
  if (n_shared > 0 && !shared) return SLICEMOE_E_INVALID_ARG;
  if (n_shared > 0 && shape->shared_sigmoid_gate && !gate_vec) return SLICEMOE_E_INVALID_ARG;
  if (workspace_bytes < kWsBytes || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SLICEMOE_E_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(x) & 15) return SLICEMOE_E_INVALID_ARG;
  const long long hsum = (long long)shape->top_k * shape->inter + (long long)n_shared * shape->shared_inter;
  if (hsum > kHCap) return SLICEMOE_E_UNSUPPORTED;
  int dev, sms;
  rc = device_setup(&dev, &sms);
  if (rc != SLICEMOE_OK) return rc;

  DecodeParams p;
  p.experts = experts;
  p.shared = shared;
  p.gate_vec = gate_vec;
  p.ws = reinterpret_cast<WsHeader*>(workspace);
  p.ws_h = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + kWsHOff);
  p.n_experts = shape->n_experts;
  p.n_shared = n_shared;
  p.k = shape->top_k;
  p.hidden = shape->hidden;
  p.inter = shape->inter;
  p.shared_inter = n_shared > 0 ? shape->shared_inter : 0;
  p.group = shape->group;
  p.sigmoid_gate = (n_shared > 0 && shape->shared_sigmoid_gate) ? 1 : 0;
  cudaStream_t st = (cudaStream_t)stream;
  for (int t = 0; t < T; ++t) {
    p.x = reinterpret_cast<const uint16_t*>(x) + (size_t)t * shape->hidden;
    p.ids = ids + (size_t)t * shape->top_k;
    p.prec = prec + (size_t)t * shape->top_k;
    p.weights = weights + (size_t)t * shape->top_k;
    p.y = y + (size_t)t * shape->hidden;
    if (shape->group == 128) rc = launch_decode<128>(p, dev, sms, 0, st);
    else if (shape->group == 64) rc = launch_decode<64>(p, dev, sms, 1, st);
    else rc = launch_decode<32>(p, dev, sms, 2, st);
    if (rc != SLICEMOE_OK) return rc;
  }
  return SLICEMOE_OK;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" size_t slicemoe_workspace_bytes(const slicemoe_shape* shape) {
  (void)shape;
  return kWsBytes;
}

extern "C" int slicemoe_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || workspace_bytes < kWsBytes || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SLICEMOE_E_INVALID_ARG;
  SM_CUDA_TRY(cudaMemsetAsync(workspace, 0, kWsHOff, (cudaStream_t)stream));
  return SLICEMOE_OK;
}

extern "C" int slicemoe_get_status(void* workspace, int* status_out, void* stream) {
  if (!workspace || !status_out) return SLICEMOE_E_INVALID_ARG;
  WsHeader* h = reinterpret_cast<WsHeader*>(workspace);
  unsigned v = 0;
  cudaStream_t st = (cudaStream_t)stream;
  SM_CUDA_TRY(cudaMemcpyAsync(&v, &h->status, sizeof(v), cudaMemcpyDeviceToHost, st));
  SM_CUDA_TRY(cudaMemsetAsync(&h->status, 0, sizeof(unsigned), st));
  SM_CUDA_TRY(cudaStreamSynchronize(st));
  *status_out = (int)v;
  return SLICEMOE_OK;
}

extern "C" int slicemoe_expert_ffn(const slicemoe_shape* shape, const slicemoe_expert* experts, const void* x, int T,
                                   const int32_t* ids, const uint8_t* prec, const float* weights, float* y,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  return run_layer(shape, experts, nullptr, 0, nullptr, x, T, ids, prec, weights, y, workspace, workspace_bytes,
                   stream);
}

extern "C" int slicemoe_layer(const slicemoe_shape* shape, const slicemoe_expert* experts,
                              const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                              const int32_t* ids, const uint8_t* prec, const float* weights, float* y,
                              void* workspace, size_t workspace_bytes, void* stream) {
  if (!shape) return SLICEMOE_E_INVALID_ARG;
  return run_layer(shape, experts, shared, shape->n_shared, shared_gate_vec, x, T, ids, prec, weights, y, workspace,
                   workspace_bytes, stream);
}

extern "C" int slicemoe_decode_step_host(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                         const slicemoe_expert* shared, const float* shared_gate_vec,
                                         const void* x_host, const float* logits_host, const float* bias, int renorm,
                                         float tau, int rank_high, float* y_host, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != SLICEMOE_OK) return rc;
  if (!x_host || !logits_host || !y_host || !workspace || workspace_bytes < kWsBytes) return SLICEMOE_E_INVALID_ARG;
  if (shape->n_experts > 512) return SLICEMOE_E_UNSUPPORTED;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  cudaStream_t st = (cudaStream_t)stream;
  void* dx = ws + kWsStX;
  float* dlogits = reinterpret_cast<float*>(ws + kWsStLogits);
  int32_t* dids = reinterpret_cast<int32_t*>(ws + kWsStIds);
  float* dw = reinterpret_cast<float*>(ws + kWsStW);
  uint8_t* dprec = ws + kWsStPrec;
  float* dy = reinterpret_cast<float*>(ws + kWsStY);
  SM_CUDA_TRY(cudaMemcpyAsync(dx, x_host, 2 * (size_t)shape->hidden, cudaMemcpyHostToDevice, st));
  SM_CUDA_TRY(cudaMemcpyAsync(dlogits, logits_host, 4 * (size_t)shape->n_experts, cudaMemcpyHostToDevice, st));
  rc = slicemoe_route_topk(dlogits, 1, shape->n_experts, shape->top_k, bias, renorm, tau, rank_high, dids, dw, dprec,
                           stream);
  if (rc != SLICEMOE_OK) return rc;
  rc = slicemoe_layer(shape, experts, shared, shared_gate_vec, dx, 1, dids, dprec, dw, dy, workspace, workspace_bytes,
                      stream);
  if (rc != SLICEMOE_OK) return rc;
  SM_CUDA_TRY(cudaMemcpyAsync(y_host, dy, 4 * (size_t)shape->hidden, cudaMemcpyDeviceToHost, st));
  SM_CUDA_TRY(cudaStreamSynchronize(st));
  return SLICEMOE_OK;
}

// ---- entry point for callers that cannot allocate -----------------------------------------------------
// The scratch that slicemoe_layer takes from the caller lives here, in the library image: kWsBytes bytes
// per GPU that loads the library, held until the process exits.
namespace slicemoe {
static __device__ __align__(256) unsigned char g_static_scratch[kWsBytes];
static void* g_static_scratch_ptr[64];  // device address of the array, per device, resolved once
}  // namespace slicemoe

extern "C" int slicemoe_layer_static(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                     const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                                     const int32_t* ids, const uint8_t* prec, const float* weights, float* y,
                                     void* stream) {
  if (!shape) return SLICEMOE_E_INVALID_ARG;
  // The built-in scratch has one fixed size; a layer that would need more is refused, never truncated.
  const long long hsum = (long long)shape->top_k * shape->inter +
                         (long long)(shape->n_shared > 0 ? shape->n_shared : 0) * shape->shared_inter;
  if (shape->hidden > kMaxHidden || hsum > kHCap) return SLICEMOE_E_UNSUPPORTED;
  int dev = 0;
  SM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SLICEMOE_E_UNSUPPORTED;
  if (!g_static_scratch_ptr[dev]) {
    // In host code the array's name is only a handle; the address a kernel can use has to be asked for,
    // with the device that will run the kernel current.
    void* ptr = nullptr;
    SM_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
    if (!ptr) return SLICEMOE_E_CUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  void* ws = g_static_scratch_ptr[dev];
  // The array keeps whatever the previous call left: the header (barrier counters, status) must start at zero.
  SM_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsHOff, (cudaStream_t)stream));
  return run_layer(shape, experts, shared, shape->n_shared, shared_gate_vec, x, T, ids, prec, weights, y, ws, kWsBytes,
                   stream);
}
