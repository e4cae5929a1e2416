// Batch-1 decode of one MoE layer from bit-sliced AMAT weights (Section 4.1 of the paper: an expert
// runs from MSB+LSB slices at full precision or from the MSB slice alone), as ONE persistent kernel.
//
// The work is a pure weight stream: every plane byte is used once, so the bound is HBM bandwidth.
// Design:
//   * One CTA per SM.  A producer thread streams 16-row x <=2048-column plane tiles (<=16 KB, one
//     contiguous run each thanks to the tiled layout) plus their scales / zero-points into an
//     8-stage shared-memory ring with cp.async.bulk + mbarriers.  The producer never waits for the
//     gate/up -> down dependency, so down-projection tiles are already in flight while the grid
//     finishes the first phase.
//   * 8 consumer warps split the K range of a tile.  Nibbles are turned into bf16 (128 + n) pairs with
//     one lop3 per two weights (the plane layout stores them in mma fragment order) and multiplied
//     with the activation vector by mma.sync m16n8k16 (bf16 x bf16 -> fp32): the tensor pipe is used
//     as a wide FMA unit because the plain ALUs cannot unpack + convert + FMA 2 nibbles per byte at
//     HBM rate.  The zero-point and the +128 bias are folded out:
//        sum_k x_k s (q_k - zp) = s (sum_k x_k (q_k + bias) - (bias + zp) sum_{k in group} x_k).
//     h is split into bf16 hi + lo parts for the down projection, so no activation precision is lost.
//   * An epilogue warp reduces the 8 per-warp partial rows, applies SwiGLU, writes h (fp32) to the
//     workspace, takes part in the single grid barrier (bounded spin) and, in the second phase,
//     performs the weighted top-k combine in a fixed order through a last-arriver ticket per
//     16-row output block (deterministic; no float atomics).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace slicemoe {

constexpr int kConsumerWarps = 8;
constexpr int kProducerWarp = 8;
constexpr int kEpilogueWarp = 9;
constexpr int kThreads = 320;
constexpr int kStages = 8;
constexpr int kChunkK = 2048;                              // K columns per ring stage
constexpr int kPlaneStageBytes = 16 * kChunkK / 2;         // 16384
constexpr int kScaleStageBytes = 16 * (kChunkK / 32) * 2;  // 2048 (group 32 is the worst case)
constexpr int kZpStageBytes = 16 * (kChunkK / 32);         // 1024
constexpr int kStageBytes = kPlaneStageBytes + kScaleStageBytes + kZpStageBytes;  // 19456
constexpr int kMaxSlots = SLICEMOE_MAX_TOP_K + SLICEMOE_MAX_SHARED;
constexpr int kMaxHidden = 4096;
constexpr int kHCap = 12288;  // sum of intermediate widths over all slots of a layer
constexpr unsigned long long kWaitCycles = 4000000000ull;  // ~2 s: every device-side wait is bounded

// ---- workspace --------------------------------------------------------------------------------
struct WsHeader {
  unsigned bar_arrive;  // grid barrier: CTAs that finished the gate/up phase
  unsigned depart;      // CTAs that finished the kernel (the last one re-zeroes the header)
  unsigned status;      // SLICEMOE_STATUS_* bits
  unsigned pad[61];
  unsigned ticket[kMaxHidden / 16];  // per 16-row output block: finished (block, slot) tasks
};
constexpr size_t kWsHeaderBytes = sizeof(WsHeader);                     // 1280
constexpr size_t kWsHOff = 2048;                                        // float h[kHCap]
constexpr size_t kWsPOff = kWsHOff + sizeof(float) * kHCap;             // float P[kMaxSlots][hidden]
constexpr size_t kWsStageOff = kWsPOff + sizeof(float) * kMaxSlots * kMaxHidden;
// host-step staging: x bf16[kMaxHidden] | logits f32[512] | ids i32[16] | w f32[16] | prec u8[16] | y f32[kMaxHidden]
constexpr size_t kWsStX = kWsStageOff;
constexpr size_t kWsStLogits = kWsStX + 2 * kMaxHidden;
constexpr size_t kWsStIds = kWsStLogits + 4 * 512;
constexpr size_t kWsStW = kWsStIds + 64;
constexpr size_t kWsStPrec = kWsStW + 64;
constexpr size_t kWsStY = kWsStPrec + 64;
constexpr size_t kWsBytes = kWsStY + 4 * kMaxHidden;

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
  float* ws_p;
  int n_experts, n_shared, k;
  int hidden, inter, shared_inter, group;
  int sigmoid_gate;
};

struct Slot {
  const uint8_t* msb[3];  // gate, up, down
  const uint8_t* lsb[3];
  const uint16_t* sc[3];
  const uint8_t* zp[3];
  int inter;
  int prec;
  float coef;
  int hoff;   // offset of this slot's h in the workspace / shared-memory h vector
  int gated;  // 1: coef is replaced by sigmoid(gate_vec . x)
  int pad_;
};

struct StageDesc {
  uint32_t flags;
  uint16_t slot, rot;
  uint32_t rb;
  uint16_t kstep0, nblocks;
};
enum : uint32_t {
  kFlagLsb = 1,           // this stage carries the LSB plane of the chunk (accumulate onto 16 x MSB sums)
  kFlagMeta = 2,          // last plane of the chunk: scales / zero-points are in the stage; fold the chunk
  kFlagLastOfMatrix = 4,  // last chunk of the matrix row block
  kFlagLastOfTask = 8,    // last matrix of the task: publish partial rows
  kFlagEnd = 16,          // sentinel, no data
  kFlagPrec8 = 32,
  kFlagPhase2 = 64,
};

struct Plan {
  int first_slot[2], first_idx[2], count[2];
  int nslots;
  int last_slot2;  // last slot this CTA touches in the down phase
};

struct SmemLayout {
  // offsets into dynamic shared memory
  static constexpr int ring = 0;
  static constexpr int hs = ring + kStages * kStageBytes;  // uint4[kHCap/4]
  static constexpr int xs = hs + kHCap * 4;                // bf16[kMaxHidden]
  static constexpr int xsum = xs + kMaxHidden * 2;         // float[kMaxHidden/32]
  static constexpr int hsum = xsum + (kMaxHidden / 32) * 4;  // float[kHCap/32]
  static constexpr int partial = hsum + (kHCap / 32) * 4;    // float[2][8][16][2]
  static constexpr int slots = partial + 2 * kConsumerWarps * 16 * 2 * 4;
  static constexpr int desc = slots + kMaxSlots * (int)sizeof(Slot);
  static constexpr int pinfo = desc + kStages * (int)sizeof(StageDesc);  // uint32[2][4]
  static constexpr int plan = pinfo + 32;
  static constexpr int bars = (plan + (int)sizeof(Plan) + 15) & ~15;  // uint64 barriers
  static constexpr int nbars = 2 * kStages + 5;
  static constexpr int dead = bars + nbars * 8;
  static constexpr int total = dead + 16;
};
static_assert(SmemLayout::total <= 227 * 1024, "shared memory budget");
static_assert(sizeof(Slot) % 8 == 0, "slot alignment");

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
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// ---- task enumeration (identical in every role) ---------------------------------------------------
__device__ __forceinline__ int nchunks_of(int K) { return (K + kChunkK - 1) / kChunkK; }
// tasks / stages-per-task of a slot in a phase
__device__ __forceinline__ int slot_ntasks(const Slot& s, int phase, int hidden) {
  return phase == 0 ? s.inter / 16 : hidden / 16;
}
__device__ __forceinline__ int slot_spt(const Slot& s, int phase, int hidden) {
  const int planes = s.prec ? 2 : 1;
  return phase == 0 ? 2 * planes * nchunks_of(hidden) : planes * nchunks_of(s.inter);
}

// First task whose cumulative stage offset is >= bound; returns its ordinal, slot and index.
__device__ void locate_task(const Slot* slots, int nslots, int phase, int hidden, long long bound, int* ord,
                            int* slot, int* idx) {
  long long off = 0;
  int o = 0;
  for (int j = 0; j < nslots; ++j) {
    const int nt = slot_ntasks(slots[j], phase, hidden), sp = slot_spt(slots[j], phase, hidden);
    const long long end = off + (long long)nt * sp;
    if (bound < end) {
      long long i = bound <= off ? 0 : (bound - off + sp - 1) / sp;
      if (i < nt) {
        *ord = o + (int)i;
        *slot = j;
        *idx = (int)i;
        return;
      }
    }
    off = end;
    o += nt;
  }
  *ord = o;
  *slot = nslots;
  *idx = 0;
}

__device__ __forceinline__ void next_task(const Slot* slots, int phase, int hidden, int& slot, int& idx) {
  if (++idx >= slot_ntasks(slots[slot], phase, hidden)) {
    idx = 0;
    ++slot;
  }
}

// ---- consumer: one ring stage ----------------------------------------------------------------------
template <int G>
struct Acc {
  static constexpr int SG = 128 / G;
  float c[2][SG][4];
};

template <int G, bool PHASE2>
__device__ __forceinline__ void consume_blocks(Acc<G>& acc, const uint8_t* stage, int b0, bool v0, int b1, bool v1,
                                               const uint8_t* bvec /* xs or hs + slot offset, byte pointer */,
                                               int kstep0, int lane) {
  constexpr int KS_PER_SG = G / 16;
  const int c = lane & 3;
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    uint4 w0 = make_uint4(0, 0, 0, 0), w1 = make_uint4(0, 0, 0, 0);
    if (v0) w0 = *reinterpret_cast<const uint4*>(stage + (2 * b0 + u) * 512 + lane * 16);
    if (v1) w1 = *reinterpret_cast<const uint4*>(stage + (2 * b1 + u) * 512 + lane * 16);
    const uint32_t ww0[4] = {w0.x, w0.y, w0.z, w0.w};
    const uint32_t ww1[4] = {w1.x, w1.y, w1.z, w1.w};
#pragma unroll
    for (int tw = 0; tw < 4; ++tw) {
      const int sg = (4 * u + tw) / KS_PER_SG;
#pragma unroll
      for (int bi = 0; bi < 2; ++bi) {
        const bool valid = bi ? v1 : v0;
        if (!valid) continue;
        const uint32_t w = bi ? ww1[tw] : ww0[tw];
        const int b = bi ? b1 : b0;
        const int kstep = kstep0 + 8 * b + 4 * u + tw;
        const uint32_t a0 = (w & 0x000f000fu) | 0x43004300u;
        const uint32_t a1 = ((w >> 4) & 0x000f000fu) | 0x43004300u;
        const uint32_t a2 = ((w >> 8) & 0x000f000fu) | 0x43004300u;
        const uint32_t a3 = ((w >> 12) & 0x000f000fu) | 0x43004300u;
        if (!PHASE2) {
          const uint2 bv = *reinterpret_cast<const uint2*>(bvec + (kstep * 16 + 4 * c) * 2);
          mma_bf16(acc.c[bi][sg], a0, a1, a2, a3, bv.x, bv.y);
        } else {
          const uint4 hv = *reinterpret_cast<const uint4*>(bvec + (kstep * 16 + 4 * c) * 4);
          mma_bf16(acc.c[bi][sg], a0, a1, a2, a3, hv.x, hv.y);
          mma_bf16(acc.c[bi][sg], a0, a1, a2, a3, hv.z, hv.w);
        }
      }
    }
  }
}

template <int G>
__device__ void consumer_loop(const DecodeParams& p, uint8_t* smem, int warp, int lane) {
  constexpr int SG = 128 / G;
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const StageDesc* descs = reinterpret_cast<const StageDesc*>(smem + SmemLayout::desc);
  const float* xsum = reinterpret_cast<const float*>(smem + SmemLayout::xsum);
  const float* hsum = reinterpret_cast<const float*>(smem + SmemLayout::hsum);
  float* partial = reinterpret_cast<float*>(smem + SmemLayout::partial);
  uint32_t* pinfo = reinterpret_cast<uint32_t*>(smem + SmemLayout::pinfo);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars, empty0 = bars + 8 * kStages, pfull0 = bars + 16 * kStages,
                 pempty0 = pfull0 + 16, hready = pempty0 + 16;
  unsigned* status = &p.ws->status;

  const int c = lane & 3, g8 = lane >> 2;
  const int r = g8 + 8 * (c & 1);  // the row of the 16-row block this lane folds in the epilogue
  Acc<G> acc;
  float rowacc = 0.f, part0 = 0.f, part1 = 0.f;
  bool h_ready_seen = false;
  int taskcount = 0;

  for (int it = 0;; ++it) {
    const int stage = it % kStages;
    if (!mbar_wait(full0 + 8 * stage, (it / kStages) & 1, dead, status)) return;
    const StageDesc d = descs[stage];
    if (d.flags & kFlagEnd) break;
    const bool phase2 = (d.flags & kFlagPhase2) != 0;
    if (phase2 && !h_ready_seen) {
      if (!mbar_wait(hready, 0, dead, status)) return;
      h_ready_seen = true;
    }
    const Slot& sl = slots[d.slot];
    const uint8_t* stg = smem + SmemLayout::ring + stage * kStageBytes;
    // blocks (128 columns) of this chunk handled by this warp: b0 and b0 + 8
    const int b0 = (warp - d.rot) & 7, b1 = b0 + 8;
    const bool v0 = b0 < d.nblocks, v1 = b1 < d.nblocks;
    if (!(d.flags & kFlagLsb)) {
#pragma unroll
      for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int sg = 0; sg < SG; ++sg)
#pragma unroll
          for (int q = 0; q < 4; ++q) acc.c[bi][sg][q] = 0.f;
    } else {
#pragma unroll
      for (int bi = 0; bi < 2; ++bi)
#pragma unroll
        for (int sg = 0; sg < SG; ++sg)
#pragma unroll
          for (int q = 0; q < 4; ++q) acc.c[bi][sg][q] *= 16.f;
    }
    if (!phase2) {
      consume_blocks<G, false>(acc, stg, b0, v0, b1, v1, smem + SmemLayout::xs, d.kstep0, lane);
    } else {
      consume_blocks<G, true>(acc, stg, b0, v0, b1, v1, smem + SmemLayout::hs + sl.hoff * 4, d.kstep0, lane);
    }
    if (d.flags & kFlagMeta) {
      const uint16_t* ms = reinterpret_cast<const uint16_t*>(stg + kPlaneStageBytes);
      const uint8_t* mz = stg + kPlaneStageBytes + kScaleStageBytes;
      const float* xs_sum = phase2 ? hsum + (sl.hoff + d.kstep0 * 16) / G : xsum + (d.kstep0 * 16) / G;
      const bool p8 = (d.flags & kFlagPrec8) != 0;
#pragma unroll
      for (int bi = 0; bi < 2; ++bi) {
        const bool valid = bi ? v1 : v0;
        if (!valid) continue;
        const int b = bi ? b1 : b0;
#pragma unroll
        for (int sg = 0; sg < SG; ++sg) {
          const int gl = b * SG + sg;
          const float cv = (c & 1) ? acc.c[bi][sg][2] : acc.c[bi][sg][0];
          const float s = __half2float(__ushort_as_half(ms[gl * 16 + r]));
          const int z = mz[gl * 16 + r];
          const float X = xs_sum[gl];
          // both slices: s (16 Cm + Cl - (16*128 + 128 + zp) X); MSB only: 16 s (Cm - (128 + (zp >> 4)) X)
          if (p8) rowacc = fmaf(s, fmaf(-(2176.f + (float)z), X, cv), rowacc);
          else rowacc = fmaf(16.f * s, fmaf(-(128.f + (float)(z >> 4)), X, cv), rowacc);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + 8 * stage);
    if (d.flags & kFlagLastOfMatrix) {
      if (!phase2 && !(d.flags & kFlagLastOfTask)) part0 = rowacc;  // gate
      else part1 = rowacc;                                            // up, or down
      rowacc = 0.f;
    }
    if (d.flags & kFlagLastOfTask) {
      const int buf = taskcount & 1;
      if (!mbar_wait(pempty0 + 8 * buf, ((taskcount >> 1) & 1) ^ 1, dead, status)) return;
      if (c < 2) {
        float* dst = partial + ((buf * kConsumerWarps + warp) * 16 + r) * 2;
        dst[0] = part0;
        dst[1] = part1;
      }
      if (warp == 0 && lane == 0) {
        pinfo[buf * 4 + 0] = phase2 ? 1u : 0u;
        pinfo[buf * 4 + 1] = d.slot;
        pinfo[buf * 4 + 2] = d.rb;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(pfull0 + 8 * buf);
      ++taskcount;
      part0 = part1 = 0.f;
    }
  }
}

// ---- producer --------------------------------------------------------------------------------------
__device__ void producer_loop(const DecodeParams& p, uint8_t* smem) {
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  StageDesc* descs = reinterpret_cast<StageDesc*>(smem + SmemLayout::desc);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars, empty0 = bars + 8 * kStages;
  const uint32_t ring = smem_u32(smem + SmemLayout::ring);
  unsigned* status = &p.ws->status;
  const int G = p.group;
  int it = 0;
  bool ok = true;
  for (int phase = 0; phase < 2 && ok; ++phase) {
    int slot = plan.first_slot[phase], idx = plan.first_idx[phase];
    for (int n = 0; n < plan.count[phase] && ok; ++n) {
      const Slot& s = slots[slot];
      const int K = phase == 0 ? p.hidden : s.inter;
      const int nch = nchunks_of(K);
      const int nmat = phase == 0 ? 2 : 1;
      const int nplanes = s.prec ? 2 : 1;
      for (int m = 0; m < nmat && ok; ++m) {
        const int mat = phase == 0 ? m : 2;
        for (int ch = 0; ch < nch && ok; ++ch) {
          const int k0 = ch * kChunkK;
          const int kc = min(kChunkK, K - k0);
          for (int pl = 0; pl < nplanes; ++pl) {
            const int stage = it % kStages;
            if (!mbar_wait(empty0 + 8 * stage, ((it / kStages) & 1) ^ 1, dead, status)) {
              ok = false;
              break;
            }
            const bool has_meta = (pl == nplanes - 1);
            StageDesc d;
            d.flags = (pl ? kFlagLsb : 0u) | (has_meta ? kFlagMeta : 0u) | (s.prec ? kFlagPrec8 : 0u) |
                      (phase ? kFlagPhase2 : 0u);
            if (has_meta && ch == nch - 1) {
              d.flags |= kFlagLastOfMatrix;
              if (m == nmat - 1) d.flags |= kFlagLastOfTask;
            }
            d.slot = (uint16_t)slot;
            d.rot = (uint16_t)(n & 7);
            d.rb = (uint32_t)idx;
            d.kstep0 = (uint16_t)(k0 / 16);
            d.nblocks = (uint16_t)(kc / 128);
            descs[stage] = d;
            const uint32_t plane_bytes = (uint32_t)kc * 8u;
            const uint32_t ngc = (uint32_t)(kc / G);
            const uint32_t bytes = plane_bytes + (has_meta ? ngc * 48u : 0u);
            const uint32_t bar = full0 + 8 * stage;
            const uint32_t dst = ring + stage * kStageBytes;
            mbar_arrive_expect_tx(bar, bytes);
            const uint8_t* plane = pl ? s.lsb[mat] : s.msb[mat];
            bulk_g2s(dst, plane + ((size_t)idx * (K >> 6) + (k0 >> 6)) * 512, plane_bytes, bar);
            if (has_meta) {
              const size_t mo = ((size_t)idx * (K / G) + (k0 / G)) * 16;
              bulk_g2s(dst + kPlaneStageBytes, s.sc[mat] + mo, ngc * 32u, bar);
              bulk_g2s(dst + kPlaneStageBytes + kScaleStageBytes, s.zp[mat] + mo, ngc * 16u, bar);
            }
            ++it;
          }
        }
      }
      next_task(slots, phase, p.hidden, slot, idx);
    }
  }
  if (ok) {
    const int stage = it % kStages;
    if (mbar_wait(empty0 + 8 * stage, ((it / kStages) & 1) ^ 1, dead, status)) {
      StageDesc d;
      d.flags = kFlagEnd;
      d.slot = d.rot = 0;
      d.rb = 0;
      d.kstep0 = d.nblocks = 0;
      descs[stage] = d;
      mbar_arrive(full0 + 8 * stage);
      ++it;
    }
  }
  // Never leave the CTA with bulk copies still landing in its shared memory: wait (bounded) for the
  // last kStages armed barriers.  In the normal path they have all completed long ago.
  for (int j = max(0, it - kStages); j < it; ++j) {
    const uint32_t bar = full0 + 8 * (j % kStages);
    const long long t0 = clock64();
    while (!mbar_try(bar, (j / kStages) & 1)) {
      if ((unsigned long long)(clock64() - t0) > kWaitCycles) break;
    }
  }
}

// ---- epilogue warp ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ void load_h_to_smem(const DecodeParams& p, uint8_t* smem, int lane, int slot_lo, int slot_hi) {
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  uint4* hs = reinterpret_cast<uint4*>(smem + SmemLayout::hs);
  float* hsum = reinterpret_cast<float*>(smem + SmemLayout::hsum);
  const int lanes_per_group = p.group / 4;  // 8, 16 or 32 consecutive lanes cover one group
  for (int j = slot_lo; j <= slot_hi; ++j) {
    const int hoff = slots[j].hoff, n4 = slots[j].inter / 4;
    for (int i = lane; i < n4; i += 32) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(p.ws_h + hoff) + i);
      const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y),
                          h2 = __float2bfloat16_rn(v.z), h3 = __float2bfloat16_rn(v.w);
      const float f0 = __bfloat162float(h0), f1 = __bfloat162float(h1), f2 = __bfloat162float(h2),
                  f3 = __bfloat162float(h3);
      const float l0 = v.x - f0, l1 = v.y - f1, l2 = v.z - f2, l3 = v.w - f3;
      const __nv_bfloat16 g0 = __float2bfloat16_rn(l0), g1 = __float2bfloat16_rn(l1),
                          g2 = __float2bfloat16_rn(l2), g3 = __float2bfloat16_rn(l3);
      uint4 o;
      o.x = pack_bf16x2(f0, f1);
      o.y = pack_bf16x2(f2, f3);
      o.z = pack_bf16x2(l0, l1);
      o.w = pack_bf16x2(l2, l3);
      hs[hoff / 4 + i] = o;
      // group sum of what the tensor cores will actually multiply: hi + lo
      float ssum = (f0 + __bfloat162float(g0)) + (f1 + __bfloat162float(g1)) + (f2 + __bfloat162float(g2)) +
                   (f3 + __bfloat162float(g3));
      for (int off = 1; off < lanes_per_group; off <<= 1) ssum += __shfl_xor_sync(0xffffffffu, ssum, off);
      if ((lane & (lanes_per_group - 1)) == 0) hsum[(hoff + 4 * i) / p.group] = ssum;
    }
  }
}

__device__ void epilogue_loop(const DecodeParams& p, uint8_t* smem, int lane) {
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  const float* partial = reinterpret_cast<const float*>(smem + SmemLayout::partial);
  const uint32_t* pinfo = reinterpret_cast<const uint32_t*>(smem + SmemLayout::pinfo);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t pfull0 = bars + 16 * kStages, pempty0 = pfull0 + 16, hready = pempty0 + 16;
  unsigned* status = &p.ws->status;
  const int nslots = plan.nslots;

  // Qwen-style shared-expert gate: sigmoid(v . x), needed only for the final combine.
  if (p.sigmoid_gate && p.n_shared > 0) {
    const __nv_bfloat16* xs = reinterpret_cast<const __nv_bfloat16*>(smem + SmemLayout::xs);
    float dot = 0.f;
    for (int i = lane; i < p.hidden; i += 32) dot = fmaf(p.gate_vec[i], __bfloat162float(xs[i]), dot);
    for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    const float cgate = 1.f / (1.f + expf(-dot));
    if (lane == 0)
      for (int j = 0; j < nslots; ++j)
        if (slots[j].gated) slots[j].coef = cgate;
    __syncwarp();
  }

  const int total = plan.count[0] + plan.count[1];
  for (int tc = 0;; ++tc) {
    if (tc == plan.count[0]) {
      // ---- grid barrier: every CTA has written its part of h ----
      __threadfence();
      __syncwarp();
      if (lane == 0) {
        atomicAdd(&p.ws->bar_arrive, 1u);
        const long long t0 = clock64();
        while (ld_acquire_u32(&p.ws->bar_arrive) < gridDim.x) {
          __nanosleep(64);
          if (*dead) break;
          if ((unsigned long long)(clock64() - t0) > kWaitCycles) {
            *dead = 1;
            atomicOr(status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
            break;
          }
        }
      }
      __syncwarp();
      if (*dead) return;
      if (plan.count[1] > 0) load_h_to_smem(p, smem, lane, plan.first_slot[1], plan.last_slot2);
      __syncwarp();
      if (lane == 0) mbar_arrive(hready);
    }
    if (tc == total) break;
    const int buf = tc & 1;
    if (!mbar_wait(pfull0 + 8 * buf, (tc >> 1) & 1, dead, status)) return;
    const uint32_t phase2 = pinfo[buf * 4 + 0], slot = pinfo[buf * 4 + 1], rb = pinfo[buf * 4 + 2];
    float a = 0.f, b = 0.f;
    if (lane < 16) {
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        const float* src = partial + ((buf * kConsumerWarps + w) * 16 + lane) * 2;
        a += src[0];
        b += src[1];
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(pempty0 + 8 * buf);
    if (!phase2) {
      if (lane < 16) {
        const float h = a / (1.f + expf(-a)) * b;  // silu(gate) * up
        p.ws_h[slots[slot].hoff + rb * 16 + lane] = h;
      }
    } else {
      if (lane < 16) p.ws_p[(size_t)slot * p.hidden + rb * 16 + lane] = b;
      __threadfence();
      __syncwarp();
      unsigned ticket = 0;
      if (lane == 0) ticket = atomicAdd(&p.ws->ticket[rb], 1u);
      ticket = __shfl_sync(0xffffffffu, ticket, 0);
      if (ticket == (unsigned)(nslots - 1)) {
        // last (block, slot) task of this output block: weighted combine in slot order
        __threadfence();
        if (lane < 16) {
          float yv = 0.f;
          for (int j = 0; j < nslots; ++j)
            yv = fmaf(slots[j].coef, __ldcg(p.ws_p + (size_t)j * p.hidden + rb * 16 + lane), yv);
          p.y[rb * 16 + lane] = yv;
        }
        if (lane == 0) p.ws->ticket[rb] = 0;
      }
    }
  }
}

// ---- the kernel ------------------------------------------------------------------------------------
template <int G>
__global__ void __launch_bounds__(kThreads, 1) decode_layer_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);
  int* dead = reinterpret_cast<int*>(smem + SmemLayout::dead);

  // x -> shared memory (bf16, as is)
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.x);
    uint32_t* dst = reinterpret_cast<uint32_t*>(smem + SmemLayout::xs);
    for (int i = tid; i < p.hidden / 2; i += kThreads) dst[i] = src[i];
  }
  if (tid == 0) {
    *dead = 0;
    // slot table: routed experts in list order, then the shared experts
    int n = 0, hoff = 0;
    for (int j = 0; j < p.k; ++j) {
      const int e = p.ids[j];
      if (e < 0 || e >= p.n_experts) {
        atomicOr(&p.ws->status, (unsigned)SLICEMOE_STATUS_BAD_EXPERT_ID);
        continue;
      }
      const slicemoe_expert& ex = p.experts[e];
      Slot& s = slots[n];
      const slicemoe_mat* m[3] = {&ex.gate, &ex.up, &ex.down};
      for (int q = 0; q < 3; ++q) {
        s.msb[q] = reinterpret_cast<const uint8_t*>(m[q]->msb);
        s.lsb[q] = reinterpret_cast<const uint8_t*>(m[q]->lsb);
        s.sc[q] = m[q]->scale;
        s.zp[q] = m[q]->zp;
      }
      s.inter = p.inter;
      s.prec = (p.prec[j] != 0 && s.lsb[0] && s.lsb[1] && s.lsb[2]) ? 1 : 0;
      s.coef = p.weights[j];
      s.gated = 0;
      s.hoff = hoff;
      hoff += p.inter;
      ++n;
    }
    for (int j = 0; j < p.n_shared; ++j) {
      const slicemoe_expert& ex = p.shared[j];
      Slot& s = slots[n];
      const slicemoe_mat* m[3] = {&ex.gate, &ex.up, &ex.down};
      for (int q = 0; q < 3; ++q) {
        s.msb[q] = reinterpret_cast<const uint8_t*>(m[q]->msb);
        s.lsb[q] = reinterpret_cast<const uint8_t*>(m[q]->lsb);
        s.sc[q] = m[q]->scale;
        s.zp[q] = m[q]->zp;
      }
      s.inter = p.shared_inter;
      s.prec = 1;
      s.coef = 1.f;
      s.gated = p.sigmoid_gate;
      s.hoff = hoff;
      hoff += p.shared_inter;
      ++n;
    }
    plan->nslots = n;
    // static partition: equal shares of ring stages per phase, at task granularity
    for (int phase = 0; phase < 2; ++phase) {
      long long S = 0;
      for (int j = 0; j < n; ++j) S += (long long)slot_ntasks(slots[j], phase, p.hidden) * slot_spt(slots[j], phase, p.hidden);
      const long long lo = ((long long)blockIdx.x * S + gridDim.x - 1) / gridDim.x;
      const long long hi = ((long long)(blockIdx.x + 1) * S + gridDim.x - 1) / gridDim.x;
      int o0, s0, i0, o1, s1, i1;
      locate_task(slots, n, phase, p.hidden, lo, &o0, &s0, &i0);
      locate_task(slots, n, phase, p.hidden, hi, &o1, &s1, &i1);
      plan->first_slot[phase] = s0;
      plan->first_idx[phase] = i0;
      plan->count[phase] = o1 - o0;
      if (phase == 1) plan->last_slot2 = (i1 == 0) ? s1 - 1 : s1;
    }
    if (plan->last_slot2 >= n) plan->last_slot2 = n - 1;
    // barriers
    const uint32_t bars = smem_u32(smem + SmemLayout::bars);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bars + 8 * s, 1);                              // full: producer's expect_tx arrive
      mbar_init(bars + 8 * kStages + 8 * s, kConsumerWarps);   // empty: one arrive per consumer warp
    }
    mbar_init(bars + 16 * kStages + 0, kConsumerWarps);  // pfull[0]
    mbar_init(bars + 16 * kStages + 8, kConsumerWarps);  // pfull[1]
    mbar_init(bars + 16 * kStages + 16, 1);              // pempty[0]
    mbar_init(bars + 16 * kStages + 24, 1);              // pempty[1]
    mbar_init(bars + 16 * kStages + 32, 1);              // hready
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  // group sums of x
  {
    const __nv_bfloat16* xs = reinterpret_cast<const __nv_bfloat16*>(smem + SmemLayout::xs);
    float* xsum = reinterpret_cast<float*>(smem + SmemLayout::xsum);
    for (int g = tid; g < p.hidden / G; g += kThreads) {
      float s = 0.f;
      for (int i = 0; i < G; ++i) s += __bfloat162float(xs[g * G + i]);
      xsum[g] = s;
    }
  }
  if (plan->nslots == 0 && blockIdx.x == 0)
    for (int i = tid; i < p.hidden; i += kThreads) p.y[i] = 0.f;
  __syncthreads();

  if (warp < kConsumerWarps) {
    consumer_loop<G>(p, smem, warp, lane);
  } else if (warp == kProducerWarp) {
    if (lane == 0) producer_loop(p, smem);
  } else {
    epilogue_loop(p, smem, lane);
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
  p.ws_p = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + kWsPOff);
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
