// Batch-1 decode of one MoE layer from bit-sliced AMAT weights (Section 4.1 of the paper: an expert
// runs from MSB+LSB slices at full precision or from the MSB slice alone), as ONE persistent kernel.
//
// The work is a pure weight stream: every plane byte is used once, so the bound is HBM bandwidth and
// everything else is arranged so that the stream never stops.
//   * One CTA per SM: 16 consumer warps in 4 groups, one epilogue warp, two producer warps (6 lanes each,
//     one per bulk copy of a chunk).  The 4 warps of a group split a chunk's 128-column blocks, so the
//     per-chunk bookkeeping is paid by 4 warps, not 16, while 4 chunks are in work at any time.  The
//     schedule is a pure function of the slot table, so every role enumerates it for itself and only
//     data and barrier phases pass between them.  The producer streams chunks - 16 rows x <=2048 columns: the MSB plane tile,
//     the LSB plane tile when the expert runs at 8 bits (<=16 KB each, one contiguous run thanks to the
//     tiled layout), scales and zero-points - into a ring of eight 19 KB units with cp.async.bulk +
//     mbarriers.  They never wait for the gate/up -> down dependency, so down-projection tiles are
//     already in flight (up to the whole ring) while the grid exchanges h.
//   * Integer arithmetic on the tensor pipe.  The activation vector (x, later h) is converted once,
//     per 128-element block, to fixed point relative to the block's largest magnitude and split into
//     three balanced base-256 digits (int8).  The digits sit in separate columns of the B operand of
//     mma.sync m16n8k32 (u8 x s8 -> s32); the A operand is the raw nibble plane: the layout stores
//     the two row halves of a fragment in the low and high nibbles of each byte, so `w & 0x0f0f0f0f`
//     and `w` itself are the whole unpack (the second half then carries 16 x its rows plus the first
//     half's, which one subtraction and the fold weight undo).  Sums are exact in int32; MSB and LSB planes combine as
//     16 * Cm + Cl.  Scale and zero-point are applied once per (row, group):
//        sum_k x_k s (q_k - zp) = s (sum_k q_k x_k - zp sum_{k in group} x_k).
//     The plain ALUs could not unpack + convert + FMA two weights per byte at HBM rate; this costs
//     about seven instructions per 512 weights.
//   * Phase 1 (gate/up + SwiGLU): tasks are (expert slot, 16-row block), split over the CTAs by
//     bytes.  The epilogue warp adds the warps' partial rows, applies SwiGLU and writes h (fp32) to
//     the workspace.  There is no barrier between the phases: readers poll the h words themselves (two
//     buffers used by alternate launches, each left "empty" by the launch before; every wait bounded).
//   * Phase 2 (down + weighted combine): a task is a 16-row block of the OUTPUT over ALL slots, so
//     the top-k combine stays inside the CTA: no atomics, no cross-CTA reduction, fixed summation
//     order (results are bit-reproducible).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "route.cuh"

namespace slicemoe {

constexpr int kConsumerWarps = 16;
constexpr int kGroups = 4;       // consumer groups: a phase-1 task belongs to one group, phase-2 chunks go round-robin
constexpr int kGroupWarps = 4;   // warps of a group; they split the 128-column blocks of the chunk
static_assert(kGroups * kGroupWarps == kConsumerWarps, "groups");
constexpr int kEpilogueWarp = kConsumerWarps;
constexpr int kProducerWarp = kConsumerWarps + 1;  // first of kProducers producer warps
constexpr int kProducers = 2;                      // they take alternate tasks (phase 1) / chunks (phase 2)
constexpr int kThreads = 32 * (kConsumerWarps + 1 + kProducers);
constexpr int kUnits2 = 16;                        // at most this many (smaller) units in phase 2
constexpr int kFull2PerGroup = 8;  // >= chunks one producer can have in flight in phase 2 (kUnits2 / 2 units)
constexpr int kUnits = 8;                                 // ring units; a chunk takes one per plane
constexpr int kChunkK = 2048;                             // K columns per chunk (16 blocks of 128)
constexpr int kBlocksPerWarp = kChunkK / 128 / kGroupWarps;
constexpr int kPlaneUnitBytes = 16 * kChunkK / 2;         // 16384
constexpr int kScaleUnitBytes = 16 * (kChunkK / 32) * 2;  // 2048 (group 32 is the worst case)
constexpr int kZpUnitBytes = 16 * (kChunkK / 32);         // 1024
constexpr int kUnitBytes = kPlaneUnitBytes + kScaleUnitBytes + kZpUnitBytes;  // 19456
constexpr int kMaxSlots = SLICEMOE_MAX_TOP_K + SLICEMOE_MAX_SHARED;
constexpr int kMaxHidden = 4096;
constexpr int kHCap = 12288;  // sum of intermediate widths over all slots of a layer
constexpr int kMaxMine = 32;   // phase-2 chunks one consumer group can have: (slots + kHCap / kChunkK) chunks per
                               // output row block, at most 4 row blocks per CTA, shared by 4 groups
// Every device-side wait is bounded: by this many clock cycles (about 50 ms; a layer takes tens of microseconds)
// unless the workspace header carries another limit.
constexpr unsigned long long kWaitCycles = 100000000ull;

// ---- optional time stamps ------------------------------------------------------------------------
// A build with -DSLICEMOE_TRACE records, per CTA and for the most recent launch, when its roles passed a few
// points: clock64 relative to the CTA's start (and the global timer at three of them).  slicemoe_trace_read hands
// the table out; `python -m paper_2512_12990_b200.trace` prints the timeline.  The ordinary build has none of it.
#ifdef SLICEMOE_TRACE
constexpr int kTraceSlots = 48;
__device__ long long g_trace[256][kTraceSlots];
__shared__ long long s_trace_t0;
__device__ __forceinline__ long long trace_gtime() {
  long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define SM_TRACE(i)                                                                   \
  do {                                                                                \
    if ((threadIdx.x & 31) == 0 && blockIdx.x < 256) g_trace[blockIdx.x][i] = clock64() - s_trace_t0; \
  } while (0)
#define SM_TRACE_G(i)                                                                 \
  do {                                                                                \
    if ((threadIdx.x & 31) == 0 && blockIdx.x < 256) g_trace[blockIdx.x][i] = trace_gtime(); \
  } while (0)
#else
#define SM_TRACE(i) do { } while (0)
#define SM_TRACE_G(i) do { } while (0)
#endif
// stamp numbers (clock64 unless noted): 1 dependency wait over, 2 plan built (warp 0), 3 x as digits (warp 3),
// 4 prologue barrier passed, 5-8 gate/up phase done (consumer groups 0-3), 9 list of down chunks built (warp 0),
// 10 own h blocks in digits (warp 0), 11 down phase done (warp 0), 12 last h value written, 13 y written;
// 14-17 own h blocks in digits (first warp of consumer groups 0-3), 23-26 the h blocks of the group's last down chunk
// flagged, 27-30 down phase done (first warp of groups 0-3), 31 producer 0 begins the down tiles, 18-19 producer 0 / 1
// has requested all its down tiles, 32-39 producer 0 has requested its gate/up chunk 0-7, 40-43 / 44-47 the down
// chunks of producer 0 / 1 have landed (in the order it waits for them); global timer: 20 kernel entry, 21 dependency
// wait over, 22 y written

// ---- workspace --------------------------------------------------------------------------------
struct WsHeader {
  unsigned readers;     // CTAs of the running launch that have read `epoch` (the last one moves it on)
  unsigned epoch;       // launches so far on this workspace; its parity selects the h buffer
  unsigned status;      // SLICEMOE_STATUS_* bits
  unsigned extra_arrivals;         // != 0: h never counts as complete (slicemoe_workspace_set_wait; 0 in real use)
  unsigned long long wait_cycles;  // limit of the device-side waits, 0 = kWaitCycles
};
// The intermediate vector h crosses the grid through the workspace without a barrier: there are two buffers,
// used by alternate launches; a buffer's words all hold kHEmpty when its launch begins (the launch before
// wrote that, after the launch before it had read them; slicemoe_workspace_init writes both), a CTA stores its
// h values with plain stores, and a reader polls the words it needs until none of them is kHEmpty any more.
// kHEmpty is a NaN pattern that no arithmetic produces (the sign bit of a generated NaN is clear).
constexpr unsigned kHEmpty = 0xffffffffu;
constexpr size_t kWsHOff = 2048;                              // float h[2][kHCap]
constexpr size_t kWsStageOff = kWsHOff + 2 * sizeof(float) * kHCap;
// host-step staging: x bf16[kMaxHidden] | logits f32[512] | ids i32[16] | w f32[16] | prec u8[16] | y f32[kMaxHidden]
constexpr size_t kWsStX = kWsStageOff;
constexpr size_t kWsStLogits = kWsStX + 2 * kMaxHidden;
constexpr size_t kWsStIds = kWsStLogits + 4 * 512;
constexpr size_t kWsStW = kWsStIds + 64;
constexpr size_t kWsStPrec = kWsStW + 64;
constexpr size_t kWsStY = kWsStPrec + 64;
constexpr size_t kWsBytes = kWsStY + 4 * kMaxHidden;
static_assert(sizeof(WsHeader) <= kWsHOff, "workspace header");
static_assert(kWsStLogits + 4 * 512 <= kWsStIds, "x and the logits fit the staging area back to back too");

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
  int shift;  // b_high - b_low: the MSB slice is worth 2^shift of the LSB slice's units
  // the routing lists were complete before the work ahead of this kernel in the stream began: they are read, and
  // the routed experts' tiles requested, while that work is still running
  int lists_resident;
  // fused routing (logits != nullptr): the list is computed from the router logits in the prologue instead of
  // read from ids / prec / weights, and written to the *_out arrays (each may be null) by one CTA
  const float* logits;
  const float* bias;
  int renorm, rank_high;
  float tau;
  int32_t* ids_out;
  uint8_t* prec_out;
  float* weights_out;
};

struct Slot {
  const uint8_t* ptr[3][4];  // [gate, up, down][MSB plane, LSB plane, scales, zero-points]: slicemoe_expert's pointers
  int inter;
  int prec;
  float coef;
  int hoff;   // offset of this slot's h in the workspace / in the digit buffer
  int gated;  // 1: the combine weight is sigmoid(gate_vec . x)
  int pad_;
};

// The schedule of a CTA.
//   phase 1: tasks n = 0 .. count1-1 are (slot, 16-row block) pairs: first count_s tasks of the shared experts,
//     from (slot_s, idx_s) on - this part follows from the shape alone, so its tiles can be requested before the
//     routing list is known - then the routed tasks from (first_slot, first_idx) on.  A
//     task of an 8-bit slot is 2 * nch chunks (gate then up; nch = 2048-column chunks of hidden), each two
//     units (MSB tile, LSB tile); a task of a 4-bit slot is nch chunks, each two units (the gate's MSB tile
//     and the up's).  Every phase-1 chunk takes two units.  Task n is consumed by group n % kGroups and
//     produced by producer n % kProducers; which units and barriers a chunk uses is stated at `struct Bars`.
//   phase 2: tasks m = 0 .. count2-1 are the output row blocks blockIdx.x + m * gridDim.x; each is one run of
//     chunks over the slots in order (p2c[j] chunks and p2u[j] units come before slot j), two units per
//     chunk for 8-bit slots and one for 4-bit slots.  Chunk number c is consumed by group c % kGroups and
//     produced by producer c % kProducers.
//     Phase 2 re-cuts the ring into nunits2 units of unit2_bytes, just large enough for the widest down
//     chunk (plane area, then scales at scale2_off, zero-points at zp2_off), so that more - for the
//     benchmark shapes all - of the phase's tiles are in shared memory before h arrives.
struct Plan {
  int slot_s, idx_s, count_s;
  int hpar;         // which h buffer this launch uses
  int never_ready;  // the time-out exercise: treat h as never complete
  int first_slot, first_idx, count1;
  int count2;
  int nslots;
  int htotal;   // sum of the slots' intermediate widths
  float gate;   // sigmoid(gate_vec . x) when the shared experts are gated
  int unit2_bytes, nunits2, scale2_off, zp2_off;
  short p2c[kMaxSlots + 1], p2u[kMaxSlots + 1];
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
  static constexpr int partial = xinv + (kMaxHidden / 128) * 4;  // float2 [warps][16]
  static constexpr int p2list = partial + kConsumerWarps * 16 * 2 * 4;  // uint4 [warps][kMaxMine]: a warp's phase-2 chunks
  static constexpr int slots = p2list + kConsumerWarps * kMaxMine * 16;
  static constexpr int plan = slots + kMaxSlots * (int)sizeof(Slot);
  static constexpr int bars = (plan + (int)sizeof(Plan) + 15) & ~15;  // uint64 barriers
  static constexpr int nbars = 2 * kUnits + kGroups * kFull2PerGroup + kUnits2 + 2 * kGroups + 6;
  static constexpr int dead = bars + nbars * 8;  // int dead flag; 8 bytes on, the wait limit in cycles
  static constexpr int hready = dead + 16;       // uint8 [kHCap / 128]: the 128-block of h is in shared memory as digits
  static constexpr int total = hready + kHCap / 128;
};
static_assert(SmemLayout::total <= 227 * 1024, "shared memory budget");
static_assert(sizeof(Slot) % 8 == 0, "slot alignment");
static_assert(SmemLayout::slots % 8 == 0 && SmemLayout::hdig % 16 == 0 && SmemLayout::xdig % 16 == 0 &&
                  SmemLayout::plan % 8 == 0 && SmemLayout::partial % 8 == 0 && SmemLayout::p2list % 16 == 0,
              "alignment");

// Barriers.  Every barrier has ONE waiter that meets its phases strictly in order, so a parity wait can never
// be a phase off (mbarrier.try_wait.parity only tells the current phase from the one before it):
//   - a chunk's "full" barrier belongs to the consumer group that consumes it: group g's i-th chunk of a phase
//     uses full[g][i % 2] in phase 1 and full2[g][i % kFull2PerGroup] in phase 2, armed with the chunk's bytes by
//     the producer that serves the group (group g is served by producer g % kProducers in both phases);
//   - an "empty" barrier belongs to the producer that refills the space: producer P owns half of the ring and
//     walks it in order.  Phase 1: P's j-th chunk takes the unit pair (4 P + 2 (j % 2), + 1) and waits on
//     empty[2 P + j % 2]; phase 2: P's units are [P h, P h + h), h = nunits2 / 2, taken in running order, one
//     empty2 barrier per unit (an arrive from each warp of the group that consumed it).
// pfull1 / pempty1 per group (phase-1 partial rows to the epilogue warp and back), pfull2 / pempty2 (phase-2
// partial rows of all warps), p1_done (every consumer warp is through with phase 1, so the ring may be re-cut), plan_ready (the
// routed part of the plan and the routed slots stand: the producers wait for it after the shared experts' tasks).
struct Bars {
  static constexpr int full = 0, empty = kUnits, full2 = 2 * kUnits, empty2 = full2 + kGroups * kFull2PerGroup,
                       pfull1 = empty2 + kUnits2,
                       pempty1 = pfull1 + kGroups, pfull2 = pempty1 + kGroups, pempty2 = pfull2 + 1, hx_go = pfull2 + 2,
                       hs_ready = pfull2 + 3, p1_done = pfull2 + 4, plan_ready = pfull2 + 5, count = pfull2 + 6;
};

static_assert(Bars::count <= SmemLayout::nbars, "barrier storage");

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
// The CTA's wait limit sits 8 bytes behind its dead flag.
__device__ __forceinline__ unsigned long long wait_limit(volatile int* dead) {
  return *reinterpret_cast<volatile unsigned long long*>(dead + 2);
}
// Bounded wait.  Returns false (and raises the CTA's dead flag) when the limit is hit or another
// role of this CTA already gave up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* dead, unsigned* status) {
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*dead) return false;
    if ((unsigned long long)(clock64() - t0) > wait_limit(dead)) {
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
// Weights are used once per token: they go through L2 marked evict-first, so that the stream does not push out
// what every launch uses again (the kernel's own instructions, expert tables, h).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// d = a * b (no accumulator input: the first step of a chain)
__device__ __forceinline__ void mma_u8s8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  const int z = 0;
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(z));
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
// balanced base-256 digits d0 + 256 d1 + 65536 d2 (each in int8 range; the low byte of X read as a signed
// byte is d0, and so on up), stored in B-fragment order; the weighted digit sums of every group of G
// elements (the zero-point term of the fold) and the block's 2^-e.
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
  // Z = (X + 0x808080) ^ 0x808080 holds the three digits in its bytes: adding 128 to a byte and flipping its top
  // bit back leaves the byte read as a signed digit, and the carry into the next byte is exactly what remains
  // after taking that digit (X1 = (X + 128) >> 8, and so on up).
  uint32_t Z[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int X = max(-4194304, min(4194304, __float2int_rn(v[j] * scale)));
    Z[j] = (uint32_t)(X + 0x808080) ^ 0x808080u;
  }
  // byte i of each of the four values -> one word (value j in byte j)
  const uint32_t d0 = __byte_perm(__byte_perm(Z[0], Z[1], 0x0040), __byte_perm(Z[2], Z[3], 0x0040), 0x5410);
  const uint32_t d1 = __byte_perm(__byte_perm(Z[0], Z[1], 0x0051), __byte_perm(Z[2], Z[3], 0x0051), 0x5410);
  const uint32_t d2 = __byte_perm(__byte_perm(Z[0], Z[1], 0x0062), __byte_perm(Z[2], Z[3], 0x0062), 0x5410);
  const int k = k0 + 4 * lane;
  *reinterpret_cast<uint32_t*>(dig + digit_offset(k, 0)) = d0;
  *reinterpret_cast<uint32_t*>(dig + digit_offset(k, 1)) = d1;
  *reinterpret_cast<uint32_t*>(dig + digit_offset(k, 2)) = d2;
  constexpr int lanes_per_group = G / 4;  // 8, 16 or 32 consecutive lanes cover one group
  const unsigned gmask = lanes_per_group == 32 ? 0xffffffffu
                                               : ((1u << lanes_per_group) - 1u) << (lane & ~(lanes_per_group - 1));
  const int s0 = __reduce_add_sync(gmask, __dp4a((int)d0, 0x01010101, 0));  // sums of the signed bytes
  const int s1 = __reduce_add_sync(gmask, __dp4a((int)d1, 0x01010101, 0));
  const int s2 = __reduce_add_sync(gmask, __dp4a((int)d2, 0x01010101, 0));
  if ((lane & (lanes_per_group - 1)) == 0) {
    sumw[(k / G) * 2 + 0] = (float)s0 + 256.f * (float)s1;
    sumw[(k / G) * 2 + 1] = 65536.f * (float)s2;
  }
  if (lane == 0) inv[k0 >> 7] = __uint_as_float((unsigned)(127 - e) << 23);
}

// ---- schedule enumeration (identical in every role) ----------------------------------------------------
__device__ __forceinline__ int nchunks_of(int K) { return (K + kChunkK - 1) / kChunkK; }
enum ChunkMode { kModeSingle = 0, kModeBoth = 1, kModePair = 2 };

// The phase-1 tasks of a CTA in order: `slot`, `idx` name task n once at(n) has been called for it.
struct TaskWalk {
  int slot, idx;
  __device__ __forceinline__ void start(const Plan& plan) {
    slot = plan.slot_s;
    idx = plan.idx_s;
  }
  __device__ __forceinline__ void at(const Plan& plan, int n) {
    if (n == plan.count_s) {  // the routed run begins
      slot = plan.first_slot;
      idx = plan.first_idx;
    }
  }
  __device__ __forceinline__ void next(const Slot* slots) {
    if (++idx >= slots[slot].inter / 16) {
      idx = 0;
      ++slot;
    }
  }
};

// ---- consumers -----------------------------------------------------------------------------------
// Phase change: every consumer warp polls its 128-blocks of the grid's h in the workspace until all of a block's
// values have been written (see kHEmpty), and turns the block into digits at once: blocks whose CTAs finished early
// are done before the last CTA's values arrive.  A block's flag in `hready` tells the other warps that its digits
// stand; nobody waits for the whole of h (see wait_h_blocks).  Returns false if the (bounded) wait ran out.
template <int G>
__device__ bool fetch_h(const DecodeParams& p, uint8_t* smem, int warp, int lane, int htotal, const float* hbuf,
                        bool never_ready, volatile int* dead, unsigned* status, uint32_t bars) {
  const int nblk = htotal >> 7;
  constexpr int kMaxIt = (kHCap / 128 + kConsumerWarps - 1) / kConsumerWarps;
  unsigned pending = 0u;  // warp-uniform
#pragma unroll
  for (int it = 0; it < kMaxIt; ++it)
    if (it * kConsumerWarps + warp < nblk) pending |= 1u << it;
  const long long t0 = clock64();
  while (pending != 0u) {
    float4 v[kMaxIt];
#pragma unroll
    for (int it = 0; it < kMaxIt; ++it)  // all of the warp's open blocks in flight together; L2 is the point of coherence
      if ((pending >> it) & 1u) v[it] = __ldcg(reinterpret_cast<const float4*>(hbuf) + (it * kConsumerWarps + warp) * 32 + lane);
#pragma unroll
    for (int it = 0; it < kMaxIt; ++it) {
      if ((pending >> it) & 1u) {
        const bool mine = __float_as_uint(v[it].x) != kHEmpty && __float_as_uint(v[it].y) != kHEmpty &&
                          __float_as_uint(v[it].z) != kHEmpty && __float_as_uint(v[it].w) != kHEmpty;
        if (__all_sync(0xffffffffu, mine) && !never_ready) {
          const float q[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
          block_to_digits<G>(q, (it * kConsumerWarps + warp) * 128, lane, smem + SmemLayout::hdig,
                             reinterpret_cast<float*>(smem + SmemLayout::hsumw), reinterpret_cast<float*>(smem + SmemLayout::hinv));
          pending &= ~(1u << it);
          __syncwarp();  // every lane's digits of the block are written ...
          if (lane == 0) {
            __threadfence_block();  // ... and visible before the flag is
            *reinterpret_cast<volatile uint8_t*>(smem + SmemLayout::hready + it * kConsumerWarps + warp) = 1;
          }
        }
      }
    }
    if (pending != 0u) {
      if (*dead) return false;
      if ((unsigned long long)(clock64() - t0) > wait_limit(dead)) {
        *dead = 1;
        atomicOr(status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Waits (bounded) until the `n` (<= 32) 128-blocks of h from block `b0` on are in shared memory as digits.
__device__ __forceinline__ bool wait_h_blocks(const uint8_t* smem, int b0, int n, int lane, volatile int* dead,
                                              unsigned* status) {
  const volatile uint8_t* flag = reinterpret_cast<const volatile uint8_t*>(smem + SmemLayout::hready) + b0 + min(lane, n - 1);
  if (!__all_sync(0xffffffffu, *flag != 0)) {
    const long long t0 = clock64();
    while (!__all_sync(0xffffffffu, *flag != 0)) {
      if (*dead) return false;
      if ((unsigned long long)(clock64() - t0) > wait_limit(dead)) {
        *dead = 1;
        atomicOr(status, (unsigned)SLICEMOE_STATUS_WAIT_TIMEOUT);
        return false;
      }
    }
  }
  __threadfence_block();
  return true;
}

// Per-lane constants of the fold (see consume_chunk).
struct LaneRole {
  int c, r, cq, boff;
  float w0, w1;
};

// One chunk: this warp's 128-column blocks of the 16-row tile(s) in unit0 (and unit1).  The A operand is
// the nibble plane, the B operand the activation digits starting at `dig`; `sumw` / `binv` are the
// digits' weighted group sums and block scales for the same columns.
//   kModeSingle: MSB tile only           -> *out0 += 2^shift s (Cm - (zp >> shift) X)
//   kModeBoth:   MSB tile, LSB tile      -> *out0 += s (2^shift Cm + Cl - zp X)
// with shift = b_high - b_low (4 for 8-bit codes with 4-bit slices; a narrower slice sits in the low bits of its
// nibble, so the planes and everything below are the same for all widths)
//   kModePair:   two matrices' MSB tiles -> *out0 += first, *out1 += second (each with its own scales)
// Unpacking: a plane byte holds row g's nibble (low) and row g + 8's (high).  The fragment registers of
// row g are the bytes masked to their low nibble; those of row g + 8 are the bytes as they are, worth
// 16 * high + low, so that accumulator rows g + 8 come out as 16 * C[g + 8] + C[g] and one subtraction per
// folded value recovers 16 * C[g + 8] (the 16 goes into the lane's fold weight).  One AND per register pair.
// Lane roles: lanes with c in {0, 1} fold row g, lanes with c in {2, 3} row g + 8; even c holds digits 0
// and 1, odd c digit 2 (and the unused fourth column).  The caller adds the two digit halves (a shuffle
// with lane ^ 1) once per task.
template <int G>
__device__ __forceinline__ void pass_mma(int (&acc)[128 / G][4], const uint8_t* ap, const uint2& bv0, const uint2& bv1,
                                         const uint2& bv2, const uint2& bv3) {
  const uint4 wlo = *reinterpret_cast<const uint4*>(ap);
  const uint4 whi = *reinterpret_cast<const uint4*>(ap + 512);
  constexpr uint32_t kLow = 0x0f0f0f0fu;
  mma_u8s8_first(acc[0], wlo.x & kLow, wlo.x, wlo.y & kLow, wlo.y, bv0.x, bv0.y);
  if (G == 32) {
    mma_u8s8_first(acc[32 / G], wlo.z & kLow, wlo.z, wlo.w & kLow, wlo.w, bv1.x, bv1.y);
    mma_u8s8_first(acc[64 / G], whi.x & kLow, whi.x, whi.y & kLow, whi.y, bv2.x, bv2.y);
    mma_u8s8_first(acc[96 / G], whi.z & kLow, whi.z, whi.w & kLow, whi.w, bv3.x, bv3.y);
  } else if (G == 64) {
    mma_u8s8_first(acc[64 / G], whi.x & kLow, whi.x, whi.y & kLow, whi.y, bv2.x, bv2.y);
    mma_u8s8(acc[0], wlo.z & kLow, wlo.z, wlo.w & kLow, wlo.w, bv1.x, bv1.y);
    mma_u8s8(acc[64 / G], whi.z & kLow, whi.z, whi.w & kLow, whi.w, bv3.x, bv3.y);
  } else {
    mma_u8s8(acc[0], wlo.z & kLow, wlo.z, wlo.w & kLow, wlo.w, bv1.x, bv1.y);
    mma_u8s8(acc[0], whi.x & kLow, whi.x, whi.y & kLow, whi.y, bv2.x, bv2.y);
    mma_u8s8(acc[0], whi.z & kLow, whi.z, whi.w & kLow, whi.w, bv3.x, bv3.y);
  }
}

template <int G>
__device__ __forceinline__ void consume_chunk(const LaneRole& lr, int lane, int gw, int rot, int mode, int nblocks,
                                              const uint8_t* unit0, const uint8_t* unit1, int scale_off, int zp_off,
                                              const uint8_t* dig, const float* sumw, const float* binv, float* out0,
                                              float* out1, int shift) {
  constexpr int SG = 128 / G;
  const bool p8 = mode == kModeBoth, pair = mode == kModePair;
  const float pfix = p8 ? 1.f : (float)(1 << shift);
  const int zsh = p8 ? 0 : shift;
  const bool hi = (lr.c >> 1) != 0;
  float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
  for (int j = 0; j < kBlocksPerWarp; ++j) {
    const int b = (gw + kGroupWarps - rot) % kGroupWarps + kGroupWarps * j;  // 128-column block of the chunk
    if (b < nblocks) {
      const uint8_t* bp = dig + lr.boff + b * 384;
      const uint2 bv0 = *reinterpret_cast<const uint2*>(bp);
      const uint2 bv1 = *reinterpret_cast<const uint2*>(bp + 96);
      const uint2 bv2 = *reinterpret_cast<const uint2*>(bp + 192);
      const uint2 bv3 = *reinterpret_cast<const uint2*>(bp + 288);
      int m[SG][4], l[SG][4];
      pass_mma<G>(m, unit0 + b * 1024 + lane * 16, bv0, bv1, bv2, bv3);
      if (mode != kModeSingle) pass_mma<G>(l, unit1 + b * 1024 + lane * 16, bv0, bv1, bv2, bv3);
      const float sfix = pfix * binv[b];
      const uint16_t* ms = reinterpret_cast<const uint16_t*>(unit0 + scale_off) + (b * SG) * 16 + lr.r;
      const uint8_t* mz = unit0 + zp_off + (b * SG) * 16 + lr.r;
#pragma unroll
      for (int sg = 0; sg < SG; ++sg) {
        // this lane's row (g, or 16 x row g + 8) and digit columns
        int ca = hi ? m[sg][2] - m[sg][0] : m[sg][0];
        int cb = hi ? m[sg][3] - m[sg][1] : m[sg][1];
        int ca1 = 0, cb1 = 0;
        if (mode != kModeSingle) {
          ca1 = hi ? l[sg][2] - l[sg][0] : l[sg][0];
          cb1 = hi ? l[sg][3] - l[sg][1] : l[sg][1];
        }
        if (p8) {  // both slices: 2^shift Cm + Cl
          ca = (ca << shift) + ca1;
          cb = (cb << shift) + cb1;
        }
        const float x0 = sumw[(b * SG + sg) * 2 + lr.cq];
        {
          const float t = fmaf((float)cb, lr.w1, (float)ca * lr.w0);
          const float sc = __half2float(__ushort_as_half(ms[sg * 16])) * sfix;
          const float z = (float)((int)mz[sg * 16] >> zsh);
          // both slices: s (2^shift Cm + Cl - zp X); MSB only: 2^shift s (Cm - (zp >> shift) X)
          acc0 = fmaf(sc, fmaf(-z, x0, t), acc0);
        }
        if (pair) {  // the second matrix' scales / zero-points travel in the second unit
          const uint16_t* ms1 = reinterpret_cast<const uint16_t*>(unit1 + scale_off) + (b * SG) * 16 + lr.r;
          const uint8_t* mz1 = unit1 + zp_off + (b * SG) * 16 + lr.r;
          const float t = fmaf((float)cb1, lr.w1, (float)ca1 * lr.w0);
          const float sc = __half2float(__ushort_as_half(ms1[sg * 16])) * sfix;
          const float z = (float)((int)mz1[sg * 16] >> shift);  // pair chunks are MSB-only
          acc1 = fmaf(sc, fmaf(-z, x0, t), acc1);
        }
      }
    }
  }
  *out0 += acc0;
  *out1 += acc1;
}

template <int G>
__device__ void consumer_loop(const DecodeParams& p, uint8_t* smem, int warp, int lane) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  float2* partial = reinterpret_cast<float2*>(smem + SmemLayout::partial);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  const uint32_t full0 = bars + 8 * Bars::full, empty0 = bars + 8 * Bars::empty;
  unsigned* status = &p.ws->status;
  const int group = warp / kGroupWarps, gw = warp % kGroupWarps;
  LaneRole lr;
  lr.c = lane & 3;
  const int g8 = lane >> 2;
  lr.r = g8 + 8 * (lr.c >> 1);
  lr.cq = lr.c & 1;
  const float rowfix = (lr.c >> 1) ? 0.0625f : 1.f;
  lr.w0 = (lr.cq ? 65536.f : 1.f) * rowfix;
  lr.w1 = (lr.cq ? 0.f : 256.f) * rowfix;
  // B column n = g8 takes digit n % 4; the fourth is unused, so those lanes re-read digit 0 and are ignored
  lr.boff = ((g8 & 3) == 3 ? 0 : (g8 & 3)) * 32 + lr.c * 8;

  // ---- phase 1: the tasks of this group ----
  const int nch = nchunks_of(p.hidden);
  const int prod = group % kProducers;  // the producer that serves this group
  {
    TaskWalk tw;
    tw.start(plan);
    int cn = 0;
    int jp = 0;  // chunks of this group's producer so far (they fix the unit pair)
    int ig = 0;  // chunks of this group so far (they fix the full barrier)
    for (int n = 0; n < plan.count1; ++n) {
      tw.at(plan, n);
      const Slot& sl = slots[tw.slot];
      const int nchunks = sl.prec ? 2 * nch : nch;
      if (n % kGroups == group) {
        float part0 = 0.f, part1 = 0.f, unused = 0.f;
        for (int q = 0; q < nchunks; ++q, ++jp, ++ig) {
          const int c = cn + q;
          const int kc = q % nch;  // which 2048-column chunk of hidden
          if (!mbar_wait(full0 + 8 * (2 * group + (ig & 1)), (ig >> 1) & 1, dead, status)) return;
          const int u0 = 4 * prod + 2 * (jp & 1);
          const int nblocks = min(kChunkK, p.hidden - kc * kChunkK) >> 7;
          const uint8_t* dig = smem + SmemLayout::xdig + kc * (kChunkK * 3);
          const float* sumw = reinterpret_cast<const float*>(smem + SmemLayout::xsumw) + kc * (kChunkK >> LG) * 2;
          const float* binv = reinterpret_cast<const float*>(smem + SmemLayout::xinv) + kc * (kChunkK >> 7);
          const uint8_t* unit0 = smem + SmemLayout::ring + u0 * kUnitBytes;
          if (sl.prec) {
            consume_chunk<G>(lr, lane, gw, c % kGroupWarps, kModeBoth, nblocks, unit0, unit0 + kUnitBytes, kPlaneUnitBytes,
                             kPlaneUnitBytes + kScaleUnitBytes, dig, sumw, binv, q < nch ? &part0 : &part1, &unused, p.shift);
          } else {
            consume_chunk<G>(lr, lane, gw, c % kGroupWarps, kModePair, nblocks, unit0, unit0 + kUnitBytes, kPlaneUnitBytes,
                             kPlaneUnitBytes + kScaleUnitBytes, dig, sumw, binv, &part0, &part1, p.shift);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty0 + 8 * (2 * prod + (jp & 1)));
        }
        // hand the four warps' shares of the K split to the epilogue warp
        part0 += __shfl_xor_sync(0xffffffffu, part0, 1);  // digits 0,1 (even c) + digit 2 (odd c)
        part1 += __shfl_xor_sync(0xffffffffu, part1, 1);
        const int round = n / kGroups;
        if (!mbar_wait(bars + 8 * (Bars::pempty1 + group), (round & 1) ^ 1, dead, status)) return;
        if (lr.cq == 0) partial[warp * 16 + lr.r] = make_float2(part0, part1);
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 8 * (Bars::pfull1 + group));
      } else if (n % kProducers == prod) {
        jp += nchunks;  // the other group this producer serves
      }
      cn += nchunks;
      tw.next(slots);
    }
  }
  __syncwarp();
  if (gw == 0) SM_TRACE(5 + group);
  if (lane == 0) mbar_arrive(bars + 8 * Bars::p1_done);  // this warp no longer reads phase-1 units
  if (plan.count2 == 0) return;

  // ---- ahead of the phase change: list this group's phase-2 chunks (the walk over all output row
  // blocks, slots and chunks costs more than consuming the group's own chunks, so it is done ahead of time) ----
  uint4* mylist = reinterpret_cast<uint4*>(smem + SmemLayout::p2list) + warp * kMaxMine;
  int nmine = 0;
  {
    const int chunks2 = plan.p2c[plan.nslots];
    const int half = plan.nunits2 / kProducers;  // units of one producer
    int xp = 0;                                   // units this group's producer has handed out so far
    for (int m = 0; m < plan.count2; ++m) {
      for (int j = 0; j < plan.nslots; ++j) {
        const int nchj = plan.p2c[j + 1] - plan.p2c[j];
        const Slot& sl = slots[j];
        const int wu = sl.prec ? 2 : 1;
        for (int kc = 0; kc < nchj; ++kc) {
          const int c = m * chunks2 + plan.p2c[j] + kc;  // chunk number within the phase
          if (c % kProducers != prod) continue;
          const int x0 = xp;
          xp += wu;
          if (c % kGroups != group) continue;
          const int ig = c / kGroups;  // this group's ordinal of the chunk
          if (lane == 0 && nmine < kMaxMine) {
            // slot, row block, rotation of the warps | the chunk's units, full barrier, parity | 128-column blocks,
            // both slices? | first column of the chunk in h
            const int k0 = kc * kChunkK;
            mylist[nmine] = make_uint4((unsigned)j | (unsigned)m << 16 | (unsigned)(ig % kGroupWarps) << 24,
                                       (unsigned)(prod * half + x0 % half) | (unsigned)(prod * half + (x0 + 1) % half) << 8 |
                                           (unsigned)(ig % kFull2PerGroup) << 16 | (unsigned)((ig / kFull2PerGroup) & 1) << 24,
                                       (unsigned)(min(kChunkK, sl.inter - k0) >> 7) | (sl.prec ? 256u : 0u),
                                       (unsigned)(sl.hoff + k0));
          }
          ++nmine;
        }
      }
    }
    nmine = min(nmine, kMaxMine);  // the host refuses launch shapes that could exceed the list
  }
  __syncwarp();
  if (warp == 0) SM_TRACE(9);

  // ---- the grid's h ----
  if (!fetch_h<G>(p, smem, warp, lane, plan.htotal, p.ws_h + (size_t)plan.hpar * kHCap, plan.never_ready != 0, dead, status,
                  bars))
    return;
  if (warp == 0) SM_TRACE(10);
  if (gw == 0) SM_TRACE(14 + group);

  // ---- phase 2: chunks round-robin over the groups, all warps contribute to every task ----
  const uint32_t full2 = bars + 8 * Bars::full2, empty2 = bars + 8 * Bars::empty2;
  int i = 0;
  for (int m = 0; m < plan.count2; ++m) {
    float part = 0.f, unused = 0.f, sacc = 0.f;
    int jcur = -1;
    for (; i < nmine; ++i) {
      const uint4 d = mylist[i];
      if ((int)((d.x >> 16) & 0xffu) != m) break;
      const int j = d.x & 0xffffu, rot = d.x >> 24;
      if (j != jcur) {  // weighted combine, in slot order
        if (jcur >= 0) part = fmaf(slots[jcur].gated ? plan.gate : slots[jcur].coef, sacc, part);
        jcur = j;
        sacc = 0.f;
      }
      const int u0 = d.y & 0xffu, u1 = (d.y >> 8) & 0xffu;
      const int nblocks = d.z & 0xffu, col = (int)d.w;
      const bool p8 = (d.z & 256u) != 0u;
      if (!mbar_wait(full2 + 8 * (kFull2PerGroup * group + ((d.y >> 16) & 0xffu)), d.y >> 24, dead, status)) return;
      if (!wait_h_blocks(smem, col >> 7, nblocks, lane, dead, status)) return;  // this chunk's part of h, no more
      if (gw == 0 && i == nmine - 1) SM_TRACE(23 + group);
      const uint8_t* dig = smem + SmemLayout::hdig + col * 3;
      const float* sumw = reinterpret_cast<const float*>(smem + SmemLayout::hsumw) + (col >> LG) * 2;
      const float* binv = reinterpret_cast<const float*>(smem + SmemLayout::hinv) + (col >> 7);
      consume_chunk<G>(lr, lane, gw, rot, p8 ? kModeBoth : kModeSingle, nblocks,
                       smem + SmemLayout::ring + u0 * plan.unit2_bytes, smem + SmemLayout::ring + u1 * plan.unit2_bytes,
                       plan.scale2_off, plan.zp2_off, dig, sumw, binv, &sacc, &unused, p.shift);
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(empty2 + 8 * u0);
        if (p8) mbar_arrive(empty2 + 8 * u1);
      }
    }
    if (jcur >= 0) part = fmaf(slots[jcur].gated ? plan.gate : slots[jcur].coef, sacc, part);
    part += __shfl_xor_sync(0xffffffffu, part, 1);
    if (!mbar_wait(bars + 8 * Bars::pempty2, (m & 1) ^ 1, dead, status)) return;
    if (lr.cq == 0) partial[warp * 16 + lr.r] = make_float2(0.f, part);
    __syncwarp();
    if (lane == 0) mbar_arrive(bars + 8 * Bars::pfull2);
  }
  if (warp == 0) SM_TRACE(11);
  if (gw == 0) SM_TRACE(27 + group);
}

// ---- epilogue warp ---------------------------------------------------------------------------------
__device__ void epilogue_loop(const DecodeParams& p, uint8_t* smem, int lane) {
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  const float2* partial = reinterpret_cast<const float2*>(smem + SmemLayout::partial);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  unsigned* status = &p.ws->status;
  // This CTA's share of the OTHER h buffer goes back to "empty" for the next launch: its last readers were the
  // launch before this one.
  {
    uint4* other = reinterpret_cast<uint4*>(p.ws_h + (size_t)(plan.hpar ^ 1) * kHCap);
    constexpr int n16 = kHCap / 4;
    const int per = (n16 + (int)gridDim.x - 1) / (int)gridDim.x;
    const int lo = (int)blockIdx.x * per, hi = min(n16, lo + per);
    for (int i = lo + lane; i < hi; i += 32) other[i] = make_uint4(kHEmpty, kHEmpty, kHEmpty, kHEmpty);
  }
  float* hbuf = p.ws_h + (size_t)plan.hpar * kHCap;
  // phase 1: one group's four partial rows per task -> SwiGLU -> h
  {
    TaskWalk tw;
    tw.start(plan);
    for (int n = 0; n < plan.count1; ++n) {
      tw.at(plan, n);
      const int slot = tw.slot, idx = tw.idx;
      const int group = n % kGroups, round = n / kGroups;
      if (!mbar_wait(bars + 8 * (Bars::pfull1 + group), round & 1, dead, status)) return;
      float a = 0.f, b = 0.f;
      if (lane < 16) {
#pragma unroll
        for (int w = 0; w < kGroupWarps; ++w) {
          const float2 v = partial[(group * kGroupWarps + w) * 16 + lane];
          a += v.x;
          b += v.y;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + 8 * (Bars::pempty1 + group));
      if (lane < 16) hbuf[slots[slot].hoff + idx * 16 + lane] = a / (1.f + expf(-a)) * b;  // silu(gate) * up
      tw.next(slots);
    }
  }
  SM_TRACE(12);
  // phase 2: all warps' partial rows per output row block -> y
  for (int m = 0; m < plan.count2; ++m) {
    if (!mbar_wait(bars + 8 * Bars::pfull2, m & 1, dead, status)) return;
    float b = 0.f;
    if (lane < 16) {
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) b += partial[w * 16 + lane].y;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bars + 8 * Bars::pempty2);
    if (lane < 16) p.y[(blockIdx.x + m * gridDim.x) * 16 + lane] = b;
  }
  SM_TRACE(13);
  SM_TRACE_G(22);
}

// ---- producer --------------------------------------------------------------------------------------
// What a producer lane copies, for a chunk of matrix A (and, in a pair chunk, matrix B):
//   lane 0  A's MSB tile            -> first unit, plane area
//   lane 1  A's LSB tile (8-bit) or B's MSB tile (pair) -> second unit, plane area
//   lane 2  A's scales, lane 3 A's zero-points          -> first unit, after the plane area
//   lane 4  B's scales, lane 5 B's zero-points (pair)   -> second unit, after the plane area
// For all of them the source of (row block rb, column block kb of 128) is
// base + (rb * (K / 128) + kb) * bytes_per_block, because planes and scale / zero-point arrays are all
// stored [row block][column][16 rows].
constexpr int kProducerLanes = 6;
struct ProducerLane {
  uint32_t bytes_per_block;  // bytes per (16 rows x 128 columns)
  int field;                 // which of the matrix' four pointers
  bool second_unit;
};
// The ring as a phase sees it.
struct RingView {
  uint32_t unit_bytes, scale_off, zp_off;
};
// Where one chunk goes: its two units, the barrier that says its space is free (with the parity to wait for)
// and the barrier its bytes complete.
struct ChunkSpace {
  int u0, u1;
  uint32_t empty_bar, empty_parity, full_bar;
  uint32_t empty_bar_first, empty_parity_first;  // phase 2, two-unit chunks: the first unit has a barrier of its own
};

// What a producer needs to wait: it starts before the kernels ahead of this one in the stream have completed, so
// a wait that does not pass at once is first the moment to wait for those (the consumers, on whom all of a
// producer's barriers depend, do not start earlier; and a bounded wait's clock must not run while an earlier
// kernel is still busy).
struct ProducerWait {
  volatile int* dead;
  unsigned* status;
  bool dep_waited;  // griddepcontrol.wait has been executed
  __device__ __forceinline__ bool operator()(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    if (!dep_waited) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      dep_waited = true;
    }
    return mbar_wait(bar, parity, dead, status);
  }
};

// One chunk of matrix A - or of matrices A and B side by side - of (slot, row block rb), columns from k0, into
// the space `cs`.  Run by the first kProducerLanes lanes of a producer warp together.  Returns false if a
// wait ran out.
template <int G>
__device__ __forceinline__ bool produce_chunk(uint8_t* smem, const RingView& rv, const ChunkSpace& cs, int lane,
                                              const ProducerLane& pl, const Slot& s, int matA, int matB, int mode, int K,
                                              int rb, int k0, ProducerWait& pw, uint64_t pol) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  const bool two = mode != kModeSingle;
  bool active;
  const uint8_t* src;
  if (lane == 1) {
    active = two;
    src = mode == kModePair ? s.ptr[matB][0] : s.ptr[matA][1];
    if (mode == kModeBoth && src == nullptr) {  // 8 bits asked of an expert without LSB planes: defined garbage, reported
      src = s.ptr[matA][0];
      atomicOr(pw.status, (unsigned)SLICEMOE_STATUS_MISSING_LSB);
    }
  } else if (lane >= 4) {
    active = mode == kModePair;
    src = s.ptr[active ? matB : matA][pl.field];
  } else {
    active = true;
    src = s.ptr[matA][pl.field];
  }
  src += (size_t)((unsigned)rb * (unsigned)(K >> 7) + (unsigned)(k0 >> 7)) * pl.bytes_per_block;
  const uint32_t nblk = (uint32_t)(min(kChunkK, K - k0) >> 7);
  // The two units of a phase-2 chunk may last have held chunks of different consumer groups: both must be free.
  if (cs.empty_bar_first != 0u && !pw(cs.empty_bar_first, cs.empty_parity_first)) return false;
  if (!pw(cs.empty_bar, cs.empty_parity)) return false;
  const uint32_t bar = cs.full_bar;
  if (lane == 0)
    mbar_arrive_expect_tx(bar, nblk * ((two ? 2048u : 1024u) + (mode == kModePair ? 2u : 1u) * ((128u >> LG) * 48u)));
  __syncwarp((1u << kProducerLanes) - 1u);
  if (active) {
    const uint32_t u = (uint32_t)(pl.second_unit ? cs.u1 : cs.u0);
    const uint32_t dst_in_unit = pl.field < 2 ? 0u : (pl.field == 2 ? rv.scale_off : rv.zp_off);
    bulk_g2s(smem_u32(smem + SmemLayout::ring) + u * rv.unit_bytes + dst_in_unit, src, nblk * pl.bytes_per_block, bar, pol);
  }
  return true;
}

// Producer warp `which` of kProducers: every producer walks the whole schedule and issues its share.
template <int G>
__device__ void producer_loop(const DecodeParams& p, uint8_t* smem, int lane, int which) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  const Slot* slots = reinterpret_cast<const Slot*>(smem + SmemLayout::slots);
  const Plan& plan = *reinterpret_cast<const Plan*>(smem + SmemLayout::plan);
  volatile int* dead = reinterpret_cast<volatile int*>(smem + SmemLayout::dead);
  const uint32_t bars = smem_u32(smem + SmemLayout::bars);
  ProducerWait pw;
  pw.dead = dead;
  pw.status = &p.ws->status;
  pw.dep_waited = false;
  const uint64_t pol = l2_evict_first_policy();
  ProducerLane pl;
  pl.field = lane < 2 ? lane : 2 + (lane & 1);  // lanes 2, 4: scales; lanes 3, 5: zero-points
  pl.bytes_per_block = lane < 2 ? 1024u : (pl.field == 2 ? (128u >> LG) * 32u : (128u >> LG) * 16u);
  pl.second_unit = lane == 1 || lane >= 4;
  bool ok = true;
  // phase 1: gate and up of (slot, row block) tasks; two units per chunk
  RingView r1;
  r1.unit_bytes = kUnitBytes;
  r1.scale_off = kPlaneUnitBytes;
  r1.zp_off = kPlaneUnitBytes + kScaleUnitBytes;
  const int nch = nchunks_of(p.hidden);
  static_assert(kGroups == 2 * kProducers, "a producer serves the groups `which` and `which + kProducers`");
  int ig_lo = 0, ig_hi = 0;  // chunks armed so far for group `which` and for group `which + kProducers`
  {
    TaskWalk tw;
    tw.start(plan);
    int jp = 0;  // this warp's chunks so far
    // The shared experts' tasks are known from the start; what follows them - and how many tasks there are - once
    // the plan stands.
    int n_end = plan.count_s;
    for (int n = 0; ok; ++n) {
      if (n == plan.count_s) {
        ok = pw(bars + 8 * Bars::plan_ready, 0);
        if (!ok) break;
        n_end = plan.count1;
      }
      if (n >= n_end) break;
      tw.at(plan, n);
      const int slot = tw.slot, idx = tw.idx;
      const Slot& s = slots[slot];
      const int nchunks = s.prec ? 2 * nch : nch;
      if (n % kProducers == which) {
        const int g = n % kGroups;
        for (int q = 0; q < nchunks && ok; ++q, ++jp) {
          const int mat = s.prec ? q / nch : 0;
          ChunkSpace cs;
          cs.u0 = 4 * which + 2 * (jp & 1);
          cs.u1 = cs.u0 + 1;
          cs.empty_bar = bars + 8 * (Bars::empty + 2 * which + (jp & 1));
          cs.empty_parity = ((jp >> 1) & 1) ^ 1;
          cs.empty_bar_first = 0u;  // a phase-1 unit pair always holds one chunk: one barrier
          cs.empty_parity_first = 0u;
          int& igg = g == which ? ig_lo : ig_hi;
          cs.full_bar = bars + 8 * (Bars::full + 2 * g + (igg & 1));
          ++igg;
          ok = produce_chunk<G>(smem, r1, cs, lane, pl, s, mat, s.prec ? mat : 1, s.prec ? kModeBoth : kModePair, p.hidden,
                                idx, (q % nch) * kChunkK, pw, pol);
          if (which == 0 && lane == 0 && jp < 8) SM_TRACE(32 + jp);
        }
      }
      tw.next(slots);
    }
  }
  // phase 2: down rows of every slot for the output row blocks of this CTA, in the re-cut ring
  RingView r2;
  r2.unit_bytes = (uint32_t)plan.unit2_bytes;
  r2.scale_off = (uint32_t)plan.scale2_off;
  r2.zp_off = (uint32_t)plan.zp2_off;
  // The re-cut units lie over the phase-1 units: nothing of phase 2 lands before phase 1 has been consumed.
  // (From then until h has crossed the grid the memory system has nothing else to do.)
  if (ok && plan.count2 > 0) ok = pw(bars + 8 * Bars::p1_done, 0);
  if (which == 0 && lane == 0 && plan.count2 > 0) SM_TRACE(31);
  const int half = plan.nunits2 / kProducers;  // this warp's units are [which * half, which * half + half)
  int c2 = 0, xp = 0;                           // chunks of the phase so far, units this warp has handed out
  for (int m = 0; m < plan.count2 && ok; ++m) {
    const int rb = blockIdx.x + m * gridDim.x;
    for (int slot = 0; slot < plan.nslots && ok; ++slot) {
      const Slot& s = slots[slot];
      const int w = s.prec ? 2 : 1;
      for (int k0 = 0; k0 < s.inter && ok; k0 += kChunkK, ++c2) {
        if (c2 % kProducers != which) continue;
        const int g = c2 % kGroups, ig = c2 / kGroups;
        const int xl = xp + w - 1;  // the chunk's last unit
        ChunkSpace cs;
        cs.u0 = which * half + xp % half;
        cs.u1 = which * half + (xp + 1) % half;
        cs.empty_bar = bars + 8 * (Bars::empty2 + which * half + xl % half);
        cs.empty_parity = ((xl / half) & 1) ^ 1;
        cs.empty_bar_first = w == 2 ? bars + 8 * (Bars::empty2 + which * half + xp % half) : 0u;
        cs.empty_parity_first = ((xp / half) & 1) ^ 1;
        cs.full_bar = bars + 8 * (Bars::full2 + kFull2PerGroup * g + ig % kFull2PerGroup);
        xp += w;
        ok = produce_chunk<G>(smem, r2, cs, lane, pl, s, 2, 2, s.prec ? kModeBoth : kModeSingle, s.inter, rb, k0, pw, pol);
      }
    }
  }
  if (lane == 0 && plan.count2 > 0) SM_TRACE(18 + which);
#ifdef SLICEMOE_TRACE
  int landed = 0;
#endif
  // Never leave the CTA with bulk copies still landing in its shared memory: wait (bounded) until every
  // barrier this warp may have armed has completed its last phase.  In the normal path they have long ago.
  for (int g = which; g < kGroups; g += kProducers) {
    const int n1 = g == which ? ig_lo : ig_hi;
    for (int i = max(0, n1 - 2); i < n1; ++i) {
      const long long t0 = clock64();
      while (!mbar_try(bars + 8 * (Bars::full + 2 * g + (i & 1)), (i >> 1) & 1)) {
        if (*dead || (unsigned long long)(clock64() - t0) > wait_limit(dead)) break;
      }
    }
    const int n2 = c2 > g ? (c2 - 1 - g) / kGroups + 1 : 0;  // chunks of the phase that went to group g
    for (int i = max(0, n2 - kFull2PerGroup); i < n2; ++i) {
      const long long t0 = clock64();
      while (!mbar_try(bars + 8 * (Bars::full2 + kFull2PerGroup * g + i % kFull2PerGroup), (i / kFull2PerGroup) & 1)) {
        if (*dead || (unsigned long long)(clock64() - t0) > wait_limit(dead)) break;
      }
#ifdef SLICEMOE_TRACE
      if (lane == 0 && landed < 4) SM_TRACE(40 + 4 * which + landed);
      ++landed;
#endif
    }
  }
}

// ---- prologue pieces ---------------------------------------------------------------------------------
// Slot order: shared experts, then the routed experts that run at 8 bits, then those that run at 4 bits,
// each group in list order.  With the larger tasks first, windows of a multiple of the larger task size cut
// the phase-1 unit sequence at task boundaries, so every CTA gets the same number of units.
//
// The routing list as one warp sees it: lane j < k holds entry j; out-of-range ids are dropped.
struct Routed {
  int e, pr;
  float w;
  bool valid;
  int pos;  // slot index of this lane's entry
  int nbig, nsmall;
};
template <bool FUSED>
__device__ __forceinline__ Routed read_routing(const DecodeParams& p, int lane, bool publish) {
  Routed rt;
  rt.e = -1;
  rt.pr = 0;
  rt.w = 0.f;
  if (FUSED) {
    // same arithmetic as the stand-alone routing kernel; the precision request is the precision
    const RouteSel sel = route_warp(p.logits, p.n_experts, p.k, p.bias, p.renorm, p.tau, p.rank_high, lane);
    if (lane < p.k) {
      rt.e = sel.id;
      rt.pr = sel.prec_req;
      rt.w = sel.w;
      if (publish && blockIdx.x == 0) {
        if (p.ids_out) p.ids_out[lane] = sel.id;
        if (p.prec_out) p.prec_out[lane] = sel.prec_req;
        if (p.weights_out) p.weights_out[lane] = sel.w;
      }
    }
  } else if (lane < p.k) {
    rt.e = p.ids[lane];
    rt.pr = p.prec[lane];
    rt.w = p.weights[lane];
  }
  rt.valid = lane < p.k && rt.e >= 0 && rt.e < p.n_experts;
  const unsigned vmask = __ballot_sync(0xffffffffu, rt.valid);
  const unsigned bigmask = __ballot_sync(0xffffffffu, rt.valid && rt.pr != 0);
  const unsigned below = (1u << lane) - 1u;
  rt.nbig = __popc(bigmask);
  rt.nsmall = __popc(vmask) - rt.nbig;
  rt.pos = p.n_shared + (rt.pr != 0 ? __popc(bigmask & below) : rt.nbig + __popc(vmask & ~bigmask & below));
  return rt;
}

// What of the plan depends on the shape and the grid alone; one lane computes it while the kernel still waits
// for the grids before it.  Assumes at least one valid routed entry when k > 0 (build_plan redoes the unit
// size in the rare case that there is none).
__device__ __forceinline__ int phase2_unit_blocks(const DecodeParams& p, bool any_routed) {
  int maxblk = 1;
  if (p.n_shared) maxblk = max(maxblk, min(kChunkK, p.shared_inter) >> 7);
  if (any_routed) maxblk = max(maxblk, min(kChunkK, p.inter) >> 7);
  return maxblk;
}
__device__ __forceinline__ void plan_units2(const DecodeParams& p, Plan* plan, int maxblk) {
  const int meta_blk = 16 * (128 / p.group);  // scale entries per 128 columns
  plan->scale2_off = maxblk * 1024;
  plan->zp2_off = maxblk * 1024 + maxblk * meta_blk * 2;
  plan->unit2_bytes = (maxblk * (1024 + meta_blk * 3) + 127) & ~127;
  plan->nunits2 = min(kUnits2, (kUnits * kUnitBytes) / plan->unit2_bytes);
}
// Shared-expert tasks before CTA c when the grid's T1 of them are dealt out evenly.
__device__ __forceinline__ unsigned shared_before(unsigned c, unsigned T1, unsigned P) {
  return (unsigned)((unsigned long long)c * T1 / P);
}
// Run by warp 0.
__device__ void build_plan_static(const DecodeParams& p, uint8_t* smem, int lane) {
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);
  if (lane < p.n_shared) {
    Slot& s = slots[lane];
    s.inter = p.shared_inter;
    s.prec = 1;
    s.coef = 1.f;
    s.gated = p.sigmoid_gate;
    s.hoff = lane * p.shared_inter;
  }
  if (lane != 0) return;
  const int nrb = p.hidden / 16;
  plan->count2 = (int)blockIdx.x < nrb ? (nrb - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  plan_units2(p, plan, phase2_unit_blocks(p, p.k > 0));
  // this CTA's share of the shared experts' phase-1 tasks
  const unsigned nts = p.n_shared ? (unsigned)p.shared_inter / 16u : 0u, T1 = (unsigned)p.n_shared * nts;
  const unsigned lo = shared_before(blockIdx.x, T1, gridDim.x), hi = shared_before(blockIdx.x + 1u, T1, gridDim.x);
  plan->slot_s = nts ? (int)(lo / nts) : 0;
  plan->idx_s = nts ? (int)(lo % nts) : 0;
  plan->count_s = (int)(hi - lo);
}

// Warp 0: slot table (all but the pointers) and the static partition, in closed form: the phase-1 unit
// sequence is three runs of equal tasks (shared, routed 8-bit, routed 4-bit).
template <bool FUSED>
__device__ void build_plan(const DecodeParams& p, uint8_t* smem, int lane) {
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);
  const Routed rt = read_routing<FUSED>(p, lane, true);
  if (lane < p.k && !rt.valid) atomicOr(&p.ws->status, (unsigned)SLICEMOE_STATUS_BAD_EXPERT_ID);
  if (rt.valid) {
    Slot& s = slots[rt.pos];
    s.inter = p.inter;
    s.prec = rt.pr != 0;
    s.coef = rt.w;
    s.gated = 0;
    s.hoff = p.n_shared * p.shared_inter + (rt.pos - p.n_shared) * p.inter;
  }
  const int nslots = p.n_shared + rt.nbig + rt.nsmall;
  // phase-2 chunk and unit counts before each slot: lane j handles slot j (8-bit: shared and the first nbig routed)
  {
    int cj = 0, uj = 0;
    if (lane < nslots) {
      const int inter = lane < p.n_shared ? p.shared_inter : p.inter;
      const bool p8 = lane < p.n_shared + rt.nbig;
      cj = nchunks_of(inter);
      uj = p8 ? 2 * cj : cj;
    }
    int ci = cj, ui = uj;  // inclusive scans
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int a = __shfl_up_sync(0xffffffffu, ci, off), b = __shfl_up_sync(0xffffffffu, ui, off);
      if (lane >= off) {
        ci += a;
        ui += b;
      }
    }
    if (lane < nslots) {
      plan->p2c[lane + 1] = (short)ci;
      plan->p2u[lane + 1] = (short)ui;
    }
    if (lane == 0) plan->p2c[0] = plan->p2u[0] = 0;
  }
  {
    const unsigned nsh = (unsigned)p.n_shared, nbig = (unsigned)rt.nbig, nsmall = (unsigned)rt.nsmall;
    const unsigned nts = nsh ? (unsigned)p.shared_inter / 16u : 0u, ntr = (unsigned)p.inter / 16u;
    const unsigned nch = (unsigned)nchunks_of(p.hidden);
    const unsigned spb = 4u * nch, sps = 2u * nch;  // units per 8-bit / 4-bit task (shared tasks are 8-bit)
    const unsigned T1 = nsh * nts, T2 = nbig * ntr, T3 = nsmall * ntr;  // tasks per run
    const unsigned U1 = T1 * spb, U2 = T2 * spb, S = U1 + U2 + T3 * sps;
    const unsigned spmax = (nsh + nbig) ? spb : sps;
    // Every CTA gets T units of work: its shared tasks (dealt out evenly, build_plan_static) and a window of the
    // routed unit sequence that fills the rest.  T and every shared share are multiples of the larger task size,
    // and the larger routed tasks come first, so the windows are cut at task boundaries.
    const unsigned T = ((S + gridDim.x - 1) / gridDim.x + spmax - 1) / spmax * spmax;
    const unsigned UR = U2 + T3 * sps;  // the routed sequence
    // ordinal of the first routed task that starts at or after a unit offset of the routed sequence
    auto ord_of = [&](unsigned bound) -> unsigned {
      if (bound >= UR) return T2 + T3;
      if (bound < U2) return (bound + spb - 1) / spb;
      return T2 + (bound - U2 + sps - 1) / sps;
    };
    // both ends of this CTA's window at once: lane 1 takes the upper one
    const unsigned cc = blockIdx.x + (unsigned)(lane & 1);
    const unsigned o = ord_of(cc * T - spb * shared_before(cc, T1, gridDim.x));
    const unsigned o0 = __shfl_sync(0xffffffffu, o, 0), o1 = __shfl_sync(0xffffffffu, o, 1);
    if (lane != 0) return;
    plan->first_slot = (int)(nsh + o0 / ntr);
    plan->first_idx = (int)(o0 % ntr);
    plan->count1 = plan->count_s + (int)(o1 - o0);
    if (nslots == 0) plan->count2 = 0;  // otherwise as build_plan_static left it
    plan->nslots = nslots;
    plan->htotal = (int)(nsh * (unsigned)p.shared_inter + (nbig + nsmall) * (unsigned)p.inter);
    // phase-2 units: as large as the widest down chunk of any slot (set ahead of time for the usual case)
    if (nbig + nsmall == 0 && p.k > 0) plan_units2(p, plan, phase2_unit_blocks(p, false));
  }
}

// Warp 1: the routed slots' plane pointers.  Warp 2: the shared slots' (they do not depend on the list).
// Each slot's twelve pointers sit in slicemoe_expert in the order the slot table keeps them.
template <bool FUSED>
__device__ void load_slot_pointers(const DecodeParams& p, uint8_t* smem, int lane, bool routed) {
  Slot* slots = reinterpret_cast<Slot*>(smem + SmemLayout::slots);
  constexpr int kRounds = (kMaxSlots * 12 + 31) / 32;
  const uint8_t* const* src[kRounds];
  int first = 0, count = p.n_shared;
  if (routed) {
    const Routed rt = read_routing<FUSED>(p, lane, false);
    first = p.n_shared;
    count = rt.nbig + rt.nsmall;
    // lane j knows its entry's slot; every lane needs every slot's expert: pass them through the slot table
    if (rt.valid) slots[rt.pos].ptr[0][0] = reinterpret_cast<const uint8_t*>(p.experts + rt.e);
    __syncwarp();
  }
#pragma unroll
  for (int rd = 0; rd < kRounds; ++rd) {
    const int i = rd * 32 + lane;
    src[rd] = nullptr;
    if (i < count * 12) {
      const int sl = first + i / 12, q = i % 12;
      const slicemoe_expert* ex = routed ? reinterpret_cast<const slicemoe_expert*>(slots[sl].ptr[0][0]) : p.shared + sl;
      src[rd] = reinterpret_cast<const uint8_t* const*>(reinterpret_cast<const slicemoe_mat*>(ex) + (q >> 2)) + (q & 3);
    }
  }
  __syncwarp();  // every lane has read the experts' addresses before the first slot pointer overwrites one
  const uint8_t* val[kRounds];
#pragma unroll
  for (int rd = 0; rd < kRounds; ++rd) val[rd] = src[rd] ? *src[rd] : nullptr;  // all loads in flight together
#pragma unroll
  for (int rd = 0; rd < kRounds; ++rd) {
    const int i = rd * 32 + lane;
    if (i < count * 12) slots[first + i / 12].ptr[(i % 12) >> 2][(i % 12) & 3] = val[rd];
  }
}

// ---- the kernel ------------------------------------------------------------------------------------
// FUSED: the routing list is computed from the router logits in the prologue (slicemoe_layer_routed); kept
// apart from the plain kernel so that the latter carries none of the routing code.
template <int G, bool FUSED>
__global__ void __launch_bounds__(kThreads, 1) decode_layer_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  Plan* plan = reinterpret_cast<Plan*>(smem + SmemLayout::plan);

  // Programmatic dependent launch: the next kernel in the stream may start launching as soon as every CTA
  // of this grid has got here (its CTAs find room only where one of ours has exited), and this kernel does
  // all it can before it waits for the grids before it.  Nothing an earlier kernel may write is touched
  // before that wait: x and the workspace always, and the routing lists unless the caller has promised that
  // they were complete earlier (lists_resident).  The weights, the expert tables and the shape are never written
  // by a kernel in flight.
#ifdef SLICEMOE_TRACE
  if (tid == 0) s_trace_t0 = clock64();
  if (tid == 0 && blockIdx.x < 256) g_trace[blockIdx.x][20] = trace_gtime();
#endif
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const bool early_lists = !FUSED && p.lists_resident != 0;
  if (warp == kProducerWarp) {
    if (lane == 0) {
      *reinterpret_cast<int*>(smem + SmemLayout::dead) = 0;
      *reinterpret_cast<unsigned long long*>(smem + SmemLayout::dead + 8) = kWaitCycles;
      for (int i = 0; i < kHCap / 128; i += 8) *reinterpret_cast<unsigned long long*>(smem + SmemLayout::hready + i) = 0ull;
      const uint32_t bars = smem_u32(smem + SmemLayout::bars);
      for (int s = 0; s < kUnits; ++s) {
        mbar_init(bars + 8 * (Bars::full + s), 1);             // lane 0's expect_tx arrive
        mbar_init(bars + 8 * (Bars::empty + s), kGroupWarps);  // one arrive per warp of the consuming group
      }
      for (int s = 0; s < kGroups * kFull2PerGroup; ++s) mbar_init(bars + 8 * (Bars::full2 + s), 1);
      for (int s = 0; s < kUnits2; ++s) mbar_init(bars + 8 * (Bars::empty2 + s), kGroupWarps);
      for (int g = 0; g < kGroups; ++g) {
        mbar_init(bars + 8 * (Bars::pfull1 + g), kGroupWarps);
        mbar_init(bars + 8 * (Bars::pempty1 + g), 1);
      }
      mbar_init(bars + 8 * Bars::pfull2, kConsumerWarps);
      mbar_init(bars + 8 * Bars::pempty2, 1);
      mbar_init(bars + 8 * Bars::p1_done, kConsumerWarps);
      mbar_init(bars + 8 * Bars::plan_ready, early_lists ? 2 : 1);  // resident lists: warps 0 and 1 each say when done
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
  }
  // Ahead of the wait: what follows from the shape alone - the shared experts' slots, pointers and this CTA's share
  // of their tasks - and the routed experts' pointer table on its way into L2 (its entries are read right after the
  // wait).
  if (warp == 0) {
    build_plan_static(p, smem, lane);
  } else if (warp == 1 && p.experts != nullptr && p.k > 0 && !early_lists) {
    const char* tab = reinterpret_cast<const char*>(p.experts);
    const size_t bytes = (size_t)p.n_experts * sizeof(slicemoe_expert);
    for (size_t off = (size_t)lane * 128; off < bytes; off += 32 * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(tab + off));
  } else if (warp == 2) {
    if (p.n_shared > 0) load_slot_pointers<FUSED>(p, smem, lane, false);
  }
  __syncthreads();
  const uint32_t plan_ready = smem_u32(smem + SmemLayout::bars) + 8 * Bars::plan_ready;
  if (warp >= kProducerWarp) {
    // The producers start on the shared experts' tiles (and, with resident lists, go on to the routed experts')
    // while the kernels ahead are still running; see ProducerWait for where they wait for those.
    if (lane < kProducerLanes) producer_loop<G>(p, smem, lane, warp - kProducerWarp);
    return;
  }

  // Everyone else waits here.  Then, in parallel and with one barrier (of these 17 warps) at the end: warp 0 reads
  // the routing list and builds the routed slots and the partition, warp 1 fetches the routed experts' plane
  // pointers, warp 2 takes the wait limit and the shared-expert gate, the other 14 warps turn x into digits, one
  // 128-element block at a time.
  // (With resident lists warps 0 and 1 do their part first, while the producers are already busy with the shared
  // experts' tiles, and tell the producers themselves.)
  if (early_lists && warp < 2) {
    if (warp == 0) build_plan<FUSED>(p, smem, lane);
    else load_slot_pointers<FUSED>(p, smem, lane, true);
    __syncwarp();
    if (lane == 0) mbar_arrive(plan_ready);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp == 3) {
    SM_TRACE(1);
    SM_TRACE_G(21);
  }
  if (warp == 0) {
    if (!early_lists) build_plan<FUSED>(p, smem, lane);
    SM_TRACE(2);
  } else if (warp == 1) {
    if (!early_lists) load_slot_pointers<FUSED>(p, smem, lane, true);
  } else if (warp == 2) {
    if (lane == 0) {
      // a wait limit set by the host for this workspace
      const unsigned long long lim = p.ws->wait_cycles;
      if (lim != 0ull) *reinterpret_cast<unsigned long long*>(smem + SmemLayout::dead + 8) = lim;
      // Which h buffer: the parity of the launch count.  The count moves on once every CTA of this launch has
      // read it (the last reader does it), so all of them see the same value, and the next launch the next.
      const unsigned epoch = p.ws->epoch;
      plan->hpar = (int)(epoch & 1u);
      plan->never_ready = p.ws->extra_arrivals != 0u ? 1 : 0;
      if (atomicAdd(&p.ws->readers, 1u) == gridDim.x - 1u) {
        p.ws->readers = 0u;
        p.ws->epoch = epoch + 1u;
        __threadfence();
      }
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
    // warps 3 .. 16
    constexpr int nw = kConsumerWarps + 1 - 3;
    for (int blk = warp - 3; blk < p.hidden / 128; blk += nw) {
      const uint2 raw = *reinterpret_cast<const uint2*>(p.x + blk * 128 + 4 * lane);
      const float v[4] = {__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                          __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u)};
      block_to_digits<G>(v, blk * 128, lane, smem + SmemLayout::xdig, reinterpret_cast<float*>(smem + SmemLayout::xsumw),
                         reinterpret_cast<float*>(smem + SmemLayout::xinv));
    }
  }
  if (warp == 3) SM_TRACE(3);
  asm volatile("bar.sync 1, %0;" ::"n"(32 * (kConsumerWarps + 1)) : "memory");
  if (warp == 3) SM_TRACE(4);
  if (!early_lists && tid == 0) mbar_arrive(plan_ready);
  if (plan->nslots == 0 && blockIdx.x == 0)
    for (int i = tid; i < p.hidden; i += 32 * (kConsumerWarps + 1)) p.y[i] = 0.f;

  if (warp < kConsumerWarps) {
    consumer_loop<G>(p, smem, warp, lane);
  } else {
    epilogue_loop(p, smem, lane);
  }
}

// ---- host side --------------------------------------------------------------------------------------
static int g_num_sms[64];
static bool g_attr_set[64][6];

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

template <int G, bool FUSED>
static int launch_decode(const DecodeParams& p, int dev, int sms, int gi, cudaStream_t st, bool cooperative = false) {
  bool& attr_set = g_attr_set[dev][2 * gi + (FUSED ? 1 : 0)];
  if (!attr_set) {
    SM_CUDA_TRY(cudaFuncSetAttribute(decode_layer_kernel<G, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     SmemLayout::total));
    // Every CTA waits for h values that the other CTAs write, so all of them must be able to be resident at
    // once: one per SM needs the kernel to fit an SM at all.  (If another kernel holds SMs at the time, the
    // bounded wait for h ends the launch with SLICEMOE_STATUS_WAIT_TIMEOUT instead of a hang.)
    int per_sm = 0;
    SM_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_layer_kernel<G, FUSED>, kThreads,
                                                              SmemLayout::total));
    if (per_sm < 1) return SLICEMOE_E_UNSUPPORTED;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sms);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = SmemLayout::total;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see the top of the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  // On request the driver is asked to guarantee that all CTAs are resident together (they wait for one another's
  // h values): the launch then fails instead of timing out when the device cannot hold the grid, at the price of
  // the CTA-by-CTA hand-over between consecutive launches.
  attr[1].id = cudaLaunchAttributeCooperative;
  attr[1].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = cooperative ? 2 : 1;
  SM_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_layer_kernel<G, FUSED>, p));
  return SLICEMOE_OK;
}

static int check_shape(const slicemoe_shape* s) {
  if (!s) return SLICEMOE_E_INVALID_ARG;
  if (!valid_widths(s->b_high, s->b_low)) return SLICEMOE_E_UNSUPPORTED;
  if (!valid_group(s->group)) return SLICEMOE_E_UNSUPPORTED;
  if (s->hidden <= 0 || s->inter <= 0 || s->n_experts <= 0 || s->top_k < 1) return SLICEMOE_E_INVALID_ARG;
  if (s->top_k > s->n_experts || s->top_k > SLICEMOE_MAX_TOP_K) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared < 0 || s->n_shared > SLICEMOE_MAX_SHARED) return SLICEMOE_E_INVALID_ARG;
  if ((s->hidden % 128) || (s->inter % 128)) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && (s->shared_inter <= 0 || (s->shared_inter % 128))) return SLICEMOE_E_INVALID_ARG;
  if (s->hidden > kMaxHidden) return SLICEMOE_E_UNSUPPORTED;
  return SLICEMOE_OK;
}

// Routing computed in the kernel (run_layer's `fused` argument): logits [T, E] in, lists [T, k] out (optional).
struct FusedRouting {
  const float* logits;
  const float* bias;
  int renorm, rank_high;
  float tau;
  int32_t* ids_out;
  uint8_t* prec_out;
  float* weights_out;
};

static int run_layer(const slicemoe_shape* shape, const slicemoe_expert* experts, const slicemoe_expert* shared,
                     int n_shared, const float* gate_vec, const void* x, int T, const int32_t* ids,
                     const uint8_t* prec, const float* weights, float* y, void* workspace, size_t workspace_bytes,
                     void* stream, const FusedRouting* fused = nullptr, unsigned flags = 0u) {
  int rc = check_shape(shape);
  if (rc != SLICEMOE_OK) return rc;
  if (!experts || !x || !y || !workspace || T <= 0) return SLICEMOE_E_INVALID_ARG;
  if (fused ? !fused->logits : (!ids || !prec || !weights)) return SLICEMOE_E_INVALID_ARG;
  if (fused && shape->n_experts > 32 * ROUTE_MAX_VPT) return SLICEMOE_E_UNSUPPORTED;
  if ((flags & ~(unsigned)(SLICEMOE_LISTS_RESIDENT | SLICEMOE_COOPERATIVE)) != 0u || (fused && flags != 0u)) return SLICEMOE_E_INVALID_ARG;
  const bool coop = (flags & SLICEMOE_COOPERATIVE) != 0u;
  if (n_shared > 0 && !shared) return SLICEMOE_E_INVALID_ARG;
  if (n_shared > 0 && shape->shared_sigmoid_gate && !gate_vec) return SLICEMOE_E_INVALID_ARG;
  if (workspace_bytes < kWsBytes || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SLICEMOE_E_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(x) & 15) return SLICEMOE_E_INVALID_ARG;
  const long long hsum = (long long)shape->top_k * shape->inter + (long long)n_shared * shape->shared_inter;
  if (hsum > kHCap) return SLICEMOE_E_UNSUPPORTED;
  int dev, sms;
  rc = device_setup(&dev, &sms);
  if (rc != SLICEMOE_OK) return rc;
  // at most 4 output row blocks per CTA: what the consumer groups' phase-2 chunk lists are sized for
  if ((shape->hidden / 16 + sms - 1) / sms > 4) return SLICEMOE_E_UNSUPPORTED;

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
  p.lists_resident = (flags & SLICEMOE_LISTS_RESIDENT) ? 1 : 0;
  p.shift = shape->b_high - shape->b_low;
  cudaStream_t st = (cudaStream_t)stream;
  p.logits = nullptr;
  p.bias = fused ? fused->bias : nullptr;
  p.renorm = fused ? fused->renorm : 0;
  p.rank_high = fused ? fused->rank_high : 0;
  p.tau = fused ? fused->tau : 0.f;
  p.ids_out = nullptr;
  p.prec_out = nullptr;
  p.weights_out = nullptr;
  p.ids = nullptr;
  p.prec = nullptr;
  p.weights = nullptr;
  for (int t = 0; t < T; ++t) {
    p.x = reinterpret_cast<const uint16_t*>(x) + (size_t)t * shape->hidden;
    if (fused) {
      const size_t o = (size_t)t * shape->top_k;
      p.logits = fused->logits + (size_t)t * shape->n_experts;
      p.ids_out = fused->ids_out ? fused->ids_out + o : nullptr;
      p.prec_out = fused->prec_out ? fused->prec_out + o : nullptr;
      p.weights_out = fused->weights_out ? fused->weights_out + o : nullptr;
    } else {
      p.ids = ids + (size_t)t * shape->top_k;
      p.prec = prec + (size_t)t * shape->top_k;
      p.weights = weights + (size_t)t * shape->top_k;
    }
    p.y = y + (size_t)t * shape->hidden;
    if (fused) {
      if (shape->group == 128) rc = launch_decode<128, true>(p, dev, sms, 0, st);
      else if (shape->group == 64) rc = launch_decode<64, true>(p, dev, sms, 1, st);
      else rc = launch_decode<32, true>(p, dev, sms, 2, st);
    } else {
      if (shape->group == 128) rc = launch_decode<128, false>(p, dev, sms, 0, st, coop);
      else if (shape->group == 64) rc = launch_decode<64, false>(p, dev, sms, 1, st, coop);
      else rc = launch_decode<32, false>(p, dev, sms, 2, st, coop);
    }
    if (rc != SLICEMOE_OK) return rc;
  }
  return SLICEMOE_OK;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" int slicemoe_trace_read(long long* out_host, int max_ctas, int* slots_out) {
#ifdef SLICEMOE_TRACE
  if (!out_host || max_ctas <= 0) return SLICEMOE_E_INVALID_ARG;
  if (slots_out) *slots_out = kTraceSlots;
  const size_t n = (size_t)(max_ctas < 256 ? max_ctas : 256) * kTraceSlots * sizeof(long long);
  SM_CUDA_TRY(cudaMemcpyFromSymbol(out_host, g_trace, n));
  return SLICEMOE_OK;
#else
  (void)out_host;
  (void)max_ctas;
  (void)slots_out;
  return SLICEMOE_E_UNSUPPORTED;  // this build carries no time stamps
#endif
}

extern "C" size_t slicemoe_workspace_bytes(const slicemoe_shape* shape) {
  (void)shape;
  return kWsBytes;
}

extern "C" int slicemoe_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || workspace_bytes < kWsBytes || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return SLICEMOE_E_INVALID_ARG;
  // header to zero, both h buffers to "empty" (every byte 0xff: see kHEmpty)
  SM_CUDA_TRY(cudaMemsetAsync(workspace, 0, kWsHOff, (cudaStream_t)stream));
  SM_CUDA_TRY(cudaMemsetAsync(reinterpret_cast<uint8_t*>(workspace) + kWsHOff, 0xff, 2 * sizeof(float) * kHCap,
                              (cudaStream_t)stream));
  return SLICEMOE_OK;
}

extern "C" int slicemoe_workspace_set_wait(void* workspace, unsigned long long wait_cycles, unsigned extra_arrivals,
                                           void* stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SLICEMOE_E_INVALID_ARG;
  WsHeader* h = reinterpret_cast<WsHeader*>(workspace);
  cudaStream_t st = (cudaStream_t)stream;
  // small host-to-device copies from pageable memory are staged by the runtime before the call returns
  SM_CUDA_TRY(cudaMemcpyAsync(&h->wait_cycles, &wait_cycles, sizeof(wait_cycles), cudaMemcpyHostToDevice, st));
  SM_CUDA_TRY(cudaMemcpyAsync(&h->extra_arrivals, &extra_arrivals, sizeof(extra_arrivals), cudaMemcpyHostToDevice, st));
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

extern "C" int slicemoe_layer_flags(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                    const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                                    const int32_t* ids, const uint8_t* prec, const float* weights, float* y,
                                    void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
  if (!shape) return SLICEMOE_E_INVALID_ARG;
  return run_layer(shape, experts, shared, shape->n_shared, shared_gate_vec, x, T, ids, prec, weights, y, workspace,
                   workspace_bytes, stream, nullptr, flags);
}

extern "C" int slicemoe_layer_routed(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                     const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                                     const float* logits, const float* bias, int renorm, float tau, int rank_high,
                                     int32_t* ids_out, uint8_t* prec_out, float* weights_out, float* y,
                                     void* workspace, size_t workspace_bytes, void* stream) {
  if (!shape) return SLICEMOE_E_INVALID_ARG;
  FusedRouting f;
  f.logits = logits;
  f.bias = bias;
  f.renorm = renorm;
  f.rank_high = rank_high;
  f.tau = tau;
  f.ids_out = ids_out;
  f.prec_out = prec_out;
  f.weights_out = weights_out;
  return run_layer(shape, experts, shared, shape->n_shared, shared_gate_vec, x, T, nullptr, nullptr, nullptr, y, workspace,
                   workspace_bytes, stream, &f);
}

extern "C" int slicemoe_decode_step_host(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                         const slicemoe_expert* shared, const float* shared_gate_vec,
                                         const void* x_host, const float* logits_host, const float* bias, int renorm,
                                         float tau, int rank_high, float* y_host, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  int rc = check_shape(shape);
  if (rc != SLICEMOE_OK) return rc;
  if (!x_host || !y_host || !workspace || workspace_bytes < kWsBytes) return SLICEMOE_E_INVALID_ARG;
  if (shape->n_experts > 512) return SLICEMOE_E_UNSUPPORTED;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  cudaStream_t st = (cudaStream_t)stream;
  void* dx = ws + kWsStX;
  // logits_host == NULL: the logits follow x in the caller's buffer (x_host is bf16 [hidden] then float32 [E]) and
  // in the staging area alike, and one copy brings both
  float* dlogits = reinterpret_cast<float*>(logits_host ? ws + kWsStLogits : ws + kWsStX + 2 * (size_t)shape->hidden);
  int32_t* dids = reinterpret_cast<int32_t*>(ws + kWsStIds);
  float* dw = reinterpret_cast<float*>(ws + kWsStW);
  uint8_t* dprec = ws + kWsStPrec;
  float* dy = reinterpret_cast<float*>(ws + kWsStY);
  // y_host in pinned (device-mapped) host memory: the kernel writes its 16 output rows per CTA straight
  // into it and the copy back falls away; otherwise y goes through the staging area.
  bool y_direct = false;
  {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, y_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
        (reinterpret_cast<uintptr_t>(attr.devicePointer) & 15) == 0) {
      dy = reinterpret_cast<float*>(attr.devicePointer);
      y_direct = true;
    } else {
      (void)cudaGetLastError();  // an unregistered pointer is not an error here
    }
  }
  if (logits_host) {
    SM_CUDA_TRY(cudaMemcpyAsync(dx, x_host, 2 * (size_t)shape->hidden, cudaMemcpyHostToDevice, st));
    SM_CUDA_TRY(cudaMemcpyAsync(dlogits, logits_host, 4 * (size_t)shape->n_experts, cudaMemcpyHostToDevice, st));
  } else {
    SM_CUDA_TRY(cudaMemcpyAsync(dx, x_host, 2 * (size_t)shape->hidden + 4 * (size_t)shape->n_experts,
                                cudaMemcpyHostToDevice, st));
  }
  rc = slicemoe_layer_routed(shape, experts, shared, shared_gate_vec, dx, 1, dlogits, bias, renorm, tau, rank_high, dids,
                             dprec, dw, dy, workspace, workspace_bytes, stream);
  if (rc != SLICEMOE_OK) return rc;
  if (!y_direct) SM_CUDA_TRY(cudaMemcpyAsync(y_host, dy, 4 * (size_t)shape->hidden, cudaMemcpyDeviceToHost, st));
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
  // The array keeps whatever the previous call left: the header (launch count, status) must start at zero, and the
  // h buffer the first launch then uses must be empty (the launches clear the other one for their successors).
  SM_CUDA_TRY(cudaMemsetAsync(ws, 0, kWsHOff, (cudaStream_t)stream));
  SM_CUDA_TRY(cudaMemsetAsync(reinterpret_cast<uint8_t*>(ws) + kWsHOff, 0xff, sizeof(float) * kHCap, (cudaStream_t)stream));
  return run_layer(shape, experts, shared, shape->n_shared, shared_gate_vec, x, T, ids, prec, weights, y, ws, kWsBytes,
                   stream);
}
