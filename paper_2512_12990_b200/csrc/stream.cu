// A measuring stick for the decode kernel: the bytes one decode step of a layer reads - the slice planes, scales
// and zero-points of the listed experts at their precisions, and of the shared experts - brought into shared
// memory with the same bulk copies, one CTA per SM, and nothing else: no arithmetic, no exchange between CTAs.
// Its time per launch is what the memory system alone needs for a step.
#include "common.cuh"

namespace slicemoe {

namespace {

constexpr int kProbeUnit = 16384;   // bytes per copy, the decode kernel's plane unit
constexpr int kProbeDepth = 12;     // copies in flight per CTA
constexpr int kProbeMaxSegs = (SLICEMOE_MAX_TOP_K + SLICEMOE_MAX_SHARED) * 12;  // 4 per (slot, matrix)
constexpr unsigned long long kProbeWaitCycles = 100000000ull;  // every wait is bounded (about 50 ms)

struct ProbeParams {
  const slicemoe_expert* experts;
  const slicemoe_expert* shared;
  const int32_t* ids;
  const uint8_t* prec;
  int n_experts, n_shared, k;
  int group;
  int dependent;
  unsigned long long* bytes_out;  // may be null: CTA 0 adds the step's bytes
  int* status;                    // may be null: set to 1 if a wait ran out
};

struct Seg {
  const uint8_t* ptr;
  unsigned long long first_unit;  // units before this segment
  unsigned bytes;
};

__device__ __forceinline__ uint32_t p_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool p_try(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool p_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!p_try(bar, parity))
    if ((unsigned long long)(clock64() - t0) > kProbeWaitCycles) return false;
  return true;
}

__global__ void __launch_bounds__(32, 1) stream_probe_kernel(const __grid_constant__ ProbeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ Seg segs[kProbeMaxSegs];
  __shared__ __align__(8) unsigned long long bars[kProbeDepth];
  __shared__ int nsegs;
  __shared__ unsigned long long total_units;
  const int lane = threadIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (lane == 0) {
    for (int i = 0; i < kProbeDepth; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(p_smem_u32(&bars[i])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (p.dependent) asm volatile("griddepcontrol.wait;" ::: "memory");
  {
    // The segment list: for every slot its three matrices' MSB plane, LSB plane (8 bits), scales, zero-points.
    // Lane l takes the (slot, matrix) pairs l and l + 32, so that the pointer loads of all pairs are in flight
    // together; a warp scan turns the pairs' unit counts into each segment's first unit.
    constexpr int kPairs = (SLICEMOE_MAX_TOP_K + SLICEMOE_MAX_SHARED) * 3;
    static_assert(kPairs <= 64, "two pairs per lane");
    const int npairs = (p.n_shared + p.k) * 3;
    const uint8_t* ptr[2][4];
    unsigned long long sz[2][4];
    unsigned long long units_of[2], bytes_of[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int pair = lane + 32 * h;
      units_of[h] = bytes_of[h] = 0;
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        ptr[h][a] = nullptr;
        sz[h][a] = 0;
      }
      if (pair >= npairs) continue;
      const int slot = pair / 3, m = pair % 3;
      const slicemoe_expert* ex = nullptr;
      bool p8 = true;
      if (slot < p.n_shared) {
        ex = p.shared + slot;
      } else {
        const int e = p.ids[slot - p.n_shared];
        if (e >= 0 && e < p.n_experts) {
          ex = p.experts + e;
          p8 = p.prec[slot - p.n_shared] != 0;
        }
      }
      if (!ex) continue;
      const slicemoe_mat mt = reinterpret_cast<const slicemoe_mat*>(ex)[m];
      const unsigned long long w = (unsigned long long)mt.N * (unsigned long long)mt.K;
      ptr[h][0] = reinterpret_cast<const uint8_t*>(mt.msb);
      ptr[h][1] = p8 ? reinterpret_cast<const uint8_t*>(mt.lsb) : nullptr;
      ptr[h][2] = reinterpret_cast<const uint8_t*>(mt.scale);
      ptr[h][3] = mt.zp;
      sz[h][0] = sz[h][1] = w / 2;
      sz[h][2] = w / (unsigned)p.group * 2;
      sz[h][3] = w / (unsigned)p.group;
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        if (!ptr[h][a]) sz[h][a] = 0;
        units_of[h] += (sz[h][a] + kProbeUnit - 1) / kProbeUnit;
        bytes_of[h] += sz[h][a];
      }
    }
    unsigned long long base = 0, bytes = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      unsigned long long incl = units_of[h], bsum = bytes_of[h];
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, off);
      unsigned long long first = base + incl - units_of[h];
      const int pair = lane + 32 * h;
      if (pair < npairs) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {  // a segment without bytes shares its first unit with the next one
          segs[pair * 4 + a].ptr = ptr[h][a];
          segs[pair * 4 + a].first_unit = first;
          segs[pair * 4 + a].bytes = (unsigned)sz[h][a];
          first += (sz[h][a] + kProbeUnit - 1) / kProbeUnit;
        }
      }
      base += __shfl_sync(0xffffffffu, incl, 31);
      bytes += bsum;
    }
    if (lane == 0) {
      nsegs = npairs * 4;
      total_units = base;
      if (blockIdx.x == 0 && p.bytes_out) atomicAdd(p.bytes_out, bytes);
    }
  }
  __syncwarp();
  if (lane != 0) return;

  // units blockIdx.x, + gridDim.x, ...: copy i of this CTA lands in ring slot i % depth once the copy that used
  // the slot before has completed (that wait is all the "consumption" there is)
  const uint32_t ring = p_smem_u32(smem);
  bool ok = true;
  int seg = 0;
  unsigned i = 0;
  for (unsigned long long u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++i) {
    while (seg + 1 < nsegs && segs[seg + 1].first_unit <= u) ++seg;
    const unsigned off = (unsigned)(u - segs[seg].first_unit) * kProbeUnit;
    const unsigned bytes = min((unsigned)kProbeUnit, segs[seg].bytes - off);
    const unsigned slot = i % kProbeDepth, round = i / kProbeDepth;
    const uint32_t bar = p_smem_u32(&bars[slot]);
    if (round > 0) ok = p_wait(bar, (round - 1) & 1);
    if (!ok) break;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     ring + slot * kProbeUnit),
                 "l"(segs[seg].ptr + off), "r"(bytes), "r"(bar)
                 : "memory");
  }
  // never leave with copies in flight
  const unsigned n_issued = i;
  for (unsigned j = n_issued > (unsigned)kProbeDepth ? n_issued - kProbeDepth : 0u; j < n_issued; ++j) {
    if (!p_wait(p_smem_u32(&bars[j % kProbeDepth]), (j / kProbeDepth) & 1)) ok = false;
  }
  if (!ok && p.status) *p.status = 1;
}

}  // namespace

}  // namespace slicemoe

using namespace slicemoe;

extern "C" int slicemoe_stream_probe(const slicemoe_shape* shape, const slicemoe_expert* experts,
                                     const slicemoe_expert* shared, const int32_t* ids, const uint8_t* prec,
                                     int dependent, unsigned long long* bytes_out_device, int* status_out_device,
                                     void* stream) {
  if (!shape || !experts || !ids || !prec) return SLICEMOE_E_INVALID_ARG;
  if (!valid_group(shape->group) || shape->top_k < 1 || shape->top_k > SLICEMOE_MAX_TOP_K || shape->n_experts <= 0)
    return SLICEMOE_E_INVALID_ARG;
  if (shape->n_shared < 0 || shape->n_shared > SLICEMOE_MAX_SHARED || (shape->n_shared > 0 && !shared))
    return SLICEMOE_E_INVALID_ARG;
  int dev = 0, sms = 0;
  SM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SLICEMOE_E_UNSUPPORTED;
  SM_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  constexpr int smem_bytes = kProbeUnit * kProbeDepth;
  static bool attr_set[64];
  if (!attr_set[dev]) {
    SM_CUDA_TRY(cudaFuncSetAttribute(stream_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
    attr_set[dev] = true;
  }
  ProbeParams p;
  p.experts = experts;
  p.shared = shared;
  p.ids = ids;
  p.prec = prec;
  p.n_experts = shape->n_experts;
  p.n_shared = shape->n_shared;
  p.k = shape->top_k;
  p.group = shape->group;
  p.dependent = dependent ? 1 : 0;
  p.bytes_out = bytes_out_device;
  p.status = status_out_device;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(sms);
  cfg.blockDim = dim3(32);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SM_CUDA_TRY(cudaLaunchKernelEx(&cfg, stream_probe_kernel, p));
  return SLICEMOE_OK;
}
