// slicemoe_route_topk: softmax + top-k with optional cache-priority bias and precision request, one warp per
// token (the arithmetic is in route.cuh).
#include "common.cuh"
#include "route.cuh"

namespace slicemoe {

__global__ void route_topk_kernel(const float* __restrict__ logits, int T, int E, int k,
                                  const float* __restrict__ bias, int renorm, float tau, int rank_high,
                                  int32_t* __restrict__ ids, float* __restrict__ weights,
                                  uint8_t* __restrict__ prec_req) {
  // Programmatic dependent launch: the kernel after this one may start launching now; this one waits for the
  // kernels before it (which may still be producing the logits) before it reads anything.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= T) return;
  const RouteSel sel = route_warp(logits + (size_t)warp * E, E, k, bias, renorm, tau, rank_high, lane);
  if (lane < k) {
    const size_t o = (size_t)warp * k + lane;
    ids[o] = sel.id;
    weights[o] = sel.w;
    if (prec_req) prec_req[o] = sel.prec_req;
  }
}

}  // namespace slicemoe

extern "C" int slicemoe_route_topk(const float* logits, int T, int E, int k, const float* bias, int renorm,
                                   float tau, int rank_high, int32_t* ids, float* weights,
                                   uint8_t* prec_req, void* stream) {
  if (!logits || !ids || !weights) return SLICEMOE_E_INVALID_ARG;
  if (T <= 0 || E <= 0 || k < 1 || k > E || k > SLICEMOE_MAX_TOP_K) return SLICEMOE_E_INVALID_ARG;
  if (E > 32 * slicemoe::ROUTE_MAX_VPT) return SLICEMOE_E_UNSUPPORTED;
  const int threads = 128;  // 4 tokens per block
  const int blocks = (T + 3) / 4;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(threads);
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SM_CUDA_TRY(cudaLaunchKernelEx(&cfg, slicemoe::route_topk_kernel, logits, T, E, k, bias, renorm, tau, rank_high, ids,
                                 weights, prec_req));
  return SLICEMOE_OK;
}
