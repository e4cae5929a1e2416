// slicemoe_route_topk: softmax + top-k with optional cache-priority bias and precision request.
//
// One warp per token.  Each lane keeps E/32 (<= 16) logits in registers; the softmax uses fp32
// expf; selection runs k rounds of a warp arg-max on key = logit + bias (one fp32 add, NaN -> -inf)
// with ties broken towards the lower expert index, so the ids are a pure function of the keys.
#include <math_constants.h>

#include "common.cuh"

namespace slicemoe {

constexpr int ROUTE_MAX_VPT = 16;  // values per lane -> E <= 512

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
  const float* row = logits + (size_t)warp * E;

  float key[ROUTE_MAX_VPT];
  float val[ROUTE_MAX_VPT];
  float vmax = -CUDART_INF_F;
#pragma unroll
  for (int v = 0; v < ROUTE_MAX_VPT; ++v) {
    const int e = v * 32 + lane;
    float l = -CUDART_INF_F, kk = -CUDART_INF_F;
    if (e < E) {
      l = row[e];
      if (isnan(l)) l = -CUDART_INF_F;
      kk = row[e];
      if (bias) kk = __fadd_rn(kk, bias[e]);
      if (isnan(kk)) kk = -CUDART_INF_F;
    }
    val[v] = l;
    key[v] = kk;
    vmax = fmaxf(vmax, l);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, off));
  float sum = 0.0f;
#pragma unroll
  for (int v = 0; v < ROUTE_MAX_VPT; ++v) {
    const int e = v * 32 + lane;
    if (e < E) sum += expf(val[v] - vmax);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  const float inv_sum = 1.0f / sum;

  uint32_t taken = 0;  // bit v: this lane's value v was already selected
  float wsel = 0.0f;   // lane j keeps the weight of selection j (k <= 16 < 32)
  int idsel = 0;
  float wtotal = 0.0f;
  for (int j = 0; j < k; ++j) {
    float best = -CUDART_INF_F;
    int best_e = 0x7fffffff;
#pragma unroll
    for (int v = 0; v < ROUTE_MAX_VPT; ++v) {
      const int e = v * 32 + lane;
      if (e < E && !((taken >> v) & 1u)) {
        if (best_e == 0x7fffffff || key[v] > best) {  // ascending e within a lane: strict > keeps the lower index
          best = key[v];
          best_e = e;
        }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, off);
      const int oe = __shfl_xor_sync(0xffffffffu, best_e, off);
      const bool other_wins = (oe != 0x7fffffff) && (best_e == 0x7fffffff || ob > best || (ob == best && oe < best_e));
      if (other_wins) {
        best = ob;
        best_e = oe;
      }
    }
    // every lane now agrees on best_e; its owner marks it and provides the probability
    const int owner = best_e & 31, ov = best_e >> 5;
    float p = 0.0f;
#pragma unroll
    for (int v = 0; v < ROUTE_MAX_VPT; ++v) {
      if (v == ov && lane == owner) {
        taken |= 1u << v;
        p = expf(val[v] - vmax) * inv_sum;
      }
    }
    p = __shfl_sync(0xffffffffu, p, owner);
    wtotal += p;
    if (lane == j) {
      wsel = p;
      idsel = best_e;
    }
  }
  if (lane < k) {
    const size_t o = (size_t)warp * k + lane;
    ids[o] = idsel;
    weights[o] = renorm ? wsel / wtotal : wsel;
    if (prec_req) prec_req[o] = (uint8_t)((wsel >= tau || lane < rank_high) ? 1 : 0);
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
