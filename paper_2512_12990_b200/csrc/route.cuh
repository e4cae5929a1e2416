// Routing of one token by one warp: softmax + top-k with optional cache-priority bias and precision request
// (Section 4.1: gating scores decide which experts run and which of them matter most).  Shared by the
// stand-alone routing kernel and the decode kernel's fused prologue, so both give the same bits.
//
// Each lane keeps E/32 (<= 16) logits in registers; the softmax uses fp32 expf; selection runs k rounds of a
// warp arg-max on key = logit + bias (one fp32 add, NaN -> -inf) with ties broken towards the lower expert
// index, so the ids are a pure function of the keys.
#pragma once

#include <math_constants.h>
#include <stdint.h>

namespace slicemoe {

constexpr int ROUTE_MAX_VPT = 16;  // values per lane -> E <= 512

struct RouteSel {  // lane j < k holds selection j
  int id;
  float w;
  uint8_t prec_req;
};

// VPT: values per lane, a compile-time bound with 32 VPT >= E.  The result does not depend on it: a lane's
// values are visited in the same order, only the unrolled loops over absent values are shorter.
template <int VPT>
__device__ __forceinline__ RouteSel route_warp_vpt(const float* __restrict__ row, int E, int k,
                                                   const float* __restrict__ bias, int renorm, float tau, int rank_high,
                                                   int lane) {
  float key[VPT];
  float val[VPT];
  float vmax = -CUDART_INF_F;
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
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
  for (int v = 0; v < VPT; ++v) {
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
    for (int v = 0; v < VPT; ++v) {
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
    for (int v = 0; v < VPT; ++v) {
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
  RouteSel sel;
  sel.id = idsel;
  sel.w = renorm ? wsel / wtotal : wsel;
  sel.prec_req = (uint8_t)((wsel >= tau || lane < rank_high) ? 1 : 0);
  return sel;
}

__device__ __forceinline__ RouteSel route_warp(const float* __restrict__ row, int E, int k, const float* __restrict__ bias,
                                               int renorm, float tau, int rank_high, int lane) {
  if (E <= 64) return route_warp_vpt<2>(row, E, k, bias, renorm, tau, rank_high, lane);
  if (E <= 128) return route_warp_vpt<4>(row, E, k, bias, renorm, tau, rank_high, lane);
  return route_warp_vpt<ROUTE_MAX_VPT>(row, E, k, bias, renorm, tau, rank_high, lane);
}

}  // namespace slicemoe
