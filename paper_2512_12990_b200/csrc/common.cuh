// Shared by the CUDA translation units: error plumbing and the physical plane layout.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "slicemoe.h"

#define SM_CUDA_TRY(expr)                          \
  do {                                             \
    cudaError_t _e = (expr);                       \
    if (_e != cudaSuccess) return SLICEMOE_E_CUDA; \
  } while (0)

#define SM_LAUNCH_CHECK()                          \
  do {                                             \
    cudaError_t _e = cudaGetLastError();           \
    if (_e != cudaSuccess) return SLICEMOE_E_CUDA; \
  } while (0)

namespace slicemoe {

// ---- physical layout of a slice plane (see slicemoe.h) --------------------------------------
// 32-bit word index of (row-block rb, k-step t = k/16, lane L) in a plane of a matrix with K columns.
__host__ __device__ inline size_t plane_word_index(int K, int rb, int t, int lane) {
  return ((size_t)rb * (K >> 6) + (t >> 2)) * 128 + (size_t)lane * 4 + (t & 3);
}

// Where element (n, k) lives: word index and nibble position within the word.
__host__ __device__ inline void plane_locate(int K, int n, int k, size_t* word, int* pos) {
  const int rb = n >> 4, r = n & 15;
  const int g = r & 7, i0 = r >> 3;
  const int t = k >> 4, kk = k & 15;
  const int c = kk >> 2, rem = kk & 3;
  const int i = i0 + 2 * (rem >> 1), hf = rem & 1;
  *word = plane_word_index(K, rb, t, g * 4 + c);
  *pos = i + 4 * hf;
}

// Index of the (scale, zp) entry of (row n, group g): [N/16][K/group][16].
__host__ __device__ inline size_t meta_index(int ngroups, int n, int g) {
  return ((size_t)(n >> 4) * ngroups + g) * 16 + (n & 15);
}

inline bool valid_group(int g) { return g == 32 || g == 64 || g == 128; }

}  // namespace slicemoe
