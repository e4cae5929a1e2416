// Shared by the CUDA translation units: error plumbing and the physical plane layout.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "slicemoe.h"

// The CUDA error behind the most recent SLICEMOE_E_CUDA (see slicemoe_last_cuda_error).
extern int g_slicemoe_last_cuda_error;

#define SM_CUDA_TRY(expr)                     \
  do {                                        \
    cudaError_t _e = (expr);                  \
    if (_e != cudaSuccess) {                  \
      g_slicemoe_last_cuda_error = (int)_e;   \
      return SLICEMOE_E_CUDA;                 \
    }                                         \
  } while (0)

#define SM_LAUNCH_CHECK()                     \
  do {                                        \
    cudaError_t _e = cudaGetLastError();      \
    if (_e != cudaSuccess) {                  \
      g_slicemoe_last_cuda_error = (int)_e;   \
      return SLICEMOE_E_CUDA;                 \
    }                                         \
  } while (0)

namespace slicemoe {

// ---- physical layout of a slice plane (see slicemoe.h) --------------------------------------
// A plane is a sequence of 512-byte blocks, one per (16-row block rb, 64-column tile st), at block index
// rb * (K / 64) + st.  A block is 32 lanes x 4 little-endian 32-bit words; lane L = 4 * g + c.  Byte j of
// word w holds the element (row 16 rb + g, k) in its low nibble and (row 16 rb + g + 8, k) in its high
// nibble, with k = 64 st + 16 w + 4 c + j.  So `word & 0x0f0f0f0f` and `(word >> 4) & 0x0f0f0f0f` are the
// two row halves of an m16n8k32 integer mma A fragment.
__host__ __device__ inline size_t plane_word_index(int K, int rb, int st, int lane, int w) {
  return ((size_t)rb * (K >> 6) + st) * 128 + (size_t)lane * 4 + w;
}

// Where element (n, k) lives: word index and nibble position within the word.
__host__ __device__ inline void plane_locate(int K, int n, int k, size_t* word, int* pos) {
  const int rb = n >> 4, r = n & 15;
  const int g = r & 7, hi = r >> 3;
  const int st = k >> 6, kk = k & 63;
  const int w = kk >> 4, c = (kk & 15) >> 2, j = kk & 3;
  *word = plane_word_index(K, rb, st, g * 4 + c, w);
  *pos = 2 * j + hi;
}

// Index of the (scale, zp) entry of (row n, group g): [N/16][K/group][16].
__host__ __device__ inline size_t meta_index(int ngroups, int n, int g) {
  return ((size_t)(n >> 4) * ngroups + g) * 16 + (n & 15);
}

inline bool valid_group(int g) { return g == 32 || g == 64 || g == 128; }
// The slice widths of Table 1: MAT84, MAT63, MAT42 (b_high-bit codes, the top b_low bits form the MSB slice).
inline bool valid_widths(int b_high, int b_low) {
  return (b_high == 8 && b_low == 4) || (b_high == 6 && b_low == 3) || (b_high == 4 && b_low == 2);
}

}  // namespace slicemoe
