// slicemoe_pack: AMAT quantiser + MSB/LSB slice planes in the tiled layout, and the inverse hooks.
//
// Two kernels per matrix.  pack_meta: one warp per (row, K-group) finds min/max and writes the
// fp16 scale and u8 zero-point.  pack_planes: one thread per 32-bit output word (2 rows x 4
// consecutive k) quantises its 8 weights and writes the MSB word and the LSB word, so stores are
// fully coalesced.  All arithmetic that decides an integer uses IEEE division and rint (no
// fast-math, no reciprocal), so the codes are bit-exact against a float32 CPU evaluation.
#include <cuda_fp16.h>

#include "common.cuh"

namespace slicemoe {

__global__ void pack_meta_kernel(const float* __restrict__ W, int N, int K, int group, int qmax,
                                 uint16_t* __restrict__ scale, uint8_t* __restrict__ zp) {
  const int ngroups = K / group;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= (long long)N * ngroups) return;
  const int n = (int)(warp / ngroups), g = (int)(warp % ngroups);
  const float* src = W + (size_t)n * K + (size_t)g * group;
  float lo = 0.0f, hi = 0.0f;  // the range always contains zero
  for (int i = lane; i < group; i += 32) {
    const float w = src[i];
    lo = fminf(lo, w);
    hi = fmaxf(hi, w);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
  }
  if (lane == 0) {
    const float s32 = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
    __half s16 = __float2half_rn(s32);
    float s = __half2float(s16);
    int z = 0;
    const bool degenerate = (hi == lo) || (s == 0.0f) || isinf(s) || isnan(s);
    if (degenerate) {
      s16 = __float2half_rn(1.0f);
    } else {
      const float zf = rintf(__fdiv_rn(-lo, s));
      z = (int)fminf(fmaxf(zf, 0.0f), (float)qmax);
    }
    const size_t idx = meta_index(ngroups, n, g);
    scale[idx] = __half_as_ushort(s16);
    zp[idx] = (uint8_t)z;
  }
}

__device__ __forceinline__ int quantise_one(float w, float s, int z, int qmax) {
  float r = rintf(__fdiv_rn(w, s));
  r = fminf(fmaxf(r, -1.0e9f), 1.0e9f);
  int q = (int)r + z;
  return min(max(q, 0), qmax);
}

__global__ void pack_planes_kernel(const float* __restrict__ W, int N, int K, int group, int qmax, int shift,
                                   const uint16_t* __restrict__ scale, const uint8_t* __restrict__ zp,
                                   uint32_t* __restrict__ msb, uint32_t* __restrict__ lsb) {
  const size_t nwords = (size_t)N * K / 8;
  const size_t widx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (widx >= nwords) return;
  // invert plane_word_index: widx = ((rb*(K/64) + st)*32 + lane)*4 + w
  const int w = (int)(widx & 3);
  const int lane = (int)((widx >> 2) & 31);
  const size_t blk = widx >> 7;
  const int st = (int)(blk % (size_t)(K >> 6));
  const int rb = (int)(blk / (size_t)(K >> 6));
  const int g8 = lane >> 2, c = lane & 3;
  const int k0 = st * 64 + w * 16 + c * 4;
  const int ngroups = K / group;
  const int grp = k0 / group;  // the 4 consecutive k share a group (group % 16 == 0)
  uint32_t mw = 0, lw = 0;
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    const int n = rb * 16 + g8 + 8 * hi;
    const float4 v = *reinterpret_cast<const float4*>(W + (size_t)n * K + k0);
    const size_t mi = meta_index(ngroups, n, grp);
    const float s = __half2float(__ushort_as_half(scale[mi]));
    const int z = zp[mi];
    const float vals[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int q = quantise_one(vals[j], s, z, qmax);
      const int pos = 2 * j + hi;
      mw |= (uint32_t)(q >> shift) << (4 * pos);  // a slice narrower than 4 bits sits in the low bits of its nibble
      lw |= (uint32_t)(q & ((1 << shift) - 1)) << (4 * pos);
    }
  }
  msb[widx] = mw;
  lsb[widx] = lw;
}

__global__ void unpack_plane_kernel(const uint32_t* __restrict__ plane, int N, int K,
                                    uint8_t* __restrict__ nibbles) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)N * K) return;
  const int n = (int)(idx / K), k = (int)(idx % K);
  size_t word;
  int pos;
  plane_locate(K, n, k, &word, &pos);
  nibbles[idx] = (uint8_t)((plane[word] >> (4 * pos)) & 15u);
}

__global__ void unpack_meta_kernel(const uint16_t* __restrict__ scale, const uint8_t* __restrict__ zp,
                                   int N, int ngroups, uint16_t* __restrict__ scale_rm,
                                   uint8_t* __restrict__ zp_rm) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)N * ngroups) return;
  const int n = (int)(idx / ngroups), g = (int)(idx % ngroups);
  const size_t mi = meta_index(ngroups, n, g);
  scale_rm[idx] = scale[mi];
  zp_rm[idx] = zp[mi];
}

// Dense storage of a slice narrower than a nibble: the plane's nibbles, in the order of its bytes (low nibble
// first), as a little-endian bit stream of `bits` bits each.  One thread per 32-bit plane word = 8 nibbles =
// `bits` bytes of the stream.
__global__ void compact_plane_kernel(const uint32_t* __restrict__ plane, size_t n_words, int bits,
                                     uint8_t* __restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_words) return;
  const uint32_t w = plane[i], mask = (1u << bits) - 1u;
  uint32_t packed = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) packed |= ((w >> (4 * j)) & mask) << (bits * j);
  for (int b = 0; b < bits; ++b) out[i * bits + b] = (uint8_t)(packed >> (8 * b));
}

__global__ void expand_plane_kernel(const uint8_t* __restrict__ in, size_t n_words, int bits,
                                    uint32_t* __restrict__ plane) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_words) return;
  uint32_t packed = 0;
  for (int b = 0; b < bits; ++b) packed |= (uint32_t)in[i * bits + b] << (8 * b);
  const uint32_t mask = (1u << bits) - 1u;
  uint32_t w = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) w |= ((packed >> (bits * j)) & mask) << (4 * j);
  plane[i] = w;
}

static int check_dims(int N, int K, int group) {
  if (N <= 0 || K <= 0 || (N % 16) != 0 || (K % 128) != 0) return SLICEMOE_E_INVALID_ARG;
  if (!valid_group(group)) return SLICEMOE_E_UNSUPPORTED;
  if ((K % group) != 0) return SLICEMOE_E_INVALID_ARG;
  return SLICEMOE_OK;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" size_t slicemoe_plane_bytes(int N, int K) {
  if (N <= 0 || K <= 0) return 0;
  return (size_t)N * K / 2;
}

extern "C" size_t slicemoe_meta_count(int N, int K, int group) {
  if (N <= 0 || K <= 0 || group <= 0) return 0;
  return (size_t)N * (K / group);
}

extern "C" int slicemoe_pack(const float* W, int N, int K, int group, int b_high, int b_low, void* msb,
                             void* lsb, uint16_t* scale, uint8_t* zp, void* stream) {
  if (!W || !msb || !lsb || !scale || !zp) return SLICEMOE_E_INVALID_ARG;
  if (!valid_widths(b_high, b_low)) return SLICEMOE_E_UNSUPPORTED;
  const int qmax = (1 << b_high) - 1, shift = b_high - b_low;
  const int rc = check_dims(N, K, group);
  if (rc != SLICEMOE_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const long long nwarps = (long long)N * (K / group);
  const int threads = 256;
  const long long blocks_meta = (nwarps * 32 + threads - 1) / threads;
  pack_meta_kernel<<<(unsigned)blocks_meta, threads, 0, st>>>(W, N, K, group, qmax, scale, zp);
  SM_LAUNCH_CHECK();
  const size_t nwords = (size_t)N * K / 8;
  const size_t blocks_planes = (nwords + threads - 1) / threads;
  pack_planes_kernel<<<(unsigned)blocks_planes, threads, 0, st>>>(
      W, N, K, group, qmax, shift, scale, zp, reinterpret_cast<uint32_t*>(msb), reinterpret_cast<uint32_t*>(lsb));
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

extern "C" int slicemoe_unpack_plane(const void* plane, int N, int K, uint8_t* nibbles, void* stream) {
  if (!plane || !nibbles) return SLICEMOE_E_INVALID_ARG;
  if (N <= 0 || K <= 0 || (N % 16) != 0 || (K % 128) != 0) return SLICEMOE_E_INVALID_ARG;
  const size_t total = (size_t)N * K;
  const int threads = 256;
  unpack_plane_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const uint32_t*>(plane), N, K, nibbles);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

extern "C" int slicemoe_unpack_meta(const uint16_t* scale, const uint8_t* zp, int N, int K, int group,
                                    uint16_t* scale_rm, uint8_t* zp_rm, void* stream) {
  if (!scale || !zp || !scale_rm || !zp_rm) return SLICEMOE_E_INVALID_ARG;
  const int rc = check_dims(N, K, group);
  if (rc != SLICEMOE_OK) return rc;
  const int ngroups = K / group;
  const size_t total = (size_t)N * ngroups;
  const int threads = 256;
  unpack_meta_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, (cudaStream_t)stream>>>(
      scale, zp, N, ngroups, scale_rm, zp_rm);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

extern "C" size_t slicemoe_compact_bytes(int N, int K, int bits) {
  if (N <= 0 || K <= 0 || bits < 2 || bits > 4) return 0;
  return (size_t)N * K / 8 * bits;
}

static int compact_args(const void* a, const void* b, int N, int K, int bits) {
  if (!a || !b) return SLICEMOE_E_INVALID_ARG;
  if (N <= 0 || K <= 0 || (N % 16) != 0 || (K % 128) != 0) return SLICEMOE_E_INVALID_ARG;
  if (bits < 2 || bits > 4) return SLICEMOE_E_UNSUPPORTED;
  return SLICEMOE_OK;
}

extern "C" int slicemoe_compact_plane(const void* plane, int N, int K, int bits, void* compact, void* stream) {
  const int rc = compact_args(plane, compact, N, K, bits);
  if (rc != SLICEMOE_OK) return rc;
  const size_t n_words = (size_t)N * K / 8;
  const int threads = 256;
  compact_plane_kernel<<<(unsigned)((n_words + threads - 1) / threads), threads, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const uint32_t*>(plane), n_words, bits, reinterpret_cast<uint8_t*>(compact));
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

extern "C" int slicemoe_expand_plane(const void* compact, int N, int K, int bits, void* plane, void* stream) {
  const int rc = compact_args(compact, plane, N, K, bits);
  if (rc != SLICEMOE_OK) return rc;
  const size_t n_words = (size_t)N * K / 8;
  const int threads = 256;
  expand_plane_kernel<<<(unsigned)((n_words + threads - 1) / threads), threads, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const uint8_t*>(compact), n_words, bits, reinterpret_cast<uint32_t*>(plane));
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}
