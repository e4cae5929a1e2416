// Prefill of one MoE layer from bit-sliced AMAT weights: many tokens at once, so the expert FFN is a
// genuine dense contraction (Section 3 of the paper: prefill loads every expert of a layer; Section 5.3:
// prefill runs at the precision each expert's cached slices allow).
//
// Steps, all on the device:
//   1. count the tokens of every routed expert, lay the experts' token rows out one after the other
//      (each expert padded to a multiple of 128 rows), list the 128-row tiles;
//   2. gather x (bf16) into that order as fp16 (exact for every bf16 value in fp16's normal range);
//   3. grouped GEMM 1: per tile  H = silu(X Wg^T) * (X Wu^T)  (fp16 out);
//   4. grouped GEMM 2: per tile  Yrow = H Wd^T  (fp32 out, one row per (token, expert) pair);
//   5. combine: y[t] = sum_j w[t,j] Yrow[pos(t,j)] + shared experts, in list order (deterministic).
// In both GEMMs the weight tile is dequantised on the fly from the nibble planes into fp16 in shared
// memory - s * (q - zp) from both slices, 16 s * (q_msb - (zp >> 4)) from the MSB slice alone - and fed
// to the tensor cores (mma.sync m16n8k16, fp16 x fp16 -> fp32).  fp16 rather than bf16: a dequantised
// weight needs 11 significant bits to stay inside the parity tolerance, bf16 has 8.
#include <cuda_fp16.h>

#include "common.cuh"

namespace slicemoe {

constexpr int kPfThreads = 512;
constexpr int kPfTileM = 128;  // token rows per tile
constexpr int kPfTileB = 128;  // weight rows per tile: 64 gate + 64 up columns of h (GEMM 1), 128 columns of y (GEMM 2)
constexpr int kPfChunkK = 64;  // contraction columns per pipeline step (one plane block)
constexpr int kPfStride = kPfChunkK + 8;  // halves per shared-memory row: 144 bytes, conflict-free for ldmatrix

// ---- workspace layout (host and device agree through this one function) --------------------------------
struct PfLayout {
  size_t counts, cursor, offsets, tile_expert, tile_row0, ntiles, row_token, posmap, gate, xs, h, yrow, total;
  int rmax, max_tiles, nexp_all;
};
__host__ __device__ inline size_t pf_align(size_t v) { return (v + 255) & ~(size_t)255; }
__host__ __device__ inline PfLayout pf_layout(int T, int E, int k, int n_shared, int hidden, int inter, int shared_inter) {
  PfLayout L;
  L.nexp_all = E + n_shared;
  // routed rows: T*k plus at most 127 rows of padding per expert; shared: T rows each, padded
  const int tpad = (T + kPfTileM - 1) / kPfTileM * kPfTileM;
  L.rmax = (T * k + E * (kPfTileM - 1) + kPfTileM - 1) / kPfTileM * kPfTileM + n_shared * tpad;
  L.max_tiles = L.rmax / kPfTileM;
  const int wide = inter > shared_inter ? inter : shared_inter;
  size_t o = 0;
  L.counts = o;       o = pf_align(o + sizeof(int) * L.nexp_all);
  L.cursor = o;       o = pf_align(o + sizeof(int) * L.nexp_all);
  L.offsets = o;      o = pf_align(o + sizeof(int) * (L.nexp_all + 1));
  L.tile_expert = o;  o = pf_align(o + sizeof(int) * L.max_tiles);
  L.tile_row0 = o;    o = pf_align(o + sizeof(int) * L.max_tiles);
  L.ntiles = o;       o = pf_align(o + sizeof(int) * 4);
  L.row_token = o;    o = pf_align(o + sizeof(int) * L.rmax);
  L.posmap = o;       o = pf_align(o + sizeof(int) * (size_t)T * (k + n_shared));
  L.gate = o;         o = pf_align(o + sizeof(float) * T);
  L.xs = o;           o = pf_align(o + sizeof(__half) * (size_t)L.rmax * hidden);
  L.h = o;            o = pf_align(o + sizeof(__half) * (size_t)L.rmax * wide);
  L.yrow = o;         o = pf_align(o + sizeof(float) * (size_t)L.rmax * hidden);
  L.total = o;
  return L;
}

// ---- step 1: token rows per expert -----------------------------------------------------------------------
__global__ void pf_count_kernel(const int32_t* __restrict__ ids, int n, int E, int* __restrict__ counts,
                                unsigned* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int e = ids[i];
  if (e < 0 || e >= E) {
    atomicOr(status, (unsigned)SLICEMOE_STATUS_BAD_EXPERT_ID);
    return;
  }
  atomicAdd(&counts[e], 1);
}

// One CTA: padded offsets of every expert (routed, then shared with T rows each) and the tile list.
__global__ void pf_scan_kernel(const int* __restrict__ counts, int E, int n_shared, int T, int* __restrict__ offsets,
                               int* __restrict__ tile_expert, int* __restrict__ tile_row0, int* __restrict__ ntiles) {
  if (threadIdx.x != 0) return;
  int off = 0, nt = 0;
  for (int e = 0; e < E + n_shared; ++e) {
    const int c = e < E ? counts[e] : T;
    offsets[e] = off;
    for (int r = 0; r < c; r += kPfTileM) {
      tile_expert[nt] = e;
      tile_row0[nt] = off + r;
      ++nt;
    }
    off += (c + kPfTileM - 1) / kPfTileM * kPfTileM;
  }
  offsets[E + n_shared] = off;
  ntiles[0] = nt;
  ntiles[1] = off;
}

// Every (token, slot) pair takes a row of its expert; shared experts take row t.  Which row a pair gets
// depends on the order of the atomics, the values computed for it do not.
__global__ void pf_scatter_kernel(const int32_t* __restrict__ ids, int T, int k, int E, int n_shared,
                                  const int* __restrict__ offsets, int* __restrict__ cursor, int* __restrict__ row_token,
                                  int* __restrict__ posmap) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int slots = k + n_shared;
  if (i >= T * slots) return;
  const int t = i / slots, j = i % slots;
  int pos = -1;
  if (j < k) {
    const int e = ids[t * k + j];
    if (e >= 0 && e < E) pos = offsets[e] + atomicAdd(&cursor[e], 1);
  } else {
    pos = offsets[E + (j - k)] + t;
  }
  posmap[i] = pos;
  if (pos >= 0) row_token[pos] = t;
}

// ---- step 2: gather x into expert order, bf16 -> fp16; padding rows are zero ----------------------------
__global__ void pf_gather_kernel(const uint16_t* __restrict__ x, int hidden, const int* __restrict__ row_token,
                                 const int* __restrict__ ntiles, __half* __restrict__ xs) {
  const int row = blockIdx.x;
  if (row >= ntiles[1]) return;
  const int t = row_token[row];
  __half2* dst = reinterpret_cast<__half2*>(xs + (size_t)row * hidden);
  if (t < 0) {
    for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) dst[i] = __floats2half2_rn(0.f, 0.f);
    return;
  }
  const uint32_t* src = reinterpret_cast<const uint32_t*>(x + (size_t)t * hidden);
  for (int i = threadIdx.x; i < hidden / 2; i += blockDim.x) {
    const uint32_t raw = src[i];
    dst[i] = __floats2half2_rn(__uint_as_float(raw << 16), __uint_as_float(raw & 0xffff0000u));
  }
}

// ---- steps 3 and 4: the grouped GEMM ------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait0() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct PfGemmParams {
  const slicemoe_expert* experts;  // routed
  const slicemoe_expert* shared;
  const uint8_t* expert_prec;      // per routed expert: 1 = both slices, 0 = MSB slice only
  const int* tile_expert;
  const int* tile_row0;
  const int* ntiles;
  const __half* a;                 // phase 1: gathered x [rows, hidden]; phase 2: h [rows, ldh]
  __half* h;                       // phase 1 output
  float* yrow;                     // phase 2 output [rows, hidden]
  unsigned* status;
  int E, hidden, inter, shared_inter, ldh;
};

// Two plane words of a thread for one pipeline step, the zero-point offsets of their two rows each,
// and (for the threads that publish them) one row's scale per quantisation group of the step.
struct PfBRegs {
  uint32_t mw[2], lw[2];
  __half2 off[2][2];  // [word][low-nibble row, high-nibble row]: 1024 + zero-point (or its top 4 bits)
  float sc[2];        // scale of B row (tid & 127), groups of this step
};

// PHASE 1: B rows 0-63 = gate rows [64 nt, 64 nt + 64), rows 64-127 = up rows of the same range; K = hidden.
// PHASE 2: B rows = down rows [128 nt, 128 nt + 128); K = the expert's intermediate width.
// The tensor cores contract x (or h) with the INTEGER q - zp, which fp16 holds exactly, one quantisation
// group at a time; at the end of each group the partial sums are scaled by the group's fp16 scale in fp32
// and added to the running result.  No weight is ever rounded.
template <int G, int PHASE>
__global__ void __launch_bounds__(kPfThreads, 1) pf_gemm_kernel(const PfGemmParams p) {
  constexpr int LG = G == 128 ? 7 : (G == 64 ? 6 : 5);
  constexpr int kStepsPerGroup = G / 16;                    // k16 MMA steps per quantisation group
  constexpr int kGroupsPerChunk = G >= kPfChunkK ? 1 : kPfChunkK / G;
  const int tile = blockIdx.x;
  if (tile >= p.ntiles[0]) return;
  const int e = p.tile_expert[tile], row0 = p.tile_row0[tile], nt = blockIdx.y;
  const bool is_shared = e >= p.E;
  const slicemoe_expert& ex = is_shared ? p.shared[e - p.E] : p.experts[e];
  const int inter = is_shared ? p.shared_inter : p.inter;
  bool prec = is_shared ? true : (p.expert_prec[e] != 0);
  if (prec && !(PHASE == 1 ? (ex.gate.lsb && ex.up.lsb) : ex.down.lsb != nullptr)) {
    // both slices asked of a matrix that has only one: run the MSB slice, tell the caller
    if (threadIdx.x == 0) atomicOr(p.status, (unsigned)SLICEMOE_STATUS_MISSING_LSB);
    prec = false;
  }
  const int K = PHASE == 1 ? p.hidden : inter;
  const int nout = PHASE == 1 ? inter / 64 : p.hidden / 128;  // n-tiles this expert has
  if (nt >= nout) return;
  const int lda = PHASE == 1 ? p.hidden : p.ldh;

  extern __shared__ __align__(16) uint8_t pf_smem[];
  __half(*As)[kPfTileM][kPfStride] = reinterpret_cast<__half(*)[kPfTileM][kPfStride]>(pf_smem);
  __half(*Bs)[kPfTileB][kPfStride] =
      reinterpret_cast<__half(*)[kPfTileB][kPfStride]>(pf_smem + 2 * sizeof(__half) * kPfTileM * kPfStride);
  float(*Ss)[2][kPfTileB] = reinterpret_cast<float(*)[2][kPfTileB]>(
      pf_smem + 2 * sizeof(__half) * (kPfTileM + kPfTileB) * kPfStride);  // [buffer][group of the step][B row]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = warp & 3, wn = warp >> 2;  // the warp's 32 token rows and 32 B rows (phase 1: 16 gate + 16 up)

  // ---- the thread's two plane words per step: which matrix, row block, position ----
  const uint32_t* msb[2];
  const uint32_t* lsb[2];
  const uint8_t* zpp[2];
  int brow[2], bk[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int ws = tid + kPfThreads * i;
    const int rbk = ws >> 7, idx = ws & 127, L = idx >> 2, w = idx & 3, g = L >> 2, c = L & 3;
    const slicemoe_mat& m = PHASE == 1 ? (rbk < 4 ? ex.gate : ex.up) : ex.down;
    const int rb = PHASE == 1 ? nt * 4 + (rbk & 3) : nt * 8 + rbk;
    msb[i] = reinterpret_cast<const uint32_t*>(m.msb) + (size_t)rb * (K >> 6) * 128 + idx;
    lsb[i] = prec ? reinterpret_cast<const uint32_t*>(m.lsb) + (size_t)rb * (K >> 6) * 128 + idx : msb[i];
    zpp[i] = m.zp + (size_t)rb * (K >> LG) * 16 + g;
    brow[i] = 16 * rbk + g;
    bk[i] = 16 * w + 4 * c;
  }
  // threads 0..127 publish the scale of B row tid for the first group of a step, 128..255 for the second
  const uint16_t* scp = nullptr;
  const int srow = tid & 127, sgrp = tid >> 7;
  if (sgrp < kGroupsPerChunk) {
    const int rbk = srow >> 4;
    const slicemoe_mat& m = PHASE == 1 ? (rbk < 4 ? ex.gate : ex.up) : ex.down;
    const int rb = PHASE == 1 ? nt * 4 + (rbk & 3) : nt * 8 + rbk;
    scp = m.scale + (size_t)rb * (K >> LG) * 16 + (srow & 15);
  }
  auto load_b = [&](PfBRegs& r, int kc) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      r.mw[i] = __ldg(msb[i] + (size_t)kc * 128);
      r.lw[i] = prec ? __ldg(lsb[i] + (size_t)kc * 128) : 0u;
      const int grp = (kc * kPfChunkK + bk[i]) >> LG;
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const int z = __ldg(zpp[i] + grp * 16 + 8 * hi);
        r.off[i][hi] = __half2half2(__int2half_rn(1024 + (prec ? z : (z >> 4))));
      }
    }
    if (scp) {
      const int grp = ((kc * kPfChunkK) >> LG) + sgrp;
      const float s = __half2float(__ushort_as_half(__ldg(scp + grp * 16)));
      r.sc[0] = prec ? s : 16.f * s;
    }
  };
  auto store_b = [&](const PfBRegs& r, int buf) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint32_t m0 = r.mw[i], l0 = r.lw[i];
      const uint32_t qlo = prec ? (((m0 & 0x0f0f0f0fu) << 4) | (l0 & 0x0f0f0f0fu)) : (m0 & 0x0f0f0f0fu);
      const uint32_t qhi = prec ? ((m0 & 0xf0f0f0f0u) | ((l0 >> 4) & 0x0f0f0f0fu)) : ((m0 >> 4) & 0x0f0f0f0fu);
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const uint32_t q = hi ? qhi : qlo;
        // bytes -> fp16 1024 + code, minus (1024 + zero-point): the integer q - zp, exact
        uint32_t h01 = __byte_perm(q, 0x64646464u, 0x4140), h23 = __byte_perm(q, 0x64646464u, 0x4342);
        __half2 w01 = __hsub2(*reinterpret_cast<__half2*>(&h01), r.off[i][hi]);
        __half2 w23 = __hsub2(*reinterpret_cast<__half2*>(&h23), r.off[i][hi]);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t*>(&w01);
        o.y = *reinterpret_cast<uint32_t*>(&w23);
        *reinterpret_cast<uint2*>(&Bs[buf][brow[i] + 8 * hi][bk[i]]) = o;
      }
    }
    if (scp) Ss[buf][sgrp][srow] = r.sc[0];
  };
  auto load_a = [&](int buf, int kc) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int ci = tid + kPfThreads * i, row = ci >> 3, seg = ci & 7;
      cp_async16(&As[buf][row][seg * 8], p.a + (size_t)(row0 + row) * lda + (size_t)kc * kPfChunkK + seg * 8);
    }
    cp_async_commit();
  };

  // B rows of the warp's four n8 tiles (tiles 2 jp, 2 jp + 1 are adjacent)
  int nrow[2];
#pragma unroll
  for (int jp = 0; jp < 2; ++jp) nrow[jp] = PHASE == 1 ? 64 * jp + 16 * wn : 32 * wn + 16 * jp;

  float acc[2][4][4], tot[2][4][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[i][j][q] = tot[i][j][q] = 0.f;

  const int nk = K / kPfChunkK;
  const int c2 = 2 * (lane & 3);
  PfBRegs breg;
  load_a(0, 0);
  load_b(breg, 0);
  store_b(breg, 0);
  cp_async_wait0();
  __syncthreads();
  for (int kc = 0; kc < nk; ++kc) {
    const int buf = kc & 1;
    const bool more = kc + 1 < nk;
    if (more) {
      load_a(buf ^ 1, kc + 1);
      load_b(breg, kc + 1);
    }
#pragma unroll
    for (int ks = 0; ks < kPfChunkK / 16; ++ks) {
      uint32_t af[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i)
        ldmatrix_x4(af[i], &As[buf][32 * wm + 16 * i + (lane & 15)][16 * ks + (lane >> 4) * 8]);
#pragma unroll
      for (int jp = 0; jp < 2; ++jp) {
        uint32_t bf[4];
        ldmatrix_x4(bf, &Bs[buf][nrow[jp] + (lane & 7) + ((lane >> 4) << 3)][16 * ks + ((lane >> 3) & 1) * 8]);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          mma_f16(acc[i][2 * jp], af[i], bf[0], bf[1]);
          mma_f16(acc[i][2 * jp + 1], af[i], bf[2], bf[3]);
        }
      }
      // end of a quantisation group: scale the group's sums, add them to the result, start over
      const int step = kc * (kPfChunkK / 16) + ks;
      if ((step + 1) % kStepsPerGroup == 0) {
        const int gi = kGroupsPerChunk == 1 ? 0 : (ks * 16) / G;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 s = *reinterpret_cast<const float2*>(&Ss[buf][gi][nrow[j >> 1] + 8 * (j & 1) + c2]);
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            tot[i][j][0] = fmaf(s.x, acc[i][j][0], tot[i][j][0]);
            tot[i][j][1] = fmaf(s.y, acc[i][j][1], tot[i][j][1]);
            tot[i][j][2] = fmaf(s.x, acc[i][j][2], tot[i][j][2]);
            tot[i][j][3] = fmaf(s.y, acc[i][j][3], tot[i][j][3]);
            acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;
          }
        }
      }
    }
    if (more) {
      store_b(breg, buf ^ 1);
      cp_async_wait0();
    }
    __syncthreads();
  }

  // ---- epilogue ----
  const int g = lane >> 2;
  if (PHASE == 1) {
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float g0 = tot[i][j][2 * hf], g1 = tot[i][j][2 * hf + 1];
          const float u0 = tot[i][j + 2][2 * hf], u1 = tot[i][j + 2][2 * hf + 1];
          const float h0 = g0 / (1.f + __expf(-g0)) * u0, h1 = g1 / (1.f + __expf(-g1)) * u1;
          const int row = row0 + 32 * wm + 16 * i + g + 8 * hf;
          const int col = 64 * nt + 16 * wn + 8 * j + c2;
          *reinterpret_cast<__half2*>(p.h + (size_t)row * p.ldh + col) = __floats2half2_rn(h0, h1);
        }
  } else {
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int row = row0 + 32 * wm + 16 * i + g + 8 * hf;
          const int col = 128 * nt + 32 * wn + 8 * j + c2;
          *reinterpret_cast<float2*>(p.yrow + (size_t)row * p.hidden + col) =
              make_float2(tot[i][j][2 * hf], tot[i][j][2 * hf + 1]);
        }
  }
}


// ---- step 5: weighted combine in list order ---------------------------------------------------------------
__global__ void pf_gate_kernel(const uint16_t* __restrict__ x, const float* __restrict__ gate_vec, int T, int hidden,
                               float* __restrict__ gate) {
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= T) return;
  float dot = 0.f;
  for (int i = lane; i < hidden; i += 32)
    dot = fmaf(gate_vec[i], __uint_as_float((uint32_t)x[(size_t)t * hidden + i] << 16), dot);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
  if (lane == 0) gate[t] = 1.f / (1.f + expf(-dot));
}

__global__ void pf_combine_kernel(const float* __restrict__ yrow, const int* __restrict__ posmap,
                                  const float* __restrict__ weights, const float* __restrict__ gate, int T, int k,
                                  int n_shared, int hidden, float* __restrict__ y) {
  const int t = blockIdx.x;
  const int slots = k + n_shared;
  for (int col = threadIdx.x * 4; col < hidden; col += blockDim.x * 4) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j = 0; j < slots; ++j) {
      const int pos = posmap[t * slots + j];
      if (pos < 0) continue;
      const float w = j < k ? weights[t * k + j] : (gate ? gate[t] : 1.f);
      const float4 v = *reinterpret_cast<const float4*>(yrow + (size_t)pos * hidden + col);
      a.x = fmaf(w, v.x, a.x);
      a.y = fmaf(w, v.y, a.y);
      a.z = fmaf(w, v.z, a.z);
      a.w = fmaf(w, v.w, a.w);
    }
    *reinterpret_cast<float4*>(y + (size_t)t * hidden + col) = a;
  }
}

// A and B tiles double-buffered (73,728 bytes) plus the scales of the step's groups
constexpr int kPfSmemBytes = 2 * (int)sizeof(__half) * (kPfTileM + kPfTileB) * kPfStride + 2 * 2 * kPfTileB * (int)sizeof(float);

template <int G>
static int pf_launch_gemms(const PfGemmParams& p, int max_tiles, int inter_max, cudaStream_t st) {
  static bool attr_set[64];
  int dev = 0;
  SM_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SLICEMOE_E_UNSUPPORTED;
  if (!attr_set[dev]) {
    SM_CUDA_TRY(cudaFuncSetAttribute(pf_gemm_kernel<G, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes));
    SM_CUDA_TRY(cudaFuncSetAttribute(pf_gemm_kernel<G, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes));
    attr_set[dev] = true;
  }
  pf_gemm_kernel<G, 1><<<dim3(max_tiles, inter_max / 64), kPfThreads, kPfSmemBytes, st>>>(p);
  SM_LAUNCH_CHECK();
  PfGemmParams p2 = p;  // the second GEMM contracts h
  p2.a = p.h;
  pf_gemm_kernel<G, 2><<<dim3(max_tiles, p.hidden / 128), kPfThreads, kPfSmemBytes, st>>>(p2);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}

static int pf_check(const slicemoe_shape* s, int T) {
  if (!s || T <= 0) return SLICEMOE_E_INVALID_ARG;
  if (s->b_high != 8 || s->b_low != 4) return SLICEMOE_E_UNSUPPORTED;
  if (!valid_group(s->group)) return SLICEMOE_E_UNSUPPORTED;
  if (s->hidden <= 0 || s->inter <= 0 || s->n_experts <= 0 || s->top_k < 1) return SLICEMOE_E_INVALID_ARG;
  if (s->top_k > s->n_experts || s->top_k > SLICEMOE_MAX_TOP_K) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared < 0 || s->n_shared > SLICEMOE_MAX_SHARED) return SLICEMOE_E_INVALID_ARG;
  if ((s->hidden % 128) || (s->inter % 128)) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && (s->shared_inter <= 0 || (s->shared_inter % 128))) return SLICEMOE_E_INVALID_ARG;
  if ((long long)T * (s->top_k + s->n_shared) > (1ll << 28)) return SLICEMOE_E_UNSUPPORTED;
  return SLICEMOE_OK;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" size_t slicemoe_prefill_workspace_bytes(const slicemoe_shape* s, int T) {
  if (pf_check(s, T) != SLICEMOE_OK) return 0;
  return pf_layout(T, s->n_experts, s->top_k, s->n_shared, s->hidden, s->inter, s->n_shared ? s->shared_inter : 0).total;
}

extern "C" int slicemoe_prefill_layer(const slicemoe_shape* s, const slicemoe_expert* experts,
                                      const slicemoe_expert* shared, const float* shared_gate_vec, const void* x, int T,
                                      const int32_t* ids, const float* weights, const uint8_t* expert_prec, float* y,
                                      void* workspace, size_t workspace_bytes, int* status_out_device, void* stream) {
  int rc = pf_check(s, T);
  if (rc != SLICEMOE_OK) return rc;
  if (!experts || !x || !ids || !weights || !expert_prec || !y || !workspace || !status_out_device)
    return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && !shared) return SLICEMOE_E_INVALID_ARG;
  if (s->n_shared > 0 && s->shared_sigmoid_gate && !shared_gate_vec) return SLICEMOE_E_INVALID_ARG;
  const int nsh = s->n_shared, E = s->n_experts, k = s->top_k;
  const int shared_inter = nsh ? s->shared_inter : 0;
  const PfLayout L = pf_layout(T, E, k, nsh, s->hidden, s->inter, shared_inter);
  if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255)) return SLICEMOE_E_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 3) || (reinterpret_cast<uintptr_t>(y) & 15)) return SLICEMOE_E_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  int* counts = reinterpret_cast<int*>(ws + L.counts);
  int* cursor = reinterpret_cast<int*>(ws + L.cursor);
  int* offsets = reinterpret_cast<int*>(ws + L.offsets);
  int* tile_expert = reinterpret_cast<int*>(ws + L.tile_expert);
  int* tile_row0 = reinterpret_cast<int*>(ws + L.tile_row0);
  int* ntiles = reinterpret_cast<int*>(ws + L.ntiles);
  int* row_token = reinterpret_cast<int*>(ws + L.row_token);
  int* posmap = reinterpret_cast<int*>(ws + L.posmap);
  float* gate = reinterpret_cast<float*>(ws + L.gate);
  __half* xs = reinterpret_cast<__half*>(ws + L.xs);
  __half* h = reinterpret_cast<__half*>(ws + L.h);
  float* yrow = reinterpret_cast<float*>(ws + L.yrow);

  // counters start at zero, unused rows are marked -1
  SM_CUDA_TRY(cudaMemsetAsync(ws + L.counts, 0, L.offsets - L.counts, st));
  SM_CUDA_TRY(cudaMemsetAsync(row_token, 0xff, sizeof(int) * (size_t)L.rmax, st));
  SM_CUDA_TRY(cudaMemsetAsync(status_out_device, 0, sizeof(int), st));
  const int npairs = T * k;
  pf_count_kernel<<<(npairs + 255) / 256, 256, 0, st>>>(ids, npairs, E, counts, reinterpret_cast<unsigned*>(status_out_device));
  SM_LAUNCH_CHECK();
  pf_scan_kernel<<<1, 32, 0, st>>>(counts, E, nsh, T, offsets, tile_expert, tile_row0, ntiles);
  SM_LAUNCH_CHECK();
  const int nslots = T * (k + nsh);
  pf_scatter_kernel<<<(nslots + 255) / 256, 256, 0, st>>>(ids, T, k, E, nsh, offsets, cursor, row_token, posmap);
  SM_LAUNCH_CHECK();
  pf_gather_kernel<<<L.rmax, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), s->hidden, row_token, ntiles, xs);
  SM_LAUNCH_CHECK();
  const bool gated = nsh > 0 && s->shared_sigmoid_gate;
  if (gated) {
    pf_gate_kernel<<<(T + 7) / 8, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), shared_gate_vec, T, s->hidden, gate);
    SM_LAUNCH_CHECK();
  }
  PfGemmParams p;
  p.experts = experts;
  p.shared = shared;
  p.expert_prec = expert_prec;
  p.tile_expert = tile_expert;
  p.tile_row0 = tile_row0;
  p.ntiles = ntiles;
  p.a = xs;
  p.h = h;
  p.yrow = yrow;
  p.status = reinterpret_cast<unsigned*>(status_out_device);
  p.E = E;
  p.hidden = s->hidden;
  p.inter = s->inter;
  p.shared_inter = shared_inter;
  p.ldh = s->inter > shared_inter ? s->inter : shared_inter;
  const int inter_max = p.ldh;
  if (s->group == 128) {
    rc = pf_launch_gemms<128>(p, L.max_tiles, inter_max, st);
  } else if (s->group == 64) {
    rc = pf_launch_gemms<64>(p, L.max_tiles, inter_max, st);
  } else {
    rc = pf_launch_gemms<32>(p, L.max_tiles, inter_max, st);
  }
  if (rc != SLICEMOE_OK) return rc;
  pf_combine_kernel<<<T, 256, 0, st>>>(yrow, posmap, weights, gated ? gate : nullptr, T, k, nsh, s->hidden, y);
  SM_LAUNCH_CHECK();
  return SLICEMOE_OK;
}
