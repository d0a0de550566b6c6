// CUDA-core (fp32 FMA) chunk step: the path for fp32 tensors and for head
// dimensions the tensor-core kernel does not cover.
//
//   attn_simt_kernel   Sec. 3.1 chunk forward: a 64-row query tile walks the
//                      visible keys [cache ; chunk prefix] in 64-key tiles with
//                      an online softmax; writes out and lse.
//   score_simt_kernel  H2O eviction score (Sec. 3.1, Sec. 4 "Common setup"):
//                      key-stationary second pass.  A block owns 64 keys of one
//                      KV head, revisits the trailing `window` query rows of
//                      the G query heads of its group, forms p = exp(s - lse)
//                      with the final normaliser and sums columns.  Every key
//                      is owned by exactly one block: no atomics, bit-stable.
//
// Thread layout (both): 256 threads as 16 (ty) x 16 (tx); a thread owns score
// rows 4*ty .. 4*ty+3 and key columns tx, tx+16, tx+32, tx+48 of the 64 x 64
// logit tile.  Shared-memory rows are padded by 4 floats so 128-bit reads of
// the two ty rows of a warp fall in different banks.
#pragma once

#include "common.cuh"

namespace reform {

constexpr int kBM = 64;
constexpr int kBN = 64;
constexpr int kSimtThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct SimtSmem {
  static constexpr int LD = D + 4;
  static constexpr int LDP = kBN + 4;
  static constexpr size_t attn_bytes = sizeof(float) * ((size_t)kBM * LD + 2 * (size_t)kBN * LD + (size_t)kBM * LDP);
  static constexpr size_t score_bytes = sizeof(float) * ((size_t)kBM * LD + (size_t)kBN * LD + 16 * kBN + kBM);
};

// rows [row0, row0 + 64) of a [n_rows, D] matrix -> smem tile (fp32), zero
// beyond n_rows.
template <typename T, int D>
__device__ __forceinline__ void load_tile(float* dst, const T* src, long long row0, long long n_rows) {
  constexpr int LD = D + 4;
  constexpr int V = D / 4;
  for (int i = threadIdx.x; i < 64 * V; i += kSimtThreads) {
    int r = i / V, c = i % V;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < n_rows) {
      const T* p = src + (row0 + r) * D + 4 * c;
      v = make_float4(to_float(p[0]), to_float(p[1]), to_float(p[2]), to_float(p[3]));
    }
    *reinterpret_cast<float4*>(dst + r * LD + 4 * c) = v;
  }
}

// acc[r][c] = <Q row 4*ty+r, K row tx+16c>
template <int D>
__device__ __forceinline__ void logit_tile(const float* Qs, const float* Ks, int ty, int tx,
                                           float (&acc)[4][4]) {
  constexpr int LD = D + 4;
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 4
  for (int e = 0; e < D; e += 4) {
    float4 q[4], k[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) q[r] = *reinterpret_cast<const float4*>(Qs + (4 * ty + r) * LD + e);
#pragma unroll
    for (int c = 0; c < 4; ++c) k[c] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * c) * LD + e);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        acc[r][c] = fmaf(q[r].x, k[c].x, acc[r][c]);
        acc[r][c] = fmaf(q[r].y, k[c].y, acc[r][c]);
        acc[r][c] = fmaf(q[r].z, k[c].z, acc[r][c]);
        acc[r][c] = fmaf(q[r].w, k[c].w, acc[r][c]);
      }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
attn_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                 T* __restrict__ out, float* __restrict__ lse, int Hq, int Hkv, int Lc, int n_cache,
                 int cap, float scale_log2) {
  extern __shared__ float smem[];
  constexpr int LD = D + 4, LDP = kBN + 4, OC = D / 64;  // OC float4 output chunks per thread
  float* Qs = smem;
  float* Ks = Qs + kBM * LD;
  float* Vs = Ks + kBN * LD;
  float* Ps = Vs + kBN * LD;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  // longest tiles first: the last query tile sees the most keys
  const int n_qt = (Lc + kBM - 1) / kBM;
  const int qt = n_qt - 1 - blockIdx.x;
  const int h = blockIdx.y % Hq, b = blockIdx.y / Hq;
  const int g = h / (Hq / Hkv);
  const int n = n_cache + Lc;
  const T* qp = q + ((long long)b * Hq + h) * (long long)Lc * D;
  const T* kp = k + ((long long)b * Hkv + g) * (long long)cap * D;
  const T* vp = v + ((long long)b * Hkv + g) * (long long)cap * D;
  const int row0 = qt * kBM;
  load_tile<T, D>(Qs, qp, row0, Lc);
  float m[4], l[4], o[4][OC][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    m[r] = -INFINITY;
    l[r] = 0.f;
#pragma unroll
    for (int c = 0; c < OC; ++c) o[r][c][0] = o[r][c][1] = o[r][c][2] = o[r][c][3] = 0.f;
  }
  int last_row = row0 + kBM - 1;
  if (last_row > Lc - 1) last_row = Lc - 1;
  const int n_vis = n_cache + last_row + 1;  // keys visible to the tile's last row
  const int n_kt = (n_vis + kBN - 1) / kBN;
  for (int kt = 0; kt < n_kt; ++kt) {
    __syncthreads();  // previous tile's Ks/Vs/Ps fully consumed
    load_tile<T, D>(Ks, kp, (long long)kt * kBN, n);
    load_tile<T, D>(Vs, vp, (long long)kt * kBN, n);
    __syncthreads();
    float s[4][4];
    logit_tile<D>(Qs, Ks, ty, tx, s);
    const bool need_mask = (kt + 1) * kBN > n_cache + row0 + 1;  // tile reaches past some row's limit
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int lim = n_cache + row0 + 4 * ty + r;  // last visible key of this row
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float x = s[r][c] * scale_log2;
        int j = kt * kBN + tx + 16 * c;
        if (need_mask && (j > lim || j >= n)) x = -INFINITY;
        s[r][c] = x;
        mx = fmaxf(mx, x);
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m[r], mx);
      const float corr = exp2f(m[r] - m_new);  // m_new is finite from the first tile on
      float ps = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float p = exp2f(s[r][c] - m_new);
        ps += p;
        Ps[(4 * ty + r) * LDP + tx + 16 * c] = p;
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l[r] = l[r] * corr + ps;
      m[r] = m_new;
#pragma unroll
      for (int c = 0; c < OC; ++c) {
        o[r][c][0] *= corr; o[r][c][1] *= corr; o[r][c][2] *= corr; o[r][c][3] *= corr;
      }
    }
    __syncthreads();
    // O += P V : rows 4*ty+r, columns 4*(tx + 16*c) .. +3
#pragma unroll 2
    for (int j = 0; j < kBN; j += 4) {
      float4 p4[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) p4[r] = *reinterpret_cast<const float4*>(Ps + (4 * ty + r) * LDP + j);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
        for (int c = 0; c < OC; ++c) {
          float4 vv = *reinterpret_cast<const float4*>(Vs + (j + jj) * LD + 4 * (tx + 16 * c));
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            float p = jj == 0 ? p4[r].x : jj == 1 ? p4[r].y : jj == 2 ? p4[r].z : p4[r].w;
            o[r][c][0] = fmaf(p, vv.x, o[r][c][0]);
            o[r][c][1] = fmaf(p, vv.y, o[r][c][1]);
            o[r][c][2] = fmaf(p, vv.z, o[r][c][2]);
            o[r][c][3] = fmaf(p, vv.w, o[r][c][3]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    int i = row0 + 4 * ty + r;
    if (i >= Lc) continue;
    float inv = 1.0f / l[r];
    T* op = out + (((long long)b * Hq + h) * Lc + i) * D;
#pragma unroll
    for (int c = 0; c < OC; ++c) {
      int col = 4 * (tx + 16 * c);
      op[col + 0] = from_float<T>(o[r][c][0] * inv);
      op[col + 1] = from_float<T>(o[r][c][1] * inv);
      op[col + 2] = from_float<T>(o[r][c][2] * inv);
      op[col + 3] = from_float<T>(o[r][c][3] * inv);
    }
    if (tx == 0) lse[((long long)b * Hq + h) * Lc + i] = (m[r] + log2f(l[r])) * kLn2;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads)
score_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const float* __restrict__ lse,
                  float* __restrict__ score, int Hq, int Hkv, int Lc, int n_cache, int cap,
                  int window, float scale_log2, int accumulate) {
  extern __shared__ float smem[];
  constexpr int LD = D + 4;
  float* Qs = smem;
  float* Ks = Qs + kBM * LD;
  float* red = Ks + kBN * LD;   // [16][64] column partials
  float* lse2 = red + 16 * kBN; // [64] row normalisers (log2 units)
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int g = blockIdx.y % Hkv, b = blockIdx.y / Hkv;
  const int G = Hq / Hkv;
  const int n = n_cache + Lc;
  const int j0 = blockIdx.x * kBN;
  const T* kp = k + ((long long)b * Hkv + g) * (long long)cap * D;
  load_tile<T, D>(Ks, kp, j0, n);
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  const int i_begin = Lc - window;
  for (int hh = 0; hh < G; ++hh) {
    const int h = g * G + hh;
    const T* qp = q + ((long long)b * Hq + h) * (long long)Lc * D;
    const float* lp = lse + ((long long)b * Hq + h) * Lc;
    for (int i0 = i_begin; i0 < Lc; i0 += kBM) {
      int i_last = i0 + kBM - 1;
      if (i_last > Lc - 1) i_last = Lc - 1;
      if (j0 > n_cache + i_last) continue;  // no row of this tile sees any key of the block
      __syncthreads();
      load_tile<T, D>(Qs, qp, i0, Lc);
      if (threadIdx.x < kBM) {
        int i = i0 + threadIdx.x;
        lse2[threadIdx.x] = (i < Lc) ? lp[i] * kLog2e : INFINITY;  // rows past the chunk add 0
      }
      __syncthreads();
      float s[4][4];
      logit_tile<D>(Qs, Ks, ty, tx, s);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = i0 + 4 * ty + r;
        const float lr = lse2[4 * ty + r];
        const int lim = n_cache + i;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int j = j0 + tx + 16 * c;
          float p = exp2f(s[r][c] * scale_log2 - lr);
          if (j <= lim && j < n) col[c] += p;
        }
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < 4; ++c) red[ty * kBN + tx + 16 * c] = col[c];
  __syncthreads();
  if (threadIdx.x < kBN) {
    int j = j0 + threadIdx.x;
    if (j < n) {
      float sum = 0.f;
#pragma unroll
      for (int y = 0; y < 16; ++y) sum += red[y * kBN + threadIdx.x];
      long long o = ((long long)b * Hkv + g) * cap + j;
      float carry = (accumulate && j < n_cache) ? score[o] : 0.f;
      score[o] = carry + sum;
    }
  }
}

template <typename T, int D>
inline int launch_chunk_simt_td(const reform_chunk_params* p, float* lse, float scale, cudaStream_t st) {
  const int n_qt = (p->Lc + kBM - 1) / kBM;
  const float scale_log2 = scale * kLog2e;
  size_t smem = SimtSmem<D>::attn_bytes;
  cudaFuncSetAttribute(attn_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  dim3 grid(n_qt, p->B * p->Hq);
  attn_simt_kernel<T, D><<<grid, kSimtThreads, smem, st>>>(
      (const T*)p->q, (const T*)p->k, (const T*)p->v, (T*)p->out, lse, p->Hq, p->Hkv, p->Lc,
      p->n_cache, p->cap, scale_log2);
  count_launch();
  int rc = check_launch();
  if (rc != REFORM_OK || (p->flags & REFORM_NO_SCORE)) return rc;
  size_t smem2 = SimtSmem<D>::score_bytes;
  cudaFuncSetAttribute(score_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
  dim3 grid2((p->n_cache + p->Lc + kBN - 1) / kBN, p->B * p->Hkv);
  score_simt_kernel<T, D><<<grid2, kSimtThreads, smem2, st>>>(
      (const T*)p->q, (const T*)p->k, lse, p->score, p->Hq, p->Hkv, p->Lc, p->n_cache, p->cap,
      p->score_window, scale_log2, (p->flags & REFORM_SCORE_ACCUMULATE) ? 1 : 0);
  count_launch();
  return check_launch();
}

inline int launch_chunk_simt(const reform_chunk_params* p, float* lse, float scale, cudaStream_t st) {
#define REFORM_SIMT_CASE(T, D) return launch_chunk_simt_td<T, D>(p, lse, scale, st);
  if (p->dtype == REFORM_F32) {
    if (p->d == 64) REFORM_SIMT_CASE(float, 64)
    if (p->d == 128) REFORM_SIMT_CASE(float, 128)
  } else {
    if (p->d == 64) REFORM_SIMT_CASE(__nv_bfloat16, 64)
    if (p->d == 128) REFORM_SIMT_CASE(__nv_bfloat16, 128)
  }
#undef REFORM_SIMT_CASE
  return REFORM_ERR_UNSUPPORTED;
}

}  // namespace reform
