// Similarity scan of the gather phase (Sec. 3.3): ts[t] = max_q scale *
// <queries[q], bank[t]>.  The bank is streamed from HBM exactly once.
//
// bf16 path: the nq dot products per bank row are a skinny contraction
// (16 tokens x E) x (E x 8 queries) done with warp-level bf16 MMAs so the
// arithmetic (nq flop per byte) never becomes the limit; bank rows go
// global -> registers directly as 128-bit loads.  A dot product does not
// depend on the order of its terms, so each thread hands the MMA the 8
// consecutive elements it loaded as if they were the k-slots its fragment
// wants, and the query fragment is read with the same permutation: no shared
// memory staging and no transposition of the streamed operand.
//
// Generic path (fp32 banks, odd shapes): one warp per bank row, fp32 FMAs.
#pragma once

#include "common.cuh"

namespace reform {

// ------------------------------------------------------------------ generic
template <typename T>
__global__ void __launch_bounds__(256)
scan_simt_kernel(const T* __restrict__ bank, const T* __restrict__ queries, float* __restrict__ ts,
                 int B, long long N, long long N_cap, int E, int nq, float scale) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long it = warp; it < (long long)B * N; it += n_warps) {
    int b = (int)(it / N);
    long long t = it % N;
    const T* row = bank + ((long long)b * N_cap + t) * E;
    const T* qb = queries + (long long)b * nq * E;
    float best = -INFINITY;
    for (int q0 = 0; q0 < nq; q0 += 8) {
      float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
      for (int e = lane; e < E; e += 32) {
        float x = to_float(row[e]);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (q0 + j < nq) acc[j] = fmaf(x, to_float(qb[(long long)(q0 + j) * E + e]), acc[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float s = warp_sum(acc[j]) * scale;
        if (q0 + j < nq) best = fmaxf(best, s);
      }
    }
    if (lane == 0) ts[(long long)b * N + t] = best;
  }
}

// --------------------------------------------------------------- bf16 MMA
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Queries sit in shared memory as [nq_pad][E] bf16 with rows rotated by 64 B
// per query (conflict-free 128-bit reads: a quarter-warp covers 2 queries x 4
// neighbouring chunks).
// NT = number of 8-query tiles (nq_pad = 8 * NT).  One warp owns 16 tokens.
template <int NT>
__global__ void __launch_bounds__(256)
scan_mma_kernel(const __nv_bfloat16* __restrict__ bank, const __nv_bfloat16* __restrict__ queries,
                float* __restrict__ ts, long long N, long long N_cap, int E, int nq, float scale,
                long long tiles_per_seq) {
  extern __shared__ uint4 qs[];  // [8*NT][E/8] 16-byte chunks, chunk c of query q stored at (c + 4q) % (E/8)
  const int lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int chunks = E >> 3;
  const int b = blockIdx.y;
  const __nv_bfloat16* qb = queries + (long long)b * nq * E;
  for (int i = threadIdx.x; i < 8 * NT * chunks; i += blockDim.x) {
    int q = i / chunks, c = i % chunks;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (q < nq) v = *reinterpret_cast<const uint4*>(qb + (long long)q * E + 8 * c);
    qs[q * chunks + (c + 4 * q) % chunks] = v;
  }
  __syncthreads();
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const __nv_bfloat16* bb = bank + (long long)b * N_cap * E;
  for (long long tile = warp; tile < tiles_per_seq; tile += n_warps) {
    const long long tok0 = tile * 16;
    // rows g and g+8 of the tile; clamp so the loads stay in range (results of
    // clamped rows are discarded)
    long long r0 = tok0 + g, r1 = tok0 + g + 8;
    const uint4* p0 = reinterpret_cast<const uint4*>(bb + (r0 < N ? r0 : N - 1) * E) + t;
    const uint4* p1 = reinterpret_cast<const uint4*>(bb + (r1 < N ? r1 : N - 1) * E) + t;
    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
    // each step consumes 32 elements (4 chunks) of both rows; 4 steps in flight
    for (int c0 = 0; c0 < chunks; c0 += 16) {
      uint4 a0[4], a1[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int c = c0 + 4 * u;
        if (c < chunks) {
          a0[u] = __ldcs(p0 + c);
          a1[u] = __ldcs(p1 + c);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int c = c0 + 4 * u;
        if (c < chunks) {
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            int q = 8 * n + g;
            uint4 bq = qs[q * chunks + (c + t + 4 * q) % chunks];
            mma_bf16_16816(acc[n], a0[u].x, a1[u].x, a0[u].y, a1[u].y, bq.x, bq.y);
            mma_bf16_16816(acc[n], a0[u].z, a1[u].z, a0[u].w, a1[u].w, bq.z, bq.w);
          }
        }
      }
    }
    // acc[n][0..1]: row g, queries 8n+2t, 8n+2t+1;  acc[n][2..3]: row g+8
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      int q = 8 * n + 2 * t;
      if (q < nq) { m0 = fmaxf(m0, acc[n][0] * scale); m1 = fmaxf(m1, acc[n][2] * scale); }
      if (q + 1 < nq) { m0 = fmaxf(m0, acc[n][1] * scale); m1 = fmaxf(m1, acc[n][3] * scale); }
    }
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
    if (t == 0) {
      if (r0 < N) ts[(long long)b * N + r0] = m0;
      if (r1 < N) ts[(long long)b * N + r1] = m1;
    }
  }
}

template <int NT>
inline void launch_scan_mma_nt(const void* bank, const void* queries, float* ts, int B, long long N,
                               long long N_cap, int E, int nq, float scale, cudaStream_t st) {
  long long tiles = (N + 15) / 16;
  size_t smem = (size_t)8 * NT * E * 2;
  cudaFuncSetAttribute(scan_mma_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  long long blocks = (tiles + 7) / 8;
  long long cap = (long long)num_sms() * (NT <= 2 ? 8 : (NT <= 4 ? 3 : 1));
  dim3 grid((unsigned)(blocks < cap ? blocks : cap), B);
  scan_mma_kernel<NT><<<grid, 256, smem, st>>>((const __nv_bfloat16*)bank,
                                               (const __nv_bfloat16*)queries, ts, N, N_cap, E, nq,
                                               scale, tiles);
}

inline int launch_scan(int dtype, const void* bank, const void* queries, float* ts, int B,
                       long long N, long long N_cap, int E, int nq, float scale, cudaStream_t st) {
  if ((long long)B * N == 0) return REFORM_OK;
  if (dtype == REFORM_BF16 && E % 32 == 0 && nq <= 64 && E <= 1024) {
    int nt = (nq + 7) / 8;
    if (nt == 1) launch_scan_mma_nt<1>(bank, queries, ts, B, N, N_cap, E, nq, scale, st);
    else if (nt == 2) launch_scan_mma_nt<2>(bank, queries, ts, B, N, N_cap, E, nq, scale, st);
    else if (nt <= 4) launch_scan_mma_nt<4>(bank, queries, ts, B, N, N_cap, E, nq, scale, st);
    else launch_scan_mma_nt<8>(bank, queries, ts, B, N, N_cap, E, nq, scale, st);
  } else {
    long long blocks = ((long long)B * N + 7) / 8;
    long long cap = (long long)num_sms() * 16;
    int grid = (int)(blocks < cap ? blocks : cap);
    if (dtype == REFORM_BF16)
      scan_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
          (const __nv_bfloat16*)bank, (const __nv_bfloat16*)queries, ts, B, N, N_cap, E, nq, scale);
    else
      scan_simt_kernel<float><<<grid, 256, 0, st>>>((const float*)bank, (const float*)queries, ts, B,
                                                    N, N_cap, E, nq, scale);
  }
  count_launch();
  return check_launch();
}

}  // namespace reform
