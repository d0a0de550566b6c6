// Decode-shaped chunk step (bf16, d = 128, Lc * G <= 16): the step that follows
// the on-demand recomputation (Sec. 3.3) -- one or a few new tokens attending
// over the recomputed cache.  With so few query rows the operation is a read
// of K and V, so it is split along the keys: a warp owns 128 keys of one KV
// head, packs the Lc * G query rows of the group into one 16-row MMA tile,
// streams its K and V rows global -> registers with 128-bit loads and keeps a
// running (max, sum, O) for its keys; a second small kernel merges the
// per-warp partials.  No shared memory: the k index of Q K^T and the column
// order of O are permuted so that what a thread loads contiguously is exactly
// what its mma.sync fragments need (a dot product does not care about the
// order of its terms, and the output columns are un-permuted when stored).
#pragma once

#include "common.cuh"
#include "chunk_simt.cuh"
#include "retrieve.cuh"  // mma_bf16_16816

namespace reform {

constexpr int kDecKeysPerWarp = 128;
constexpr int kDecWarps = 4;
constexpr int kDecMaxRows = 16;

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// partial layout: part_o [splits][BH][R][128] fp32 ; part_ml [splits][BH][R][2] fp32 (max in log2 units, sum)
__global__ void __launch_bounds__(32 * kDecWarps)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, float* __restrict__ part_o,
                    float* __restrict__ part_ml, int Hq, int Hkv, int Lc, int n_cache, int cap,
                    float scale_log2, int n_splits) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int split = blockIdx.x * kDecWarps + warp;
  if (split >= n_splits) return;
  const int bh = blockIdx.y, b = bh / Hkv, kvh = bh % Hkv;
  const int G = Hq / Hkv, R = Lc * G, n = n_cache + Lc;
  const int BH = gridDim.y;
  const __nv_bfloat16* kp = k + ((long long)bh * cap) * 128;
  const __nv_bfloat16* vp = v + ((long long)bh * cap) * 128;

  // Q fragments: rows g and g + 8 of the packed tile (row r = chunk row r / G, head r % G of the group)
  uint4 qa[4], qb[4];
  {
    const int r0 = g, r1 = g + 8;
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) {
      qa[kb] = make_uint4(0, 0, 0, 0);
      qb[kb] = make_uint4(0, 0, 0, 0);
      if (r0 < R)
        qa[kb] = *reinterpret_cast<const uint4*>(q + (((long long)b * Hq + kvh * G + r0 % G) * Lc + r0 / G) * 128 + 32 * kb + 8 * t);
      if (r1 < R)
        qb[kb] = *reinterpret_cast<const uint4*>(q + (((long long)b * Hq + kvh * G + r1 % G) * Lc + r1 / G) * 128 + 32 * kb + 8 * t);
    }
  }
  const int lim0 = n_cache + g / G, lim1 = n_cache + (g + 8) / G;  // last visible key of rows g, g + 8
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

  for (int blk = 0; blk < kDecKeysPerWarp / 64; ++blk) {
    const int kbase = split * kDecKeysPerWarp + 64 * blk;
    if (kbase >= n) break;
    // S = Q K^T for 64 keys: 8 n-tiles of 8 keys
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
      int key = kbase + 8 * nt + g;
      if (key > n - 1) key = n - 1;  // clamped rows are masked below
      const uint4* kr = reinterpret_cast<const uint4*>(kp + (long long)key * 128) + t;
      uint4 kk[4];
#pragma unroll
      for (int kb = 0; kb < 4; ++kb) kk[kb] = __ldg(kr + 4 * kb);
#pragma unroll
      for (int kb = 0; kb < 4; ++kb) {
        mma_bf16_16816(s[nt], qa[kb].x, qb[kb].x, qa[kb].y, qb[kb].y, kk[kb].x, kk[kb].y);
        mma_bf16_16816(s[nt], qa[kb].z, qb[kb].z, qa[kb].w, qb[kb].w, kk[kb].z, kk[kb].w);
      }
    }
    // mask, block max per row (rows g and g + 8), quad reduce
    float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int key = kbase + 8 * nt + 2 * t + c;
        if (key > lim0 || key >= n) s[nt][c] = -INFINITY;
        if (key > lim1 || key >= n) s[nt][2 + c] = -INFINITY;
        bm0 = fmaxf(bm0, s[nt][c]);
        bm1 = fmaxf(bm1, s[nt][2 + c]);
      }
    }
    bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1));
    bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
    bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1));
    bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
    const float mn0 = fmaxf(m0, bm0 * scale_log2), mn1 = fmaxf(m1, bm1 * scale_log2);
    const float a0 = (mn0 == -INFINITY) ? 1.f : exp2f(m0 - mn0);  // nothing visible yet: keep zeros
    const float a1 = (mn1 == -INFINITY) ? 1.f : exp2f(m1 - mn1);
    const float sub0 = (mn0 == -INFINITY) ? 0.f : mn0, sub1 = (mn1 == -INFINITY) ? 0.f : mn1;
    m0 = mn0;
    m1 = mn1;
    float ps0 = 0.f, ps1 = 0.f;
    uint32_t pa[8][2];  // per n-tile: packed P of row g, of row g + 8
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p00 = exp2f(fmaf(s[nt][0], scale_log2, -sub0)), p01 = exp2f(fmaf(s[nt][1], scale_log2, -sub0));
      const float p10 = exp2f(fmaf(s[nt][2], scale_log2, -sub1)), p11 = exp2f(fmaf(s[nt][3], scale_log2, -sub1));
      ps0 += p00 + p01;
      ps1 += p10 + p11;
      pa[nt][0] = pack2_bf16(p00, p01);
      pa[nt][1] = pack2_bf16(p10, p11);
    }
    l0 = l0 * a0 + ps0;  // quad-partial sums: reduced once at the end
    l1 = l1 * a1 + ps1;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      o[j][0] *= a0; o[j][1] *= a0; o[j][2] *= a1; o[j][3] *= a1;
    }
    // O += P V, 16 keys at a time; this thread's k-slots are keys 2t, 2t+1, 2t+8, 2t+9 of the group and its
    // B columns are V columns [16 g, 16 g + 16): n-tile j, column c of the MMA <-> V column 16 c + j
#pragma unroll
    for (int kg = 0; kg < 4; ++kg) {
      const int key0 = kbase + 16 * kg + 2 * t;
      uint4 va[2], vb[2], vc[2], vd[2];  // rows key0, key0 + 1, key0 + 8, key0 + 9
      {
        const int ka = min(key0, n - 1), kb2 = min(key0 + 1, n - 1), kc = min(key0 + 8, n - 1), kd = min(key0 + 9, n - 1);
        const uint4* ra = reinterpret_cast<const uint4*>(vp + (long long)ka * 128 + 16 * g);
        const uint4* rb = reinterpret_cast<const uint4*>(vp + (long long)kb2 * 128 + 16 * g);
        const uint4* rc = reinterpret_cast<const uint4*>(vp + (long long)kc * 128 + 16 * g);
        const uint4* rd = reinterpret_cast<const uint4*>(vp + (long long)kd * 128 + 16 * g);
        va[0] = __ldg(ra); va[1] = __ldg(ra + 1);
        vb[0] = __ldg(rb); vb[1] = __ldg(rb + 1);
        vc[0] = __ldg(rc); vc[1] = __ldg(rc + 1);
        vd[0] = __ldg(rd); vd[1] = __ldg(rd + 1);
      }
      const uint32_t* A = reinterpret_cast<const uint32_t*>(va);
      const uint32_t* Bv = reinterpret_cast<const uint32_t*>(vb);
      const uint32_t* C = reinterpret_cast<const uint32_t*>(vc);
      const uint32_t* D = reinterpret_cast<const uint32_t*>(vd);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;  // high or low halves of the two rows
        const uint32_t b0 = __byte_perm(A[j >> 1], Bv[j >> 1], sel);
        const uint32_t b1 = __byte_perm(C[j >> 1], D[j >> 1], sel);
        mma_bf16_16816(o[j], pa[2 * kg][0], pa[2 * kg][1], pa[2 * kg + 1][0], pa[2 * kg + 1][1], b0, b1);
      }
    }
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  // store partials: row g (and g + 8): V columns 32 t + j (c0 of n-tile j) and 32 t + 16 + j (c1)
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int r = g + 8 * half;
    if (r >= R) continue;
    float* po = part_o + (((long long)split * BH + bh) * R + r) * 128 + 32 * t;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      po[j] = o[j][2 * half];
      po[16 + j] = o[j][2 * half + 1];
    }
    if (t == 0) {
      float* pm = part_ml + (((long long)split * BH + bh) * R + r) * 2;
      pm[0] = half ? m1 : m0;
      pm[1] = half ? l1 : l0;
    }
  }
}

// Merge the per-warp partials of one (b, kv head, packed row): out = sum_s O_s 2^(m_s - M) / L.
// One block per row: 8 groups of 128 threads (one thread per output column) take every 8th split,
// then the groups are summed through shared memory.
constexpr int kDecMergeGroups = 8;

__global__ void __launch_bounds__(128 * kDecMergeGroups)
decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                    __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int Hq, int Hkv, int Lc,
                    int n_splits) {
  __shared__ float red_m[kDecMergeGroups];
  __shared__ float red_l[kDecMergeGroups];
  __shared__ float red_o[kDecMergeGroups][128];
  const int G = Hq / Hkv, R = Lc * G;
  const int r = blockIdx.x, bh = blockIdx.y, BH = gridDim.y;
  const int b = bh / Hkv, kvh = bh % Hkv;
  const int col = threadIdx.x & 127, grp = threadIdx.x >> 7;
  const long long stride = (long long)BH * R;  // partial rows between consecutive splits
  const long long row0 = (long long)bh * R + r;
  float M = -INFINITY;
  for (int s = grp; s < n_splits; s += kDecMergeGroups) M = fmaxf(M, __ldg(part_ml + (s * stride + row0) * 2));
  if (col == 0) red_m[grp] = M;
  __syncthreads();
  M = red_m[0];
#pragma unroll
  for (int q = 1; q < kDecMergeGroups; ++q) M = fmaxf(M, red_m[q]);
  float L = 0.f, acc = 0.f;
#pragma unroll 4
  for (int s = grp; s < n_splits; s += kDecMergeGroups) {
    const long long base = s * stride + row0;
    const float ms = __ldg(part_ml + base * 2);
    const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - M);  // a split that saw no visible key adds nothing
    L = fmaf(__ldg(part_ml + base * 2 + 1), w, L);
    acc = fmaf(__ldg(part_o + base * 128 + col), w, acc);
  }
  red_o[grp][col] = acc;
  if (col == 0) red_l[grp] = L;
  __syncthreads();
  if (grp == 0) {
#pragma unroll
    for (int q = 1; q < kDecMergeGroups; ++q) {
      acc += red_o[q][col];
      L += red_l[q];
    }
    const int head = kvh * G + r % G, i = r / G;
    const long long row = ((long long)b * Hq + head) * Lc + i;
    out[row * 128 + col] = __float2bfloat16_rn(acc / L);
    if (col == 0) lse[row] = (M + log2f(L)) * kLn2;
  }
}

inline bool decode_shape(const reform_chunk_params* p) {
  return p->dtype == REFORM_BF16 && p->d == 128 && p->Lc * (p->Hq / p->Hkv) <= kDecMaxRows;
}

inline int decode_splits(const reform_chunk_params* p) {
  return (p->n_cache + p->Lc + kDecKeysPerWarp - 1) / kDecKeysPerWarp;
}

inline size_t decode_workspace_bytes(const reform_chunk_params* p) {
  const size_t rows = (size_t)decode_splits(p) * p->B * p->Hkv * p->Lc * (p->Hq / p->Hkv);
  return align_up(rows * 128 * sizeof(float), 256) + align_up(rows * 2 * sizeof(float), 256);
}

// ws: decode_workspace_bytes(p) bytes
inline int launch_decode(const reform_chunk_params* p, float* lse, float scale, void* ws, cudaStream_t st) {
  const int n_splits = decode_splits(p);
  const int R = p->Lc * (p->Hq / p->Hkv), BH = p->B * p->Hkv;
  const size_t rows = (size_t)n_splits * BH * R;
  float* part_o = reinterpret_cast<float*>(ws);
  float* part_ml = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + align_up(rows * 128 * sizeof(float), 256));
  dim3 grid((n_splits + kDecWarps - 1) / kDecWarps, BH);
  decode_split_kernel<<<grid, 32 * kDecWarps, 0, st>>>(
      (const __nv_bfloat16*)p->q, (const __nv_bfloat16*)p->k, (const __nv_bfloat16*)p->v, part_o, part_ml,
      p->Hq, p->Hkv, p->Lc, p->n_cache, p->cap, scale * kLog2e, n_splits);
  count_launch();
  int rc = check_launch();
  if (rc != REFORM_OK) return rc;
  decode_merge_kernel<<<dim3(R, BH), 128 * kDecMergeGroups, 0, st>>>(part_o, part_ml, (__nv_bfloat16*)p->out, lse, p->Hq,
                                                  p->Hkv, p->Lc, n_splits);
  count_launch();
  return check_launch();
}

}  // namespace reform
