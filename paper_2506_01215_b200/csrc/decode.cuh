// Decode-shaped chunk step (bf16, d = 128, Lc * G <= 16): the step that follows
// the on-demand recomputation (Sec. 3.3) -- one or a few new tokens attending
// over the recomputed cache.  With so few query rows the operation is a read
// of K and V, so it is split along the keys: a warp owns runs of 32 keys of one KV
// head, packs the Lc * G query rows of the group into one 16-row MMA tile,
// streams its K and V rows global -> registers with 128-bit loads and takes
// the softmax of its keys; the partials are merged per block and then, in a
// second small kernel, per KV head.  The k index of Q K^T and the column
// order of O are permuted so that what a thread loads contiguously is exactly
// what its mma.sync fragments need (a dot product does not care about the
// order of its terms, and the output columns are un-permuted when stored).
#pragma once

#include "common.cuh"
#include "chunk_simt.cuh"
#include "retrieve.cuh"  // mma_bf16_16816

namespace reform {

constexpr int kDecGroup = 32;              // keys a warp has in flight at a time (8 KB of K, then 8 KB of V)
constexpr int kDecWarps = 8;
constexpr int kDecMaxBlocksPerHead = 40;   // partials the last block has to merge
constexpr int kDecMaxRows = 16;
// the warps' partials [warps][16][128] and their (max, sum) [warps][16][2]; the last block reuses the
// first part for the blocks' weights [kDecMaxBlocksPerHead][16] followed by [warps][16][128] sums
constexpr size_t kDecSmemBytes =
    ((size_t)kDecMaxBlocksPerHead * kDecMaxRows + (size_t)kDecWarps * kDecMaxRows * 128 + kDecWarps * kDecMaxRows * 2) *
    sizeof(float);

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// A warp owns `groups` runs of 32 consecutive keys of one KV head; for each run it issues all of
// the run's K loads (sixteen 128-bit loads per thread) before the first MMA, takes S = Q K^T,
// issues all of the run's V loads, and folds the run into its running (max, sum, O).  The eight
// warps of a block merge their partials through shared memory and store one partial per block:
//   part_o [blocks_per_head][BH][R][128] fp32;  part_ml [blocks_per_head][BH][R][2] (max in log2 units, sum)
// decode_merge_kernel then folds the blocks' partials of each KV head.  (Folding them in the same
// launch, by the block that arrives last at a per-head counter, was measured: with some thirty
// blocks per head arriving together the atomic exchanges on one word queue up for longer than a
// second launch costs.)
__global__ void __launch_bounds__(32 * kDecWarps)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, float* __restrict__ part_o,
                    float* __restrict__ part_ml, int Hq, int Hkv, int Lc, int n_cache, int cap,
                    float scale_log2, int groups) {
  extern __shared__ float dec_smem[];
  float* so = dec_smem;                                        // [warps][16][128] (+ room for the last block's weights)
  float* sml = dec_smem + kDecMaxBlocksPerHead * kDecMaxRows + kDecWarps * kDecMaxRows * 128;   // [warps][16][2]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int bh = blockIdx.y, b = bh / Hkv, kvh = bh % Hkv;
  const int G = Hq / Hkv, R = Lc * G, n = n_cache + Lc;
  const int BH = gridDim.y;
  const __nv_bfloat16* kp = k + ((long long)bh * cap) * 128;
  const __nv_bfloat16* vp = v + ((long long)bh * cap) * 128;
  constexpr int NT = kDecGroup / 8;

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

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

#pragma unroll 1
  for (int it = 0; it < groups; ++it) {
    const int kbase = ((blockIdx.x * groups + it) * kDecWarps + warp) * kDecGroup;
    if (kbase >= n) break;
    // all K loads of the run first: 32 keys x 256 B in flight per warp
    uint4 kk[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      int key = kbase + 8 * nt + g;
      if (key > n - 1) key = n - 1;  // clamped rows are masked below
      const uint4* kr = reinterpret_cast<const uint4*>(kp + (long long)key * 128) + t;
#pragma unroll
      for (int kb = 0; kb < 4; ++kb) kk[nt][kb] = __ldg(kr + 4 * kb);
    }
    float s[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int kb = 0; kb < 4; ++kb) {
        mma_bf16_16816(s[nt], qa[kb].x, qb[kb].x, qa[kb].y, qb[kb].y, kk[nt][kb].x, kk[nt][kb].y);
        mma_bf16_16816(s[nt], qa[kb].z, qb[kb].z, qa[kb].w, qb[kb].w, kk[nt][kb].z, kk[nt][kb].w);
      }
    }
    // all V loads of the run, in flight under the softmax arithmetic: rows key0, key0 + 1, key0 + 8,
    // key0 + 9 of each 16-key group, 32 bytes of each (V columns [16 g, 16 g + 16))
    uint4 vr[NT / 2][4][2];
#pragma unroll
    for (int kg = 0; kg < NT / 2; ++kg) {
      const int key0 = kbase + 16 * kg + 2 * t;
      const int kr4[4] = {min(key0, n - 1), min(key0 + 1, n - 1), min(key0 + 8, n - 1), min(key0 + 9, n - 1)};
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const uint4* rp = reinterpret_cast<const uint4*>(vp + (long long)kr4[x] * 128 + 16 * g);
        vr[kg][x][0] = __ldg(rp);
        vr[kg][x][1] = __ldg(rp + 1);
      }
    }
    // mask, maximum per row (rows g and g + 8), quad reduce
    float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
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
    uint32_t pa[NT][2];  // per n-tile: packed P of row g, of row g + 8
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float p00 = exp2f(fmaf(s[nt][0], scale_log2, -sub0)), p01 = exp2f(fmaf(s[nt][1], scale_log2, -sub0));
      const float p10 = exp2f(fmaf(s[nt][2], scale_log2, -sub1)), p11 = exp2f(fmaf(s[nt][3], scale_log2, -sub1));
      ps0 += p00 + p01;
      ps1 += p10 + p11;
      pa[nt][0] = pack2_bf16(p00, p01);
      pa[nt][1] = pack2_bf16(p10, p11);
    }
    l0 = l0 * a0 + ps0;  // quad-partial sums: reduced once at the end
    l1 = l1 * a1 + ps1;
    if (it > 0) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        o[j][0] *= a0; o[j][1] *= a0; o[j][2] *= a1; o[j][3] *= a1;
      }
    }
    // O += P V, 16 keys at a time; this thread's k-slots are keys 2t, 2t+1, 2t+8, 2t+9 of the group and its
    // B columns are V columns [16 g, 16 g + 16): n-tile j, column c of the MMA <-> V column 16 c + j
#pragma unroll
    for (int kg = 0; kg < NT / 2; ++kg) {
      const uint32_t* A = reinterpret_cast<const uint32_t*>(vr[kg][0]);
      const uint32_t* Bv = reinterpret_cast<const uint32_t*>(vr[kg][1]);
      const uint32_t* C = reinterpret_cast<const uint32_t*>(vr[kg][2]);
      const uint32_t* D = reinterpret_cast<const uint32_t*>(vr[kg][3]);
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
  // the warp's partial into shared memory: row g (and g + 8), V columns 32 t + j (c0 of n-tile j)
  // and 32 t + 16 + j (c1)
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int r = g + 8 * half;
    float* po = so + ((warp * kDecMaxRows + r) * 128) + 32 * t;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      po[j] = o[j][2 * half];
      po[16 + j] = o[j][2 * half + 1];
    }
    if (t == 0) {
      sml[(warp * kDecMaxRows + r) * 2] = half ? m1 : m0;
      sml[(warp * kDecMaxRows + r) * 2 + 1] = half ? l1 : l0;
    }
  }
  __syncthreads();
  // merge the warps of the block: thread = (column, every kRowStep-th row)
  const int col = threadIdx.x & 127;
  constexpr int kRowStep = 32 * kDecWarps / 128;   // threads = columns x kRowStep rows at a time
  for (int r = threadIdx.x >> 7; r < R; r += kRowStep) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) M = fmaxf(M, sml[(w * kDecMaxRows + r) * 2]);
    float L = 0.f, acc = 0.f;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
      const float ms = sml[(w * kDecMaxRows + r) * 2];
      const float wgt = (ms == -INFINITY) ? 0.f : exp2f(ms - M);   // a warp that saw no visible key adds nothing
      L = fmaf(sml[(w * kDecMaxRows + r) * 2 + 1], wgt, L);
      acc = fmaf(so[(w * kDecMaxRows + r) * 128 + col], wgt, acc);
    }
    const long long row = ((long long)blockIdx.x * BH + bh) * R + r;
    __stcg(part_o + row * 128 + col, acc);
    if (col == 0) {
      __stcg(part_ml + row * 2, M);
      __stcg(part_ml + row * 2 + 1, L);
    }
  }
}

// out = sum_b O_b 2^(m_b - M) / L over the blocks' partials of one KV head (one block per head).
// Every load is independent of every other, and they are issued that way: first all (max, sum)
// pairs into shared memory, then each warp takes every kDecWarps-th block's O rows as 128-bit
// loads, and the warps' sums meet in shared memory.
__global__ void __launch_bounds__(32 * kDecWarps)
decode_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                    __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int Hq, int Hkv, int Lc,
                    int n_blocks) {
  extern __shared__ float dec_smem[];
  float* so = dec_smem;
  float* sml = dec_smem + kDecMaxBlocksPerHead * kDecMaxRows + kDecWarps * kDecMaxRows * 128;
  // launched while decode_split_kernel may still be running (programmatic dependent launch): its
  // partials are complete and visible only from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bh = blockIdx.x, b = bh / Hkv, kvh = bh % Hkv, BH = gridDim.x;
  const int G = Hq / Hkv, R = Lc * G;
  const int col = threadIdx.x & 127;
  constexpr int kRowStep = 32 * kDecWarps / 128;
  float* wgt = so;                                   // [n_blocks][16] weights 2^(m_b - M)
  float* red = so + kDecMaxBlocksPerHead * kDecMaxRows;   // [warps][16][128] partial sums
  float* rowML = sml;                                // [16][2] merged (M, L) per row
  const long long stride = (long long)BH * R;       // partial rows between consecutive blocks
  const long long row00 = (long long)bh * R;
  float* sums = red;                                 // [n_blocks][16] the blocks' row sums, until red is needed
  for (int i = threadIdx.x; i < n_blocks * R; i += blockDim.x) {
    const int bb = i / R, r = i - bb * R;
    const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + (bb * stride + row00 + r) * 2));
    wgt[bb * kDecMaxRows + r] = ml.x;       // m_b for now
    sums[bb * kDecMaxRows + r] = ml.y;
  }
  __syncthreads();
  if (threadIdx.x < R) {
    const int r = threadIdx.x;
    float M = -INFINITY;
    for (int bb = 0; bb < n_blocks; ++bb) M = fmaxf(M, wgt[bb * kDecMaxRows + r]);
    rowML[2 * r] = M;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_blocks * R; i += blockDim.x) {
    const int bb = i / R, r = i - bb * R;
    const float ms = wgt[bb * kDecMaxRows + r];
    wgt[bb * kDecMaxRows + r] = (ms == -INFINITY) ? 0.f : exp2f(ms - rowML[2 * r]);
  }
  __syncthreads();
  if (threadIdx.x < R) {
    const int r = threadIdx.x;
    float L = 0.f;
    for (int bb = 0; bb < n_blocks; ++bb) L = fmaf(sums[bb * kDecMaxRows + r], wgt[bb * kDecMaxRows + r], L);
    rowML[2 * r + 1] = L;
  }
  __syncthreads();   // sums has been read: red may be written
  {
    // warp w sums one row over a share of the blocks: with R <= 8 rows, row w % R and every
    // (8 / R)-th block; with more rows, rows w and w + 8 over all blocks.  All of a warp's loads
    // are independent and issued together.
    const int c4 = lane;   // columns 4 * lane .. 4 * lane + 3
    const int shares = R <= kDecWarps ? kDecWarps / R : 1;
    for (int r = R <= kDecWarps ? warp % R : warp; r < R; r += kDecWarps) {
      const int first = R <= kDecWarps ? warp / R : 0;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (first < shares) {
#pragma unroll 8
        for (int bb = first; bb < n_blocks; bb += shares) {
          const float4 x = __ldcg(reinterpret_cast<const float4*>(part_o + (bb * stride + row00 + r) * 128) + c4);
          const float wv = wgt[bb * kDecMaxRows + r];
          acc.x = fmaf(x.x, wv, acc.x);
          acc.y = fmaf(x.y, wv, acc.y);
          acc.z = fmaf(x.z, wv, acc.z);
          acc.w = fmaf(x.w, wv, acc.w);
        }
      }
      reinterpret_cast<float4*>(red + ((R <= kDecWarps ? first : 0) * kDecMaxRows + r) * 128)[c4] = acc;
    }
  }
  __syncthreads();
  const int shares_used = R <= kDecWarps ? kDecWarps / R : 1;
  for (int r = threadIdx.x >> 7; r < R; r += kRowStep) {
    float acc = 0.f;
    for (int w = 0; w < shares_used; ++w) acc += red[(w * kDecMaxRows + r) * 128 + col];
    const int head = kvh * G + r % G, i = r / G;
    const long long orow = ((long long)b * Hq + head) * Lc + i;
    out[orow * 128 + col] = __float2bfloat16_rn(acc / rowML[2 * r + 1]);
    if (col == 0) lse[orow] = (rowML[2 * r] + log2f(rowML[2 * r + 1])) * kLn2;
  }
}

inline bool decode_shape(const reform_chunk_params* p) {
  return p->dtype == REFORM_BF16 && p->d == 128 && p->Lc * (p->Hq / p->Hkv) <= kDecMaxRows;
}

// 32-key runs per warp: enough that all blocks of the call fit the device in one wave, and that no
// KV head has more than kDecMaxBlocksPerHead blocks
inline int decode_groups(const reform_chunk_params* p) {
  const long long n = (long long)p->n_cache + p->Lc;
  const long long per_block = (long long)kDecWarps * kDecGroup;
  long long per_head = num_sms() / ((long long)p->B * p->Hkv);   // blocks per KV head in one wave (one block per SM)
  if (per_head < 1) per_head = 1;
  if (per_head > kDecMaxBlocksPerHead) per_head = kDecMaxBlocksPerHead;
  const long long gr = (n + per_block * per_head - 1) / (per_block * per_head);
  return (int)(gr < 1 ? 1 : gr);
}

inline int decode_blocks(const reform_chunk_params* p) {
  const long long per_block = (long long)kDecWarps * kDecGroup * decode_groups(p);
  return (int)(((long long)p->n_cache + p->Lc + per_block - 1) / per_block);
}

inline size_t decode_workspace_bytes(const reform_chunk_params* p) {
  // sized for the most blocks any device could be given (one 256-key run per block)
  const size_t blocks = ((size_t)p->n_cache + p->Lc + kDecWarps * kDecGroup - 1) / (kDecWarps * kDecGroup);
  const size_t most = blocks < (size_t)kDecMaxBlocksPerHead ? blocks : (size_t)kDecMaxBlocksPerHead;
  const size_t rows = most * p->B * p->Hkv * p->Lc * (p->Hq / p->Hkv);
  return align_up(rows * 128 * sizeof(float), 256) + align_up(rows * 2 * sizeof(float), 256);
}

// ws: decode_workspace_bytes(p) bytes
inline int launch_decode(const reform_chunk_params* p, float* lse, float scale, void* ws, cudaStream_t st) {
  const int n_blocks = decode_blocks(p);
  const int R = p->Lc * (p->Hq / p->Hkv), BH = p->B * p->Hkv;
  const size_t rows = (size_t)n_blocks * BH * R;
  char* w = reinterpret_cast<char*>(ws);
  float* part_o = reinterpret_cast<float*>(w);
  w += align_up(rows * 128 * sizeof(float), 256);
  float* part_ml = reinterpret_cast<float*>(w);
  cudaFuncSetAttribute(decode_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
  cudaFuncSetAttribute(decode_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
  decode_split_kernel<<<dim3(n_blocks, BH), 32 * kDecWarps, kDecSmemBytes, st>>>(
      (const __nv_bfloat16*)p->q, (const __nv_bfloat16*)p->k, (const __nv_bfloat16*)p->v, part_o, part_ml,
      p->Hq, p->Hkv, p->Lc, p->n_cache, p->cap, scale * kLog2e, decode_groups(p));
  count_launch();
  int rc = check_launch();
  if (rc != REFORM_OK) return rc;
  {
    // the merge kernel is queued behind the split kernel with programmatic serialisation: its blocks
    // are placed while the split kernel drains and wait on griddepcontrol.wait for its completion
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(BH);
    cfg.blockDim = dim3(32 * kDecWarps);
    cfg.dynamicSmemBytes = kDecSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* po = part_o;
    const float* pm = part_ml;
    __nv_bfloat16* outp = (__nv_bfloat16*)p->out;
    int Hq = p->Hq, Hkv = p->Hkv, Lc = p->Lc, nb = n_blocks;
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_merge_kernel, po, pm, outp, lse, Hq, Hkv, Lc, nb);
    if (e != cudaSuccess) {
      g_last_cuda_error = (int)e;
      return REFORM_ERR_CUDA;
    }
  }
  count_launch();
  return check_launch();
}

}  // namespace reform
