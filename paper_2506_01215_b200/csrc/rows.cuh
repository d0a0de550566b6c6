// Row movers: the gather of Sec. 3.3 and the compaction half of the cache
// compression of Sec. 3.1.  Both are pure HBM traffic: 128-bit loads and
// stores, LANES threads per row so a warp always touches whole 128-byte lines,
// several independent loads in flight per thread before the first store.
#pragma once

#include "common.cuh"

namespace reform {

constexpr int kRowThreads = 256;

// dst[b, r, :] = src[b, idx[b, r], :].  vec = row_bytes / 16.
template <int LANES>
__global__ void __launch_bounds__(kRowThreads)
gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ idx,
                   uint4* __restrict__ dst, long long total_rows, int k, long long n_rows, int vec,
                   int32_t* dev_status) {
  constexpr int ROWS = kRowThreads / LANES;
  const int lane = threadIdx.x % LANES;
  const int sub = threadIdx.x / LANES;
  for (long long r = (long long)blockIdx.x * ROWS + sub; r < total_rows;
       r += (long long)gridDim.x * ROWS) {
    long long b = r / k;
    long long j = idx[r];
    uint4* d = dst + r * vec;
    if (j < 0 || j >= n_rows) {
      if (lane == 0) report_device_error(dev_status, REFORM_DEV_BAD_INDEX);
      for (int c = lane; c < vec; c += LANES) d[c] = make_uint4(0, 0, 0, 0);
      continue;
    }
    const uint4* s = src + (b * n_rows + j) * vec;
    int c = lane;
    for (; c + 3 * LANES < vec; c += 4 * LANES) {
      uint4 a0 = __ldcs(s + c), a1 = __ldcs(s + c + LANES), a2 = __ldcs(s + c + 2 * LANES),
            a3 = __ldcs(s + c + 3 * LANES);
      __stcs(d + c, a0);
      __stcs(d + c + LANES, a1);
      __stcs(d + c + 2 * LANES, a2);
      __stcs(d + c + 3 * LANES, a3);
    }
    for (; c < vec; c += LANES) __stcs(d + c, __ldcs(s + c));
  }
}

inline int launch_gather(const uint4* src, const int32_t* idx, uint4* dst, int B, int k,
                         long long n_rows, long long row_bytes, int32_t* dev_status,
                         cudaStream_t st) {
  long long total = (long long)B * k;
  if (total == 0) return REFORM_OK;
  int vec = (int)(row_bytes / 16);
  int lanes = 1;  // power of two, <= 256, about four 16-byte chunks per lane so four loads are in flight
  while (4 * lanes < vec && lanes < kRowThreads) lanes <<= 1;
  long long rows_per_block = kRowThreads / lanes;
  long long blocks = (total + rows_per_block - 1) / rows_per_block;
  long long cap = (long long)num_sms() * 16;
  int grid = (int)(blocks < cap ? blocks : cap);
#define REFORM_GATHER_CASE(L)                                                                    \
  case L:                                                                                        \
    gather_rows_kernel<L><<<grid, kRowThreads, 0, st>>>(src, idx, dst, total, k, n_rows, vec,    \
                                                        dev_status);                             \
    break;
  switch (lanes) {
    REFORM_GATHER_CASE(1)
    REFORM_GATHER_CASE(2)
    REFORM_GATHER_CASE(4)
    REFORM_GATHER_CASE(8)
    REFORM_GATHER_CASE(16)
    REFORM_GATHER_CASE(32)
    REFORM_GATHER_CASE(64)
    REFORM_GATHER_CASE(128)
    REFORM_GATHER_CASE(256)
  }
#undef REFORM_GATHER_CASE
  count_launch();
  return check_launch();
}

// Compaction: for segment s = (b, kv head) and kept rank r < n_kept,
//   k_dst[s, r, :] = k_src[s, kept[s, r], :] (blockIdx.y == 0), same for v
//   (blockIdx.y == 1); the y == 0 blocks also move score and position.
template <int LANES>
__global__ void __launch_bounds__(kRowThreads)
evict_compact_kernel(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                     uint4* __restrict__ k_dst, uint4* __restrict__ v_dst,
                     const float* __restrict__ score_src, float* __restrict__ score_dst,
                     const int32_t* __restrict__ pos_src, int32_t* __restrict__ pos_dst,
                     const int32_t* __restrict__ kept, int kept_stride, int segs, int n_kept,
                     int cap_src, int cap_dst, int vec) {
  constexpr int ROWS = kRowThreads / LANES;
  const int lane = threadIdx.x % LANES;
  const int sub = threadIdx.x / LANES;
  const uint4* src = blockIdx.y ? v_src : k_src;
  uint4* dst = blockIdx.y ? v_dst : k_dst;
  const long long total = (long long)segs * n_kept;
  for (long long r = (long long)blockIdx.x * ROWS + sub; r < total;
       r += (long long)gridDim.x * ROWS) {
    int s = (int)(r / n_kept);
    int rank = (int)(r % n_kept);
    int j = kept[(long long)s * kept_stride + rank];
    const uint4* sp = src + ((long long)s * cap_src + j) * vec;
    uint4* dp = dst + ((long long)s * cap_dst + rank) * vec;
    int c = lane;
    for (; c + 3 * LANES < vec; c += 4 * LANES) {
      uint4 a0 = __ldcs(sp + c), a1 = __ldcs(sp + c + LANES), a2 = __ldcs(sp + c + 2 * LANES),
            a3 = __ldcs(sp + c + 3 * LANES);
      __stcs(dp + c, a0);
      __stcs(dp + c + LANES, a1);
      __stcs(dp + c + 2 * LANES, a2);
      __stcs(dp + c + 3 * LANES, a3);
    }
    for (; c < vec; c += LANES) __stcs(dp + c, __ldcs(sp + c));
    if (blockIdx.y == 0 && lane == 0) {
      if (score_dst) score_dst[(long long)s * cap_dst + rank] = score_src[(long long)s * cap_src + j];
      if (pos_dst) pos_dst[(long long)s * cap_dst + rank] = pos_src[(long long)s * cap_src + j];
    }
  }
}

inline int launch_evict_compact(const void* k_src, const void* v_src, void* k_dst, void* v_dst,
                                const float* score_src, float* score_dst, const int32_t* pos_src,
                                int32_t* pos_dst, const int32_t* kept, int kept_stride, int segs,
                                int n_kept, int cap_src, int cap_dst, int row_bytes,
                                cudaStream_t st) {
  long long total = (long long)segs * n_kept;
  if (total == 0) return REFORM_OK;
  int vec = row_bytes / 16;
  int lanes = 1;
  while (4 * lanes < vec && lanes < 32) lanes <<= 1;
  long long rows_per_block = kRowThreads / lanes;
  long long blocks = (total + rows_per_block - 1) / rows_per_block;
  long long cap = (long long)num_sms() * 8;
  dim3 grid((unsigned)(blocks < cap ? blocks : cap), 2);
#define REFORM_COMPACT_CASE(L)                                                                   \
  case L:                                                                                        \
    evict_compact_kernel<L><<<grid, kRowThreads, 0, st>>>(                                       \
        (const uint4*)k_src, (const uint4*)v_src, (uint4*)k_dst, (uint4*)v_dst, score_src,       \
        score_dst, pos_src, pos_dst, kept, kept_stride, segs, n_kept, cap_src, cap_dst, vec);    \
    break;
  switch (lanes) {
    REFORM_COMPACT_CASE(1)
    REFORM_COMPACT_CASE(2)
    REFORM_COMPACT_CASE(4)
    REFORM_COMPACT_CASE(8)
    REFORM_COMPACT_CASE(16)
    REFORM_COMPACT_CASE(32)
  }
#undef REFORM_COMPACT_CASE
  count_launch();
  return check_launch();
}

}  // namespace reform
