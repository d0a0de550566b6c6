// Segmented top-m selection by one thread-block cluster per segment, for segments of up to
// 16 x 8192 values: the cache compression of one layer (Sec. 3.1, followed in the same launch by
// the compaction of K, V, score and position rows) and the token selection of the gather phase over
// a bank of up to 131,072 tokens (Sec. 3.3, preceded in the same launch by the pooling).
//
// Same total order and same radix passes as select.cuh (value descending, index ascending; 11 + 11
// + 10 bits of the order-preserving key).  What differs is where the blocks of a segment meet: every
// thread keeps its eight keys in registers from the first pass to the last, each block histograms in
// its own shared memory, and the blocks combine through distributed shared memory and the cluster's
// hardware barrier.  Per pass: every block adds its non-empty bins into every block's copy of the
// segment histogram (remote shared-memory atomics), the cluster meets once, and every block walks
// its own copy to the same digit decision.  Nothing lives in global memory
// between the passes, nothing has to be cleared beforehand, and there is no software spin-wait: a
// cluster's blocks are co-scheduled by the hardware, and clusters of different segments never wait
// for one another, so any number of segments can be launched.
#pragma once

#include <cooperative_groups.h>

#include <mutex>

#include "common.cuh"
#include "select.cuh"

namespace reform {

namespace cg = cooperative_groups;

constexpr int kClPer = 8;                        // consecutive keys per thread
constexpr int kClTile = kSelThreads * kClPer;    // values per block at most
constexpr int kClMaxCluster = 16;
constexpr int kClMinBlocksForCopy = 96;          // cache compression: fewer blocks than this stream the kept rows too slowly

struct ClusterSelArgs {
  const float* vals;     // value (seg, i) at vals[seg * stride + i]; with pooling: the raw token scores
  long long stride;
  int n, lo, hi, m;      // segment length, candidate range [lo, hi), number to choose among the candidates
  int32_t* out;          // [segs, out_stride]
  int out_stride;
  int chunk;             // values per block: a multiple of 8, at most kClTile, cluster size * chunk >= n
  // pooling (token selection)
  float* pooled_out;     // optional [segs, stride]
  int radius, pool_mode;
  // compaction (cache compression)
  const uint4* k_src;
  const uint4* v_src;
  uint4* k_dst;
  uint4* v_dst;
  const float* score_src;
  float* score_dst;
  const int32_t* pos_src;
  int32_t* pos_dst;
  int n_kept, cap_src, cap_dst, vec, in_place;
};

struct ClusterSelSmem {
  uint32_t hist[3][kSelBins];            // this block's histogram of each pass
  uint32_t full[3][kSelBins];            // each pass's histogram of the whole segment: every block adds its own into every block's copy
  uint2 cnt[kClMaxCluster];              // every block's (keys above the threshold, keys equal to it)
  uint32_t scratch[33];
  uint32_t result[2];
  uint32_t pad[1];                       // the pooling tile that follows is read with 128-bit loads
};
static_assert(sizeof(ClusterSelSmem) % 16 == 0, "the pooling tile must start on a 16-byte boundary");

inline size_t cluster_sel_smem_bytes(bool pool, int chunk, int radius) {
  return sizeof(ClusterSelSmem) + (pool ? sizeof(float) * pool_tile_floats(chunk, radius) : 0);
}

// MODE 0: pooling + selection (token selection).  MODE 1: selection + compaction (cache compression).
template <int MODE>
__global__ void __launch_bounds__(kSelThreads) cluster_select_kernel(const ClusterSelArgs a) {
  constexpr bool POOL = MODE == 0, EVICT = MODE == 1;
  extern __shared__ __align__(16) unsigned char cl_smem_raw[];
  ClusterSelSmem& sm = *reinterpret_cast<ClusterSelSmem*>(cl_smem_raw);
  cg::cluster_group cl = cg::this_cluster();
  const int C = (int)gridDim.x;          // cluster = all blocks of one segment
  const int rank = (int)blockIdx.x, seg = (int)blockIdx.y, tid = (int)threadIdx.x;
  const int base = rank * a.chunk;
  const int end = min(base + a.chunk, a.n);
  const float* src = a.vals + (long long)seg * a.stride;

  for (int i = tid; i < 3 * kSelBins; i += kSelThreads) {
    (&sm.hist[0][0])[i] = 0;
    (&sm.full[0][0])[i] = 0;
  }
  __syncthreads();
  cl.barrier_arrive();   // this block's arrays are clear; the wait comes before the first remote add

  // this thread's values: elements base + 8 tid + j of the segment, j = 0..7
  uint32_t key[kClPer];
  uint32_t cand = 0;   // bit j: the element is a candidate
  const int g0 = base + kClPer * tid;
  {
    float x[kClPer];
#pragma unroll
    for (int j = 0; j < kClPer; ++j) x[j] = 0.f;
    if (POOL) {
      asm volatile("griddepcontrol.wait;" ::: "memory");   // the scan's scores are complete from here on
      float* tile = reinterpret_cast<float*>(cl_smem_raw + sizeof(ClusterSelSmem));
      const PoolTile pt = pool_prepare(tile, src, base, a.n, a.radius, a.pool_mode, a.chunk);
      if (kClPer * tid < a.chunk) pool_result8(pt, kClPer * tid, x);   // elements past the bank's end are not used
      if (a.pooled_out) {
        float* dst = a.pooled_out + (long long)seg * a.stride;
        if ((a.stride & 3) == 0 && g0 + kClPer <= end) {
          reinterpret_cast<float4*>(dst + g0)[0] = make_float4(x[0], x[1], x[2], x[3]);
          reinterpret_cast<float4*>(dst + g0)[1] = make_float4(x[4], x[5], x[6], x[7]);
        } else {
#pragma unroll
          for (int j = 0; j < kClPer; ++j)
            if (g0 + j < end) dst[g0 + j] = x[j];
        }
      }
    } else if ((a.stride & 3) == 0 && g0 + kClPer <= end) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(src + g0));
      const float4 w = __ldcg(reinterpret_cast<const float4*>(src + g0) + 1);
      x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
      x[4] = w.x; x[5] = w.y; x[6] = w.z; x[7] = w.w;
    } else {
#pragma unroll
      for (int j = 0; j < kClPer; ++j)
        if (g0 + j < end) x[j] = __ldcg(src + g0 + j);
    }
#pragma unroll
    for (int j = 0; j < kClPer; ++j) {
      const int g = g0 + j;
      const bool c = g < end && g >= a.lo && g < a.hi;
      key[j] = c ? float_to_key(x[j]) : 0u;
      cand |= (c ? 1u : 0u) << j;
    }
  }
  __syncthreads();

  uint32_t thr = 0xFFFFFFFFu, need_eq = 0;   // m == 0: the threshold lies above every key
  if (a.m <= 0) cl.barrier_wait();
  if (a.m > 0) {
    uint32_t prefix = 0, remaining = (uint32_t)a.m;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      int shift;
      uint32_t dmask, pmask;
      sel_pass_params(pass, shift, dmask, pmask);
      uint32_t* h = sm.hist[pass];
#pragma unroll
      for (int j = 0; j < kClPer; ++j)
        hist_add(h, (key[j] >> shift) & dmask, ((cand >> j) & 1u) && (key[j] & pmask) == prefix);
      __syncthreads();
      if (pass == 0) cl.barrier_wait();   // every block of the cluster has cleared its arrays
      // the block's non-empty bins go into every block's copy of the segment histogram
#pragma unroll
      for (int u = 0; u < kSelBins / kSelThreads; ++u) {
        const int i = u * kSelThreads + tid;
        const uint32_t v = h[i];
        if (v)
          for (int r = 0; r < C; ++r) atomicAdd(cl.map_shared_rank(&sm.full[pass][0], r) + i, v);
      }
      cl.sync();   // every block's contribution has arrived everywhere
      uint32_t bin, rem;
      find_bin_shared(sm.full[pass], remaining, sm.scratch, sm.result, bin, rem);
      prefix |= bin << shift;
      remaining = rem;
    }
    thr = prefix;
    need_eq = remaining;
  }

  // ordered write: ranks among the chosen come from one scan over the threads, the totals of the
  // blocks before this one, and a walk over the thread's own consecutive keys
  {
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < kClPer; ++j) {
      const bool c = (cand >> j) & 1u;
      mine += (c && key[j] > thr ? 1u : 0u) + (c && key[j] == thr ? 1u << 16 : 0u);
    }
    if (a.m > 0) {
      uint32_t tt;
      const uint32_t pp = block_excl_scan(mine, sm.scratch, tt);
      if (tid < C) cl.map_shared_rank(&sm.cnt[0], tid)[rank] = make_uint2(tt & 0xFFFFu, tt >> 16);
      cl.sync();   // also the last access to another block's shared memory
      uint32_t g_b = pp & 0xFFFFu, e_b = pp >> 16;
      for (int r = 0; r < rank; ++r) { g_b += sm.cnt[r].x; e_b += sm.cnt[r].y; }
      int32_t* out = a.out + (long long)seg * a.out_stride;
#pragma unroll
      for (int j = 0; j < kClPer; ++j) {
        const bool c = (cand >> j) & 1u;
        const bool is_gt = c && key[j] > thr, is_eq = c && key[j] == thr;
        if (is_gt || (is_eq && e_b < need_eq)) out[a.lo + g_b + (e_b < need_eq ? e_b : need_eq)] = g0 + j;
        g_b += is_gt;
        e_b += is_eq;
      }
    }
    if (rank == 0) {   // forced head and tail
      int32_t* out = a.out + (long long)seg * a.out_stride;
      for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
      const int tail = a.n - a.hi;
      for (int i = tid; i < tail; i += kSelThreads) out[a.lo + a.m + i] = a.hi + i;
    }
  }

  if (EVICT) {
    // compaction by the same cluster.  Kept rows only ever move down (kept[r] >= r, ascending), so
    // in place the ranks are taken in waves: every thread of the cluster loads its share of the
    // wave, the cluster meets, every thread stores.  A wave's stores land in rank positions below
    // everything a later wave still has to read.
    __threadfence();
    cl.sync();   // the segment's kept list is complete
    const int32_t* kept = a.out + (long long)seg * a.out_stride;
    const int T = C * kSelThreads, gtid = rank * kSelThreads + tid;
    const long long so0 = (long long)seg * a.cap_src, dn0 = (long long)seg * a.cap_dst;
    const long long items = (long long)a.n_kept * a.vec;
    for (long long i0 = 0; i0 < items; i0 += 4LL * T) {
      uint4 kk[4], vv[4];
      long long dn[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const long long i = i0 + (long long)u * T + gtid;
        dn[u] = -1;
        if (i < items) {
          const int row = (int)(i / a.vec), c = (int)(i - (long long)row * a.vec);
          const int j = __ldcg(kept + row);
          const long long so = (so0 + j) * a.vec + c;
          dn[u] = (dn0 + row) * a.vec + c;
          kk[u] = __ldcs(a.k_src + so);
          vv[u] = __ldcs(a.v_src + so);
        }
      }
      if (a.in_place) {
        __threadfence();
        cl.sync();
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (dn[u] >= 0) {
          __stcs(a.k_dst + dn[u], kk[u]);
          __stcs(a.v_dst + dn[u], vv[u]);
        }
    }
    for (int r0 = 0; r0 < a.n_kept; r0 += T) {
      const int row = r0 + gtid;
      float sc = 0.f;
      int32_t ps = 0;
      if (row < a.n_kept) {
        const int j = __ldcg(kept + row);
        sc = __ldcg(a.score_src + so0 + j);
        if (a.pos_dst) ps = __ldcg(a.pos_src + so0 + j);
      }
      if (a.in_place) {
        __threadfence();
        cl.sync();
      }
      if (row < a.n_kept) {
        a.score_dst[dn0 + row] = sc;
        if (a.pos_dst) a.pos_dst[dn0 + row] = ps;
      }
    }
  }
}

// How many clusters of 2^i blocks of cluster_select_kernel<MODE> the current device runs at once
// (i = 0..4), asked once per device with the largest shared-memory size seen so far; all zero if
// cluster launches are not available.
struct ClusterCapacity {
  int active[5];
};

template <int MODE>
inline ClusterCapacity cluster_select_capacity(size_t smem) {
  constexpr int kMaxDevices = 64;
  static ClusterCapacity cache[kMaxDevices] = {};
  static size_t cache_smem[kMaxDevices] = {0};
  static std::mutex guard;   // host threads may make their first call at the same time
  const ClusterCapacity none = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return none;
  std::lock_guard<std::mutex> lock(guard);
  if (cache_smem[dev] != 0 && smem <= cache_smem[dev]) return cache[dev];
  ClusterCapacity cap = {};
  const void* fn = (const void*)cluster_select_kernel<MODE>;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess &&
      cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
    for (int i = 0; i < 5; ++i) {
      const int c = 1 << i;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(c, 1, 1);
      cfg.blockDim = dim3(kSelThreads);
      cfg.dynamicSmemBytes = smem;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = c;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &cfg) == cudaSuccess) cap.active[i] = n_clusters;
      else cudaGetLastError();
    }
  } else {
    cudaGetLastError();
  }
  cache[dev] = cap;
  cache_smem[dev] = smem;
  return cap;
}

// Cluster size for `segs` segments of n values: the smallest power of two whose blocks hold a
// segment, doubled while all clusters of the call still run at once and every thread keeps at
// least two values.  0 if the segment is too long for the largest cluster the device takes.
inline int cluster_select_size(int segs, long long n, const ClusterCapacity& cap) {
  int i = 0;
  while (i < 5 && (long long)(1 << i) * kClTile < n) ++i;
  if (i >= 5 || cap.active[i] < 1) return 0;
  while (i + 1 < 5 && cap.active[i + 1] >= segs && n >= (2LL << i) * 2 * kSelThreads) ++i;
  return 1 << i;
}

// True if `segs` clusters of c blocks all run at the same time on the device.
inline bool cluster_select_one_wave(int segs, int c, const ClusterCapacity& cap) {
  int i = 0;
  while ((1 << i) < c) ++i;
  return i < 5 && cap.active[i] >= segs;
}

template <int MODE>
inline int launch_cluster_select(ClusterSelArgs a, int segs, int c, cudaStream_t st) {
  a.chunk = (int)align_up((size_t)((a.n + c - 1) / c), kClPer);
  if (a.chunk < kClPer) a.chunk = kClPer;
  const size_t smem = cluster_sel_smem_bytes(MODE == 0, a.chunk, a.radius);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(c, segs, 1);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = c;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // token selection: placed while the scan that writes its scores drains (the kernel waits for the
  // scan's completion before its first read of them)
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = MODE == 0 ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, cluster_select_kernel<MODE>, a);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return REFORM_ERR_CUDA;
  }
  count_launch();
  return check_launch();
}

}  // namespace reform
