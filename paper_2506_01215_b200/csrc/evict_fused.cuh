// Cache compression (Sec. 3.1) as one cooperative launch: per (sequence, KV head)
// segment the top-m selection and then the compaction of K, V, score and
// position rows, with two grid-level hand-offs instead of one per radix pass.
//
// Selection blocks (1024 threads, 8 consecutive keys per thread held in
// registers, nb blocks per segment):
//   A  histogram of the top 11 key bits in shared memory, published as this
//      block's own slice (plain stores: nothing in the workspace has to be
//      zero beforehand, and there are no global atomics).
//   -- hand-off 1: every block of the segment has published --
//   B  each block adds the nb slices, finds the bin b1 that holds the m-th key,
//      and appends its own keys of that bin to the segment's candidate list at
//      an offset it computes from the slices; the slices also tell it how many
//      keys of the blocks before it lie in bins above b1.
//   -- hand-off 2 --
//   C  each block walks the candidate list (typically a few thousand keys) and
//      resolves the remaining 21 bits with two shared-memory histograms, then
//      counts, among the candidates of the blocks before it, the keys above
//      and equal to the threshold: with that it writes its kept indices at
//      their final, ordered positions (ties to the lowest index).
//   -- hand-off 3: the kept lists of all segments are complete --
// Then every block of the grid streams kept rows (128-bit loads and stores).
//
// In place (destinations == sources): kept rows only ever move down (kept[r] >= r, ascending), so
// the ranks are taken in waves of as many rows as the grid can hold in registers at once: every
// block loads its rows of the wave, all blocks meet (one more flag per block), then every block
// stores.  A wave's stores land in rank positions [w R, (w+1) R) of each segment; every row that
// still has to be read from there belongs to this wave or an earlier one and is in registers by
// then, and later waves read from beyond (w+1) R.
//
// Hand-offs are 64-bit flags, one per selection block, that carry the call's
// epoch and the phase reached; a stale flag from an earlier call (or whatever
// the workspace held before) never matches the epoch, so the workspace needs no
// clearing.  Every wait is bounded; a block that gives up records the epoch in
// the segment-independent abort word, raises REFORM_DEV_TIMEOUT and the launch
// winds down.
#pragma once

#include "common.cuh"
#include "rows.cuh"
#include "select.cuh"

namespace reform {

constexpr int kEvPerThread = 8;            // consecutive keys a thread holds in registers
constexpr int kEvTile = kSelThreads * kEvPerThread;   // keys per selection block
constexpr int kEvMaxBlocksPerSeg = 32;     // slices each block has to add up (segments up to 262,144 keys)
constexpr long long kEvWaitCycles = 400000000LL;  // about 0.2 s; real waits are microseconds
constexpr unsigned long long kEvPhaseMask = 0xFFull;   // a flag is (epoch with these bits clear) | phase
constexpr int kEvMaxGrid = 1024;           // blocks a launch may have (one flag each for the in-place copy)
constexpr int kEvMaxWaves = 200;           // in-place copy: phases 4 .. 4 + waves - 1 must fit the phase field

struct EvictFusedArgs {
  // selection
  const float* vals;
  long long stride;
  int n, lo, hi, m;
  int32_t* out;
  int out_stride;
  int segs, nb;
  uint32_t* slices;            // [segs][nb][kSelBins]
  uint32_t* cand;              // [segs][n]
  unsigned long long* flags;   // [segs * nb] one flag per selection block, the abort word, a slot nothing writes, [kEvMaxGrid] one flag per block of the grid
  int expect_extra;            // diagnostic: the first hand-off also waits for the slot nothing writes (0 in normal use)
  unsigned long long epoch;    // low 8 bits clear: the phase goes there
  int in_place;                // destinations are the sources: rows move down inside their own buffers
  long long wait_cycles;
  // compaction
  const uint4* k_src;
  const uint4* v_src;
  uint4* k_dst;
  uint4* v_dst;
  const float* score_src;
  float* score_dst;
  const int32_t* pos_src;
  int32_t* pos_dst;
  int n_kept, cap_src, cap_dst, vec;
  int32_t* dev_status;
};

struct EvictFusedLayout {
  size_t flags, slices, cand, total;
  int nb;
};

inline EvictFusedLayout evict_fused_layout(int segs, int n) {
  EvictFusedLayout L;
  L.nb = (n + kEvTile - 1) / kEvTile;
  if (L.nb < 1) L.nb = 1;
  size_t off = 0;
  L.flags = off;
  off += align_up(sizeof(unsigned long long) * ((size_t)segs * L.nb + 2 + kEvMaxGrid), 256);
  L.slices = off;
  off += align_up(sizeof(uint32_t) * (size_t)segs * L.nb * kSelBins, 256);
  L.cand = off;
  off += align_up(sizeof(uint32_t) * (size_t)segs * (n > 0 ? n : 1), 256);
  L.total = off;
  return L;
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Waits until each of the `count` flags at `flags` (and the one at `extra`, if given) carries this
// call's epoch and a phase >= phase.  Called by all threads of the block; returns false (to all of
// them) if the wait ran out or another block gave up.  sleep_ns > 0 spaces the polls of a wait that
// is expected to be long.
__device__ __forceinline__ bool wait_flags(const unsigned long long* flags, int count, const unsigned long long* extra,
                                           unsigned long long epoch, unsigned phase, unsigned long long* abort_word,
                                           long long wait_cycles, unsigned sleep_ns, int32_t* dev_status) {
  __shared__ int wf_failed;
  if (threadIdx.x == 0) wf_failed = 0;
  __syncthreads();
  const long long t0 = clock64();
  const int total = count + (extra ? 1 : 0);
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const unsigned long long* f = i < count ? flags + i : extra;
    for (uint32_t it = 0;; ++it) {
      const unsigned long long v = ld_acquire_u64(f);
      if ((v & ~kEvPhaseMask) == epoch && (unsigned)(v & kEvPhaseMask) >= phase) break;
      if (sleep_ns) __nanosleep(sleep_ns);
      if ((it & 15u) == 15u || sleep_ns) {
        if (ld_acquire_u64(abort_word) == epoch || *(volatile int*)&wf_failed) { wf_failed = 1; break; }
        if (clock64() - t0 > wait_cycles) {
          st_release_u64(abort_word, epoch);
          report_device_error(dev_status, REFORM_DEV_TIMEOUT);
          wf_failed = 1;
          break;
        }
      }
    }
  }
  __syncthreads();   // the polling threads' acquire loads, then the barrier, order every thread's later reads
  const bool ok = wf_failed == 0;
  __syncthreads();
  return ok;
}

// Publishes phase `phase` of this block: everything the block stored before is visible to whoever
// reads the flag with acquire semantics.  Called by all threads.
__device__ __forceinline__ void publish_phase(unsigned long long* flag, unsigned long long epoch, unsigned phase) {
  __syncthreads();   // the block's stores are ordered before thread 0's fence, which makes them visible device-wide
  if (threadIdx.x == 0) {
    __threadfence();
    st_release_u64(flag, epoch | phase);
  }
}

constexpr int kEvCandSmem = 8192;   // candidates of a segment staged in shared memory when they fit

// key i of a segment's candidate list: from shared memory if the list was staged there
__device__ __forceinline__ uint32_t cand_key(const uint32_t* staged, const uint32_t* global, bool in_smem, uint32_t i) {
  return in_smem ? staged[i] : __ldcg(global + i);
}

__global__ void __launch_bounds__(kSelThreads)
evict_fused_kernel(const EvictFusedArgs a) {
  __shared__ uint32_t hist[kSelBins];
  __shared__ uint32_t cbuf[kEvCandSmem];
  __shared__ uint32_t scratch[33];
  __shared__ uint32_t result[2];
  __shared__ uint32_t counter, shared_base;
  const int tid = threadIdx.x;
  const int n_sel_blocks = a.m > 0 ? a.segs * a.nb : 0;
  unsigned long long* abort_word = a.flags + (size_t)a.segs * a.nb;
  const unsigned long long* never_set = abort_word + 1;
  const bool selects = (int)blockIdx.x < n_sel_blocks;

  if (selects) {
    const int seg = blockIdx.x / a.nb, blk = blockIdx.x % a.nb;
    unsigned long long* seg_flags = a.flags + (size_t)seg * a.nb;
    uint32_t* seg_slices = a.slices + (size_t)seg * a.nb * kSelBins;
    uint32_t* seg_cand = a.cand + (size_t)seg * a.n;
    const float* src = a.vals + (long long)seg * a.stride;
    const int base = blk * kEvTile;
    uint32_t key[kEvPerThread];
    bool cand[kEvPerThread];
    {  // a thread owns eight consecutive keys: two 128-bit loads where the row allows them
      const int g0 = base + kEvPerThread * tid;
      float f[kEvPerThread];
      if ((a.stride & 3) == 0 && g0 + kEvPerThread <= a.n) {
        const float4 x = __ldcg(reinterpret_cast<const float4*>(src + g0));
        const float4 y = __ldcg(reinterpret_cast<const float4*>(src + g0) + 1);
        f[0] = x.x; f[1] = x.y; f[2] = x.z; f[3] = x.w;
        f[4] = y.x; f[5] = y.y; f[6] = y.z; f[7] = y.w;
      } else {
#pragma unroll
        for (int j = 0; j < kEvPerThread; ++j) f[j] = g0 + j < a.n ? __ldcg(src + g0 + j) : 0.f;
      }
#pragma unroll
      for (int j = 0; j < kEvPerThread; ++j) {
        cand[j] = g0 + j >= a.lo && g0 + j < a.hi;
        key[j] = cand[j] ? float_to_key(f[j]) : 0u;
      }
    }
    // A: this block's histogram of the top 11 bits, published as its slice
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kEvPerThread; ++j) hist_add(hist, key[j] >> 21, cand[j]);
    __syncthreads();
    for (int i = tid; i < kSelBins; i += kSelThreads) __stcg(seg_slices + (size_t)blk * kSelBins + i, hist[i]);
    publish_phase(seg_flags + blk, a.epoch, 1);
    if (!wait_flags(seg_flags, a.nb, a.expect_extra ? never_set : nullptr, a.epoch, 1, abort_word, a.wait_cycles, 0,
                    a.dev_status))
      return;

    // B: the segment's histogram and the threshold bin; from the slices of the blocks before this
    // one, its offset in the candidate list and the number of keys above the threshold bin
    uint32_t p0 = 0, p1 = 0;   // this thread's two bins summed over the blocks before this one
    const int b0 = kSelBins - 1 - 2 * tid;
    {
      uint32_t s0 = 0, s1 = 0;
#pragma unroll 8
      for (int bb = 0; bb < a.nb; ++bb) {
        const uint32_t v0 = __ldcg(seg_slices + (size_t)bb * kSelBins + b0);
        const uint32_t v1 = __ldcg(seg_slices + (size_t)bb * kSelBins + b0 - 1);
        s0 += v0;
        s1 += v1;
        if (bb < blk) { p0 += v0; p1 += v1; }
      }
      __syncthreads();
      hist[b0] = s0;
      hist[b0 - 1] = s1;
      if (tid == 0) counter = 0;
      __syncthreads();
    }
    uint32_t b1, rem1;
    find_bin_shared(hist, (uint32_t)a.m, scratch, result, b1, rem1);
    const uint32_t n_cand = hist[b1];
    if ((uint32_t)b0 == b1) shared_base = p0;
    if ((uint32_t)(b0 - 1) == b1) shared_base = p1;
    uint32_t gt_before;
    block_excl_scan(((uint32_t)b0 > b1 ? p0 : 0u) + ((uint32_t)(b0 - 1) > b1 ? p1 : 0u), scratch, gt_before);
    const uint32_t cand_base = shared_base;   // candidates of the blocks before this one (the scan synchronised)
    // own keys of the threshold bin go to the candidate list (their order inside it is irrelevant)
#pragma unroll
    for (int j = 0; j < kEvPerThread; ++j)
      if (cand[j] && (key[j] >> 21) == b1) __stcg(seg_cand + cand_base + atomicAdd(&counter, 1u), key[j]);
    publish_phase(seg_flags + blk, a.epoch, 2);
    if (!wait_flags(seg_flags, a.nb, nullptr, a.epoch, 2, abort_word, a.wait_cycles, 0, a.dev_status)) return;

    // C: the remaining 21 bits from the candidate list, in two local passes
    const bool staged = n_cand <= (uint32_t)kEvCandSmem;
    if (staged)
      for (uint32_t i = tid; i < n_cand; i += kSelThreads) cbuf[i] = __ldcg(seg_cand + i);
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    uint32_t eq_before = 0;
    for (uint32_t i0 = 0; i0 < n_cand; i0 += kSelThreads) {   // uniform trip count: every lane calls hist_add
      const uint32_t i = i0 + tid;
      const uint32_t k = i < n_cand ? cand_key(cbuf, seg_cand, staged, i) : 0u;
      hist_add(hist, (k >> 10) & 0x7FFu, i < n_cand);
    }
    __syncthreads();
    uint32_t b2, rem2;
    find_bin_shared(hist, rem1, scratch, result, b2, rem2);
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    for (uint32_t i0 = 0; i0 < n_cand; i0 += kSelThreads) {
      const uint32_t i = i0 + tid;
      const uint32_t k = i < n_cand ? cand_key(cbuf, seg_cand, staged, i) : 0u;
      hist_add(hist, k & 0x3FFu, i < n_cand && ((k >> 10) & 0x7FFu) == b2);
    }
    __syncthreads();
    uint32_t b3, need_eq;
    find_bin_shared(hist, rem2, scratch, result, b3, need_eq);   // bins above 1023 are empty in this pass
    const uint32_t thr = (b1 << 21) | (b2 << 10) | b3;
    {  // candidates of the blocks before this one: above / equal to the threshold
      uint32_t g = 0, e = 0;
      for (uint32_t i = tid; i < cand_base; i += kSelThreads) {
        const uint32_t k = cand_key(cbuf, seg_cand, staged, i);
        g += k > thr;
        e += k == thr;
      }
      uint32_t tg, te;
      block_excl_scan(g, scratch, tg);
      block_excl_scan(e, scratch, te);
      gt_before += tg;
      eq_before += te;
    }
    // ordered write of this block's kept indices: one scan over the threads, then each thread
    // walks its eight consecutive keys
    int32_t* out = a.out + (long long)seg * a.out_stride;
    {
      uint32_t mine = 0;
#pragma unroll
      for (int j = 0; j < kEvPerThread; ++j)
        mine += (cand[j] && key[j] > thr ? 1u : 0u) + (cand[j] && key[j] == thr ? 1u << 16 : 0u);
      uint32_t tt;
      const uint32_t pp = block_excl_scan(mine, scratch, tt);
      uint32_t g_b = gt_before + (pp & 0xFFFFu), e_b = eq_before + (pp >> 16);
#pragma unroll
      for (int j = 0; j < kEvPerThread; ++j) {
        const bool is_gt = cand[j] && key[j] > thr, is_eq = cand[j] && key[j] == thr;
        if (is_gt || (is_eq && e_b < need_eq))
          out[a.lo + g_b + (e_b < need_eq ? e_b : need_eq)] = base + kEvPerThread * tid + j;
        g_b += is_gt;
        e_b += is_eq;
      }
    }
    if (blk == 0) {  // forced head and tail
      for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
      const int tail = a.n - a.hi;
      for (int i = tid; i < tail; i += kSelThreads) out[a.lo + a.m + i] = a.hi + i;
    }
    publish_phase(seg_flags + blk, a.epoch, 3);
  } else if (a.m == 0 && (int)blockIdx.x < a.segs) {
    // nothing to choose (keep all, or forced rows only): the list is the forced head and tail
    int32_t* out = a.out + (long long)blockIdx.x * a.out_stride;
    for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
    const int tail = a.n - a.hi;
    for (int i = tid; i < tail; i += kSelThreads) out[a.lo + i] = a.hi + i;
    publish_phase(a.flags + blockIdx.x, a.epoch, 3);   // no selection blocks in this mode: flag s stands for segment s
  }

  // compaction: wait for every kept list, then stream the rows
  if (a.m > 0) {
    if (!wait_flags(a.flags, n_sel_blocks, nullptr, a.epoch, 3, abort_word, a.wait_cycles, 100, a.dev_status)) return;
  } else {
    if (!wait_flags(a.flags, a.segs, nullptr, a.epoch, 3, abort_word, a.wait_cycles, 100, a.dev_status)) return;
  }
  constexpr int LANES = 4;
  constexpr int ROWS = kSelThreads / LANES;
  const int lane = tid % LANES, sub = tid / LANES;
  if (a.in_place) {   // rows of at most 16 chunks (checked by the launcher): four per lane and tensor
    unsigned long long* gflags = abort_word + 2;
    const int per_wave = (int)gridDim.x * ROWS;
    const int Rw = per_wave / a.segs > 0 ? per_wave / a.segs : 1;   // ranks per segment and wave
    const int waves = (a.n_kept + Rw - 1) / Rw;
    const int item = (int)blockIdx.x * ROWS + sub;
    const int s = item / Rw;
    for (int w = 0; w < waves; ++w) {
      const int rank = w * Rw + item % Rw;
      const bool live = s < a.segs && rank < a.n_kept;
      uint4 kk[4], vv[4];
      float sc = 0.f;
      int32_t ps = 0;
      long long dn = 0;
      if (live) {
        const int j = __ldcg(a.out + (long long)s * a.out_stride + rank);
        const long long so = ((long long)s * a.cap_src + j) * a.vec;
        dn = ((long long)s * a.cap_dst + rank) * a.vec;
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (lane + u * LANES < a.vec) {
            kk[u] = __ldcg(a.k_src + so + lane + u * LANES);
            vv[u] = __ldcg(a.v_src + so + lane + u * LANES);
          }
        if (lane == 0) {
          sc = __ldcg(a.score_src + (long long)s * a.cap_src + j);
          if (a.pos_dst) ps = __ldcg(a.pos_src + (long long)s * a.cap_src + j);
        }
      }
      __threadfence();   // every thread's loads of this wave have been performed before the block says so
      publish_phase(gflags + blockIdx.x, a.epoch, 4 + w);
      if (!wait_flags(gflags, (int)gridDim.x, nullptr, a.epoch, 4 + w, abort_word, a.wait_cycles, 0, a.dev_status)) return;
      if (live) {
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (lane + u * LANES < a.vec) {
            __stcg(a.k_dst + dn + lane + u * LANES, kk[u]);
            __stcg(a.v_dst + dn + lane + u * LANES, vv[u]);
          }
        if (lane == 0) {
          a.score_dst[(long long)s * a.cap_dst + rank] = sc;
          if (a.pos_dst) a.pos_dst[(long long)s * a.cap_dst + rank] = ps;
        }
      }
    }
    return;
  }
  const long long total = (long long)a.segs * a.n_kept;
  for (long long r = (long long)blockIdx.x * ROWS + sub; r < total; r += (long long)gridDim.x * ROWS) {
    const int s = (int)(r / a.n_kept), rank = (int)(r % a.n_kept);
    const int j = __ldcg(a.out + (long long)s * a.out_stride + rank);
    const long long so = ((long long)s * a.cap_src + j) * a.vec, dn = ((long long)s * a.cap_dst + rank) * a.vec;
    for (int c = lane; c < a.vec; c += 4 * LANES) {   // up to four loads of K and of V in flight per thread
      uint4 kk[4], vv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c + u * LANES < a.vec) {
          kk[u] = __ldcs(a.k_src + so + c + u * LANES);
          vv[u] = __ldcs(a.v_src + so + c + u * LANES);
        }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c + u * LANES < a.vec) {
          __stcs(a.k_dst + dn + c + u * LANES, kk[u]);
          __stcs(a.v_dst + dn + c + u * LANES, vv[u]);
        }
    }
    if (lane == 0) {
      a.score_dst[(long long)s * a.cap_dst + rank] = __ldcg(a.score_src + (long long)s * a.cap_src + j);
      if (a.pos_dst) a.pos_dst[(long long)s * a.cap_dst + rank] = a.pos_src[(long long)s * a.cap_src + j];
    }
  }
}

// Blocks of evict_fused_kernel that can be resident at once on the current device (0 if unknown).
inline int evict_fused_capacity() {
  constexpr int kMaxDevices = 64;
  static int cache[kMaxDevices] = {0};
  int dev = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  if (cache[dev] <= 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, evict_fused_kernel, kSelThreads, 0) != cudaSuccess)
      return 0;
    cache[dev] = per_sm * num_sms();
  }
  return cache[dev];
}

// Process-wide source of epochs: never 0, unique per call, salted so that memory left behind by
// another process cannot carry the same value.
unsigned long long next_epoch();

// True if the one-launch form applies to this shape on this device.
inline bool evict_fused_applies(int segs, int n, size_t workspace_bytes, size_t kept_bytes) {
  const EvictFusedLayout L = evict_fused_layout(segs, n);
  if (L.nb > kEvMaxBlocksPerSeg) return false;
  if (workspace_bytes < L.total + kept_bytes) return false;
  const int capacity = evict_fused_capacity() < kEvMaxGrid ? evict_fused_capacity() : kEvMaxGrid;
  return (long long)segs * L.nb <= capacity;
}

// In-place compaction holds a wave of rows in registers: rows of at most 256 bytes, and few enough
// waves for the phase field.
inline bool evict_fused_in_place_ok(int segs, int n_kept, int vec, int grid) {
  if (vec > 16) return false;
  const int per_wave = grid * (kSelThreads / 4);
  const int Rw = per_wave / segs > 0 ? per_wave / segs : 1;
  return (n_kept + Rw - 1) / Rw <= kEvMaxWaves;
}

inline int evict_fused_grid(const EvictFusedArgs& a) {
  const int capacity = evict_fused_capacity() < kEvMaxGrid ? evict_fused_capacity() : kEvMaxGrid;
  const long long rows = (long long)a.segs * a.n_kept;
  long long want = (rows + (kSelThreads / 4) - 1) / (kSelThreads / 4);   // blocks that find a row to move
  const long long sel_blocks = (long long)a.segs * a.nb;
  if (want < sel_blocks) want = sel_blocks;
  if (want < a.segs) want = a.segs;
  return (int)(want < capacity ? want : capacity);
}

inline int launch_evict_fused(EvictFusedArgs a, cudaStream_t st) {
  const int grid = evict_fused_grid(a);
  if (a.in_place && !evict_fused_in_place_ok(a.segs, a.n_kept, a.vec, grid)) return REFORM_ERR_UNSUPPORTED;
  void* args[] = {&a};
  cudaError_t e = cudaLaunchCooperativeKernel((const void*)evict_fused_kernel, dim3(grid), dim3(kSelThreads), args, 0, st);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return REFORM_ERR_CUDA;
  }
  count_launch();
  return check_launch();
}

}  // namespace reform
