// Deterministic segmented top-m selection used by the cache compression
// (Sec. 3.1) and by the token selection of the gather phase (Sec. 3.3).
//
// For each segment: of the candidates [lo, hi) choose the m largest values
// under the total order (value descending, index ascending) and write, in
// ascending index order, [0, lo) ++ chosen ++ [hi, n).  The k-th key is found
// by a most-significant-digit radix select over the order-preserving uint32
// image of the floats (11 + 11 + 10 bits, one histogram pass each); equal keys
// are admitted lowest index first through an ordered prefix count, so there is
// no atomics-dependent ordering anywhere and the result is bit-reproducible.
//
// The optional pooling (Sec. 3.3: max over the 2r+1 adjacent tokens) is fused
// into the first histogram pass: a grouped sliding maximum in shared memory.
#pragma once

#include "common.cuh"

namespace reform {

constexpr int kSelThreads = 1024;
constexpr int kSelPerThread = 4;
constexpr int kSelTile = kSelThreads * kSelPerThread;  // elements per block
constexpr int kSelBins = 2048;
constexpr int kSelMaxRadius = 2048;  // pool_window <= 4097

struct SelState {      // per segment, in the workspace
  uint32_t prefix;     // key bits fixed so far (after the last pass: the threshold key)
  uint32_t remaining;  // how many of the still-undecided candidates must be taken
  uint32_t done[4];    // blocks finished, per pass (3 histogram passes + the count pass)
  uint32_t pad[2];
};

struct SelLayout {  // offsets into the workspace, per call
  size_t state, hist, ctl, zero_bytes, blockcnt, total;  // [state, hist, ctl] are contiguous
  int blocks_per_seg;
};

inline SelLayout sel_layout(int segs, long long n_max) {
  SelLayout L;
  L.blocks_per_seg = (int)((n_max + kSelTile - 1) / kSelTile);
  if (L.blocks_per_seg < 1) L.blocks_per_seg = 1;
  size_t off = 0;
  L.state = off;
  off += align_up(sizeof(SelState) * segs, 256);
  L.hist = off;
  off += align_up(sizeof(uint32_t) * 3 * kSelBins * segs, 256);
  L.ctl = off;
  off += align_up(16 * (size_t)segs, 256);
  L.zero_bytes = off;  // everything up to here is cleared at the start of a fused launch
  L.blockcnt = off;
  off += align_up(sizeof(uint2) * 2 * (size_t)L.blocks_per_seg * segs, 256);
  L.total = off;
  return L;
}

struct SelArgs {
  const float* vals;     // candidate values; element (seg, i) at vals[seg * stride + i]
  long long stride;
  int n, lo, hi, m;      // segment length, candidate range, number to choose
  int32_t* out;          // [segs, out_stride]
  int out_stride;
  SelState* state;
  uint32_t* hist;        // [segs, 3, kSelBins]
  uint2* blockcnt;       // [segs, 2, blocks_per_seg]: counts then exclusive offsets
  int blocks_per_seg;
};

__global__ void sel_init_kernel(SelArgs a, int segs) {
  int seg = blockIdx.x;
  if (seg >= segs) return;
  uint32_t* h = a.hist + (size_t)seg * 3 * kSelBins;
  for (int i = threadIdx.x; i < 3 * kSelBins; i += blockDim.x) h[i] = 0;
  if (threadIdx.x == 0) {
    SelState s;
    s.prefix = 0;
    s.remaining = (uint32_t)a.m;
    s.done[0] = s.done[1] = s.done[2] = s.done[3] = 0;
    s.pad[0] = s.pad[1] = 0;
    a.state[seg] = s;
  }
}

// Block-wide exclusive scan of one uint per thread (1024 threads); returns the
// exclusive prefix and, through total, the block sum.  scratch: 33 uints.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* scratch, uint32_t& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) scratch[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = scratch[lane];
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    scratch[lane] = winc - w;
    if (lane == 31) scratch[32] = winc;
  }
  __syncthreads();
  uint32_t res = scratch[warp] + inc - v;
  total = scratch[32];
  __syncthreads();
  return res;
}

// Histogram increment.  When every participating lane of the warp hits the same bin (constant
// or heavily tied scores, where same-address atomics would serialise) the warp issues one atomic
// for all of them; otherwise each lane adds its own.  Every lane of the warp must call this
// (valid = false to sit out).
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t bin, bool valid) {
  const unsigned active = __ballot_sync(0xffffffffu, valid);
  if (valid) {
    int same;
    __match_all_sync(active, bin, &same);
    if (!same) atomicAdd(&hist[bin], 1u);
    else if ((threadIdx.x & 31) == (unsigned)(__ffs(active) - 1)) atomicAdd(&hist[bin], (uint32_t)__popc(active));
  }
}

// Executed by the last block of a histogram pass: walk the bins from the top
// until the running count reaches `remaining`; fix that digit.
__device__ void sel_find_bin(SelState* st, const uint32_t* hist, int shift, uint32_t* scratch) {
  const uint32_t remaining = st->remaining;
  // thread t owns bins (2047 - 2t) and (2046 - 2t): descending order
  int b0 = kSelBins - 1 - 2 * (int)threadIdx.x;
  uint32_t c0 = __ldcg(hist + b0), c1 = __ldcg(hist + b0 - 1);
  uint32_t total;
  uint32_t before = block_excl_scan(c0 + c1, scratch, total);
  if (before < remaining && remaining <= before + c0 + c1) {
    int bin;
    uint32_t rem;
    if (remaining <= before + c0) {
      bin = b0;
      rem = remaining - before;
    } else {
      bin = b0 - 1;
      rem = remaining - before - c0;
    }
    st->prefix |= (uint32_t)bin << shift;
    st->remaining = rem;
  } else if (remaining == 0 && threadIdx.x == 0) {
    st->prefix |= (uint32_t)(kSelBins - 1) << shift;  // nothing to take: threshold above every key
  }
}

__device__ __forceinline__ void sel_pass_params(int pass, int& shift, uint32_t& digit_mask,
                                                uint32_t& prefix_mask) {
  if (pass == 0) { shift = 21; digit_mask = 0x7FFu; prefix_mask = 0u; }
  else if (pass == 1) { shift = 10; digit_mask = 0x7FFu; prefix_mask = 0xFFE00000u; }
  else { shift = 0; digit_mask = 0x3FFu; prefix_mask = 0xFFFFFC00u; }
}

// Bin walk over a shared-memory histogram of kSelBins bins from the top: the bin in which the
// running count reaches `remaining`, and how many are still to take inside it.  All threads get
// the same answer.  result: 2 uints of shared memory; scratch: 33.
__device__ __forceinline__ void find_bin_shared(const uint32_t* hist, uint32_t remaining, uint32_t* scratch,
                                                uint32_t* result, uint32_t& bin_out, uint32_t& rem_out) {
  const int b0 = kSelBins - 1 - 2 * (int)threadIdx.x;
  const uint32_t c0 = hist[b0], c1 = hist[b0 - 1];
  uint32_t total;
  const uint32_t before = block_excl_scan(c0 + c1, scratch, total);
  if (threadIdx.x == 0) { result[0] = kSelBins - 1; result[1] = 0; }
  __syncthreads();
  if (before < remaining && remaining <= before + c0 + c1) {
    if (remaining <= before + c0) { result[0] = b0; result[1] = remaining - before; }
    else { result[0] = b0 - 1; result[1] = remaining - before - c0; }
  }
  __syncthreads();
  bin_out = result[0];
  rem_out = result[1];
  __syncthreads();
}

// Pools the raw token scores of one block's tile (Sec. 3.3).  tile: pool_tile_floats(tile_len,
// radius) floats of shared memory, 16-byte aligned.  On return the pooled score of the block's
// element i (0 <= i < tile_len, token base + i < n) is available through pool_result().
//
// mode 0, maximum over the clipped window [t - r, t + r]: the tile (with its halo of r on either
// side, -inf outside the bank) is cut into aligned groups of eight; one pass leaves, per group, the
// running maximum from its left end, the running maximum from its right end and the group's
// maximum.  A window is then a suffix of its first group, a prefix of its last group and whole
// groups in between: pooled = max(suffix[t - r], prefix[t + r], the groups strictly between).
// One barrier, and r / 4 + 2 reads per element whatever the window.  Windows of fewer than nine
// tokens are read directly.
// mode 1, mean over the clipped window: direct summation in ascending token order.
constexpr int kPoolGroup = 8;

__host__ __device__ inline size_t pool_tile_floats(int tile_len, int radius) {
  const size_t span8 = align_up((size_t)tile_len + 2 * (size_t)radius, kPoolGroup);
  return 2 * span8 + span8 / kPoolGroup;
}

struct PoolTile {
  const float* x;     // mode 1 and short windows: the raw scores of the tile with its halo
  const float* pre;   // grouped maximum: running maximum from the left end of each group
  const float* suf;   //                  running maximum from the right end of each group
  const float* grp;   //                  each group's maximum
  int radius, mode;
  bool grouped;
  long long base;     // first token of the block's tile
  int n;
};

__device__ __forceinline__ PoolTile pool_prepare(float* tile, const float* __restrict__ src, long long base, int n,
                                                 int radius, int mode, int tile_len = kSelTile) {
  const int tid = threadIdx.x;
  const int span8 = (int)align_up((size_t)tile_len + 2 * (size_t)radius, kPoolGroup);
  float* x = tile;
  float* pre = tile + span8;
  float* grp = tile + 2 * span8;
  PoolTile p;
  p.radius = radius;
  p.mode = mode;
  p.grouped = mode == 0 && radius >= kPoolGroup / 2;   // the window then always reaches into a second group
  p.base = base;
  p.n = n;
  p.x = x;
  p.pre = pre;
  p.suf = x;
  p.grp = grp;
  // eight independent loads per thread in flight at a time
  for (int i0 = 0; i0 < span8; i0 += 8 * kSelThreads) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kSelThreads + tid;
      const long long g = base - radius + i;
      v[u] = (i < span8 && g >= 0 && g < n) ? __ldcg(src + g) : -INFINITY;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kSelThreads + tid;
      if (i < span8) x[i] = v[u];
    }
  }
  __syncthreads();
  if (p.grouped) {
    for (int g = tid; g < span8 / kPoolGroup; g += kSelThreads) {
      float4* xg = reinterpret_cast<float4*>(x + kPoolGroup * g);
      const float4 a = xg[0], b = xg[1];
      float4 pa, pb, sa, sb;
      pa.x = a.x;                 pa.y = fmaxf(pa.x, a.y);  pa.z = fmaxf(pa.y, a.z);  pa.w = fmaxf(pa.z, a.w);
      pb.x = fmaxf(pa.w, b.x);    pb.y = fmaxf(pb.x, b.y);  pb.z = fmaxf(pb.y, b.z);  pb.w = fmaxf(pb.z, b.w);
      sb.w = b.w;                 sb.z = fmaxf(sb.w, b.z);  sb.y = fmaxf(sb.z, b.y);  sb.x = fmaxf(sb.y, b.x);
      sa.w = fmaxf(sb.x, a.w);    sa.z = fmaxf(sa.w, a.z);  sa.y = fmaxf(sa.z, a.y);  sa.x = fmaxf(sa.y, a.x);
      float4* pg = reinterpret_cast<float4*>(pre + kPoolGroup * g);
      pg[0] = pa;
      pg[1] = pb;
      xg[0] = sa;   // the suffix maxima replace the group's raw scores (nobody else reads this group's x)
      xg[1] = sb;
      grp[g] = pb.w;
    }
    __syncthreads();
  }
  return p;
}

// pooled score of the tile's element i (token base + i, which must be < n)
__device__ __forceinline__ float pool_result(const PoolTile& p, int i) {
  if (p.mode == 0) {
    const int L = i, R = i + 2 * p.radius;   // the window in tile coordinates (the tile starts r before its first element)
    if (!p.grouped) {
      float m = p.x[L];
      for (int u = L + 1; u <= R; ++u) m = fmaxf(m, p.x[u]);
      return m;
    }
    float m = fmaxf(p.suf[L], p.pre[R]);
    for (int g = L / kPoolGroup + 1; g < R / kPoolGroup; ++g) m = fmaxf(m, p.grp[g]);
    return m;
  }
  const long long g = p.base + i;
  const int lo = (int)(g - p.radius < 0 ? -g : -p.radius);                  // offsets of the clipped window
  const int hi = (int)(g + p.radius > p.n - 1 ? p.n - 1 - g : p.radius);
  float sum = 0.f;
  for (int u = lo; u <= hi; ++u) sum += p.x[i + p.radius + u];
  return sum / (float)(hi - lo + 1);
}

// The same for the eight consecutive elements i0 .. i0 + 7 (i0 a multiple of eight, every token
// < n or its result unused): the eight windows start in one group and end in one or two, so the
// whole groups they all cover are read once.
__device__ __forceinline__ void pool_result8(const PoolTile& p, int i0, float (&out)[8]) {
  if (!p.grouped) {
#pragma unroll
    for (int j = 0; j < 8; ++j) out[j] = pool_result(p, i0 + j);
    return;
  }
  const int gl = i0 / kPoolGroup;                       // first group of every window
  const int q = (i0 + 2 * p.radius) / kPoolGroup;       // last group of window j: q, or q + 1 from j = 8 - rem on
  const int rem = (i0 + 2 * p.radius) % kPoolGroup;
  float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
  int g = gl + 1;
  for (; g + 3 < q; g += 4) {
    c0 = fmaxf(c0, p.grp[g]);
    c1 = fmaxf(c1, p.grp[g + 1]);
    c2 = fmaxf(c2, p.grp[g + 2]);
    c3 = fmaxf(c3, p.grp[g + 3]);
  }
  for (; g < q; ++g) c0 = fmaxf(c0, p.grp[g]);
  const float core = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));       // groups gl + 1 .. q - 1
  const float core_q = q > gl ? fmaxf(core, p.grp[q]) : core;   // and group q, for the windows that end in q + 1
  const float4 sa = *reinterpret_cast<const float4*>(p.suf + i0), sb = *reinterpret_cast<const float4*>(p.suf + i0 + 4);
  const float sfx[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
#pragma unroll
  for (int j = 0; j < 8; ++j)
    out[j] = fmaxf(fmaxf(sfx[j], p.pre[i0 + 2 * p.radius + j]), rem + j < kPoolGroup ? core : core_q);
}

// One histogram pass.  POOL (pass 0 only): vals_in holds the raw token scores
// ts; the block computes pooled[i] = max ts[i-r .. i+r] (clipped), writes it
// to pooled_out, and histograms that.
template <bool POOL>
__global__ void __launch_bounds__(kSelThreads)
sel_hist_kernel(SelArgs a, int pass, const float* __restrict__ ts, float* __restrict__ pooled_out,
                int radius, int pool_mode) {
  extern __shared__ __align__(16) float tile[];  // POOL: pool_tile_floats(kSelTile, radius) floats
  __shared__ uint32_t hist[kSelBins];
  __shared__ uint32_t scratch[33];
  __shared__ bool is_last;
  const int seg = blockIdx.y;
  const int tid = threadIdx.x;
  int shift;
  uint32_t dmask, pmask;
  sel_pass_params(pass, shift, dmask, pmask);
  for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
  SelState* st = a.state + seg;
  const uint32_t prefix = (pass == 0) ? 0u : __ldcg(&st->prefix);
  const long long base = (long long)blockIdx.x * kSelTile;  // offset inside [0, n)
  if (POOL) {
    // tile covers ts[base - radius, base + kSelTile + radius)
    const PoolTile pt = pool_prepare(tile, ts + (long long)seg * a.stride, base, a.n, radius, pool_mode);
    float* dst = pooled_out + (long long)seg * a.stride;
    for (int j = 0; j < kSelPerThread; ++j) {
      int i = j * kSelThreads + tid;
      long long g = base + i;
      const float v = g < a.n ? pool_result(pt, i) : 0.f;
      if (g < a.n) dst[g] = v;
      hist_add(hist, float_to_key(v) >> shift, g >= a.lo && g < a.hi);  // every lane calls; hi <= n
    }
  } else {
    __syncthreads();
    const float* src = a.vals + (long long)seg * a.stride;
    for (int j = 0; j < kSelPerThread; ++j) {
      long long g = base + j * kSelThreads + tid;
      const bool in = g >= a.lo && g < a.hi;
      const uint32_t key = in ? float_to_key(src[g]) : 0u;
      hist_add(hist, (key >> shift) & dmask, in && (key & pmask) == prefix);
    }
  }
  __syncthreads();
  uint32_t* gh = a.hist + ((size_t)seg * 3 + pass) * kSelBins;
  for (int i = tid; i < kSelBins; i += kSelThreads) {
    uint32_t c = hist[i];
    if (c) atomicAdd(gh + i, c);
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&st->done[pass], 1u) == gridDim.x - 1);
  __syncthreads();
  if (is_last) {
    __threadfence();
    sel_find_bin(st, gh, shift, scratch);
  }
}

// Count pass: per block, how many candidates lie above the threshold key and
// how many equal it; the last block turns the counts into exclusive offsets.
__global__ void __launch_bounds__(kSelThreads) sel_count_kernel(SelArgs a) {
  __shared__ uint32_t scratch[33];
  __shared__ bool is_last;
  const int seg = blockIdx.y, tid = threadIdx.x;
  SelState* st = a.state + seg;
  const uint32_t thr = __ldcg(&st->prefix);
  const float* src = a.vals + (long long)seg * a.stride;
  const long long base = (long long)blockIdx.x * kSelTile;
  uint32_t gt = 0, eq = 0;
  for (int j = 0; j < kSelPerThread; ++j) {
    long long g = base + j * kSelThreads + tid;
    if (g >= a.lo && g < a.hi) {
      uint32_t key = float_to_key(src[g]);
      gt += key > thr;
      eq += key == thr;
    }
  }
  uint32_t tot;  // both counts are <= kSelTile < 2^16: one scan of (gt | eq << 16) serves both
  block_excl_scan(gt | (eq << 16), scratch, tot);
  const uint32_t tot_gt = tot & 0xFFFFu, tot_eq = tot >> 16;
  uint2* cnt = a.blockcnt + (size_t)seg * 2 * a.blocks_per_seg;
  uint2* off = cnt + a.blocks_per_seg;
  if (tid == 0) {
    cnt[blockIdx.x] = make_uint2(tot_gt, tot_eq);
    __threadfence();
    is_last = (atomicAdd(&st->done[3], 1u) == gridDim.x - 1);
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    // exclusive scan over the blocks of this segment, kSelThreads at a time
    uint32_t run_gt = 0, run_eq = 0;
    for (int b0 = 0; b0 < a.blocks_per_seg; b0 += kSelThreads) {
      int b = b0 + tid;
      uint2 c = (b < a.blocks_per_seg) ? __ldcg(cnt + b) : make_uint2(0, 0);
      uint32_t tg, te;
      uint32_t eg = block_excl_scan(c.x, scratch, tg);
      uint32_t ee = block_excl_scan(c.y, scratch, te);
      if (b < a.blocks_per_seg) off[b] = make_uint2(run_gt + eg, run_eq + ee);
      run_gt += tg;
      run_eq += te;
    }
  }
}

// Write pass: ordered compaction.  A candidate is chosen if its key is above
// the threshold, or equals it and fewer than need_eq equal keys precede it.
__global__ void __launch_bounds__(kSelThreads) sel_write_kernel(SelArgs a) {
  __shared__ uint32_t scratch[33];
  const int seg = blockIdx.y, tid = threadIdx.x;
  const SelState* st = a.state + seg;
  const uint32_t thr = __ldcg(&st->prefix);
  const uint32_t need_eq = __ldcg(&st->remaining);
  const float* src = a.vals + (long long)seg * a.stride;
  int32_t* out = a.out + (long long)seg * a.out_stride;
  const uint2 boff = __ldcg(a.blockcnt + (size_t)seg * 2 * a.blocks_per_seg + a.blocks_per_seg + blockIdx.x);
  const long long base = (long long)blockIdx.x * kSelTile;
  uint32_t run_gt = boff.x, run_eq = boff.y;
  for (int j = 0; j < kSelPerThread; ++j) {
    long long g = base + j * kSelThreads + tid;
    uint32_t is_gt = 0, is_eq = 0;
    if (g >= a.lo && g < a.hi) {
      uint32_t key = float_to_key(src[g]);
      is_gt = key > thr;
      is_eq = key == thr;
    }
    uint32_t tt;
    const uint32_t pp = block_excl_scan(is_gt | (is_eq << 16), scratch, tt);
    const uint32_t tg = tt & 0xFFFFu, te = tt >> 16;
    uint32_t gt_before = run_gt + (pp & 0xFFFFu), eq_before = run_eq + (pp >> 16);
    if (is_gt || (is_eq && eq_before < need_eq)) {
      uint32_t pos = a.lo + gt_before + (eq_before < need_eq ? eq_before : need_eq);
      out[pos] = (int32_t)g;
    }
    run_gt += tg;
    run_eq += te;
  }
  if (blockIdx.x == 0) {  // forced head and tail
    for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
    int tail = a.n - a.hi;
    for (int i = tid; i < tail; i += kSelThreads) out[a.lo + a.m + i] = a.hi + i;
  }
}


// ---------------------------------------------------------------------------
// Single-launch form of the same selection for inputs whose blocks are all
// resident at once (cooperative launch): the three histogram passes, the count
// and the ordered write run in one kernel, separated by per-segment barriers
// over a global counter, and every thread keeps its four keys in registers
// from the first pass to the last.  Each block re-derives the digit decisions
// from the global histograms itself, so no block depends on another block's
// private state.  The barrier wait is bounded: a block that gives up sets
// REFORM_DEV_TIMEOUT in *dev_status and the launch winds down.
// ---------------------------------------------------------------------------
struct SelFusedCtl {   // per segment, zeroed before the launch
  uint32_t arrived;    // barrier counter (monotonic)
  uint32_t abort;
  uint32_t pad[2];
};

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ bool sel_seg_barrier(SelFusedCtl* ctl, uint32_t expected, int32_t* dev_status) {
  __shared__ int failed;
  __syncthreads();
  if (threadIdx.x == 0) {
    failed = 0;
    __threadfence();
    atomicAdd(&ctl->arrived, 1u);
    const long long t0 = clock64();
    while (ld_acquire_u32(&ctl->arrived) < expected) {  // plain acquire loads: polling with atomics would serialise in L2
      if (*reinterpret_cast<volatile uint32_t*>(&ctl->abort) || clock64() - t0 > 400000000LL) {
        atomicExch(&ctl->abort, 1u);
        report_device_error(dev_status, REFORM_DEV_TIMEOUT);
        failed = 1;
        break;
      }
    }
    __threadfence();
  }
  __syncthreads();
  return failed == 0;
}

// Walk the 2048 bins of one pass from the top; every thread returns the same (bin, remaining).
__device__ __forceinline__ void sel_find_bin_local(const uint32_t* hist, uint32_t remaining, uint32_t* scratch,
                                                   uint32_t* result, uint32_t& bin_out, uint32_t& rem_out) {
  int b0 = kSelBins - 1 - 2 * (int)threadIdx.x;
  uint32_t c0 = __ldcg(hist + b0), c1 = __ldcg(hist + b0 - 1);
  uint32_t total;
  uint32_t before = block_excl_scan(c0 + c1, scratch, total);
  if (threadIdx.x == 0) { result[0] = kSelBins - 1; result[1] = 0; }  // remaining == 0: above every key
  __syncthreads();
  if (before < remaining && remaining <= before + c0 + c1) {
    if (remaining <= before + c0) { result[0] = b0; result[1] = remaining - before; }
    else { result[0] = b0 - 1; result[1] = remaining - before - c0; }
  }
  __syncthreads();
  bin_out = result[0];
  rem_out = result[1];
  __syncthreads();
}

// Two blocks per SM (32 registers per thread): the cooperative launch has to hold all blocks of the
// call at once, 256 of them for a bank of 2^20 tokens.
template <bool POOL>
__global__ void __launch_bounds__(kSelThreads, 2)
sel_fused_kernel(SelArgs a, SelFusedCtl* ctl_all, const float* __restrict__ ts,
                 float* __restrict__ pooled_out, int radius, int pool_mode, int32_t* dev_status) {
  extern __shared__ __align__(16) float tile[];  // POOL: pool_tile_floats(kSelTile, radius) floats
  __shared__ uint32_t hist[kSelBins];
  __shared__ uint32_t scratch[33];
  __shared__ uint32_t result[2];
  const int seg = blockIdx.y, tid = threadIdx.x;
  const uint32_t nblk = gridDim.x;
  SelFusedCtl* ctl = ctl_all + seg;
  const long long base = (long long)blockIdx.x * kSelTile;
  uint32_t key[kSelPerThread];
  bool cand[kSelPerThread];

  if (POOL) {
    const PoolTile pt = pool_prepare(tile, ts + (long long)seg * a.stride, base, a.n, radius, pool_mode);
    float* dst = pooled_out + (long long)seg * a.stride;
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j) {
      int i = j * kSelThreads + tid;
      long long g = base + i;
      cand[j] = g >= a.lo && g < a.hi;
      key[j] = 0;
      if (g < a.n) {
        float v = pool_result(pt, i);
        dst[g] = v;
        key[j] = float_to_key(v);
      }
    }
  } else {
    const float* src = a.vals + (long long)seg * a.stride;
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j) {
      long long g = base + j * kSelThreads + tid;
      cand[j] = g >= a.lo && g < a.hi;
      key[j] = cand[j] ? float_to_key(src[g]) : 0u;
    }
  }

  uint32_t prefix = 0, remaining = (uint32_t)a.m;
  uint32_t phase = 0;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    int shift;
    uint32_t dmask, pmask;
    sel_pass_params(pass, shift, dmask, pmask);
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kSelPerThread; ++j)
      hist_add(hist, (key[j] >> shift) & dmask, cand[j] && (key[j] & pmask) == prefix);
    __syncthreads();
    uint32_t* gh = a.hist + ((size_t)seg * 3 + pass) * kSelBins;
    for (int i = tid; i < kSelBins; i += kSelThreads) {
      uint32_t c = hist[i];
      if (c) atomicAdd(gh + i, c);
    }
    if (!sel_seg_barrier(ctl, ++phase * nblk, dev_status)) return;
    uint32_t bin, rem;
    sel_find_bin_local(gh, remaining, scratch, result, bin, rem);
    prefix |= bin << shift;
    remaining = rem;
  }
  const uint32_t thr = prefix, need_eq = remaining;

  // per-block counts in index order, then offsets from the blocks before this one
  uint32_t is_gt[kSelPerThread], is_eq[kSelPerThread];
  uint32_t gt = 0, eq = 0;
#pragma unroll
  for (int j = 0; j < kSelPerThread; ++j) {
    is_gt[j] = cand[j] && key[j] > thr;
    is_eq[j] = cand[j] && key[j] == thr;
    gt += is_gt[j];
    eq += is_eq[j];
  }
  uint32_t tot;  // both counts are <= kSelTile < 2^16: one scan of (gt | eq << 16) serves both
  block_excl_scan(gt | (eq << 16), scratch, tot);
  const uint32_t tot_gt = tot & 0xFFFFu, tot_eq = tot >> 16;
  uint2* cnt = a.blockcnt + (size_t)seg * 2 * a.blocks_per_seg;
  if (tid == 0) cnt[blockIdx.x] = make_uint2(tot_gt, tot_eq);
  if (!sel_seg_barrier(ctl, ++phase * nblk, dev_status)) return;
  uint32_t pg = 0, pe = 0;
  for (int bb = tid; bb < (int)blockIdx.x; bb += kSelThreads) {
    uint2 c = __ldcg(cnt + bb);
    pg += c.x;
    pe += c.y;
  }
  uint32_t run_gt, run_eq, dummy;
  block_excl_scan(pg, scratch, run_gt);
  block_excl_scan(pe, scratch, run_eq);
  (void)dummy;

  int32_t* out = a.out + (long long)seg * a.out_stride;
#pragma unroll
  for (int j = 0; j < kSelPerThread; ++j) {
    uint32_t tt;
    const uint32_t pp = block_excl_scan(is_gt[j] | (is_eq[j] << 16), scratch, tt);
    const uint32_t tg = tt & 0xFFFFu, te = tt >> 16;
    uint32_t gt_before = run_gt + (pp & 0xFFFFu), eq_before = run_eq + (pp >> 16);
    if (is_gt[j] || (is_eq[j] && eq_before < need_eq)) {
      uint32_t pos = a.lo + gt_before + (eq_before < need_eq ? eq_before : need_eq);
      out[pos] = (int32_t)(base + j * kSelThreads + tid);
    }
    run_gt += tg;
    run_eq += te;
  }
  if (blockIdx.x == 0) {
    for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
    int tail = a.n - a.hi;
    for (int i = tid; i < tail; i += kSelThreads) out[a.lo + a.m + i] = a.hi + i;
  }
}

// Enqueue the whole selection.  If ts != nullptr the first pass pools ts with
// the given radius into pooled (which must then be a.vals).

// ---------------------------------------------------------------------------
// One block per segment, used when a call batches many short segments (cache
// compression of many layers / sequences / KV heads at once, each up to 64K
// keys): the whole selection is block-local -- the
// three digit passes histogram in shared memory, the digit decision is made by
// the block itself, and the ordered write walks the segment once more with
// warp ballots (each warp owns a contiguous range, so ranks come from popc on
// ballot masks and a single scan over the 32 warp totals).  No global atomics,
// no grid-wide waits, nothing to initialise; segments run in parallel.
// ---------------------------------------------------------------------------
constexpr int kSelBlockMaxN = 65536;
constexpr int kSelBlockUnroll = 8;
constexpr int kSelBlockMinSegs = 48;  // fewer segments than this: spread each one over several blocks instead

__global__ void __launch_bounds__(kSelThreads) sel_block_kernel(SelArgs a) {
  __shared__ uint32_t hist[kSelBins];
  __shared__ uint32_t scratch[33];
  __shared__ uint32_t result[2];
  __shared__ uint32_t warp_gt[32], warp_eq[32];
  const int seg = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* src = a.vals + (long long)seg * a.stride;
  int32_t* out = a.out + (long long)seg * a.out_stride;
  const int ncand = a.hi - a.lo;
  uint32_t prefix = 0, remaining = (uint32_t)a.m;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    int shift;
    uint32_t dmask, pmask;
    sel_pass_params(pass, shift, dmask, pmask);
    for (int i = tid; i < kSelBins; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    // uniform trip count (every lane calls hist_add); eight independent loads per thread in flight
    for (int i0 = 0; i0 < ncand; i0 += kSelBlockUnroll * kSelThreads) {
      uint32_t key[kSelBlockUnroll];
#pragma unroll
      for (int u = 0; u < kSelBlockUnroll; ++u) {
        const int i = i0 + u * kSelThreads + tid;
        key[u] = (i < ncand) ? float_to_key(__ldg(src + a.lo + i)) : 0u;
      }
#pragma unroll
      for (int u = 0; u < kSelBlockUnroll; ++u) {
        const bool in = i0 + u * kSelThreads + tid < ncand;
        hist_add(hist, (key[u] >> shift) & dmask, in && (key[u] & pmask) == prefix);
      }
    }
    __syncthreads();
    int b0 = kSelBins - 1 - 2 * tid;
    uint32_t c0 = hist[b0], c1 = hist[b0 - 1];
    uint32_t total;
    uint32_t before = block_excl_scan(c0 + c1, scratch, total);
    if (tid == 0) { result[0] = kSelBins - 1; result[1] = 0; }
    __syncthreads();
    if (before < remaining && remaining <= before + c0 + c1) {
      if (remaining <= before + c0) { result[0] = b0; result[1] = remaining - before; }
      else { result[0] = b0 - 1; result[1] = remaining - before - c0; }
    }
    __syncthreads();
    prefix |= result[0] << shift;
    remaining = result[1];
    __syncthreads();
  }
  const uint32_t thr = prefix, need_eq = remaining;
  // ordered write: warp w owns candidates [w * per_warp, (w + 1) * per_warp)
  constexpr int kStep = 32 * kSelBlockUnroll;
  const int per_warp = ((ncand + 31) / 32 + kStep - 1) / kStep * kStep;  // multiple of 32 * unroll
  const int w0 = warp * per_warp;
  uint32_t gt = 0, eq = 0;
  for (int i0 = 0; i0 < per_warp; i0 += kStep) {
    uint32_t key[kSelBlockUnroll];
#pragma unroll
    for (int u = 0; u < kSelBlockUnroll; ++u) {
      const int i = w0 + i0 + 32 * u + lane;
      key[u] = (i < ncand) ? float_to_key(__ldg(src + a.lo + i)) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kSelBlockUnroll; ++u) {
      const bool in = w0 + i0 + 32 * u + lane < ncand;
      gt += __popc(__ballot_sync(0xffffffffu, in && key[u] > thr));
      eq += __popc(__ballot_sync(0xffffffffu, in && key[u] == thr));
    }
  }
  if (lane == 0) { warp_gt[warp] = gt; warp_eq[warp] = eq; }
  __syncthreads();
  uint32_t run_gt = 0, run_eq = 0;
  for (int ww = 0; ww < warp; ++ww) { run_gt += warp_gt[ww]; run_eq += warp_eq[ww]; }
  const uint32_t below = (1u << lane) - 1u;
  for (int i0 = 0; i0 < per_warp; i0 += kStep) {
    uint32_t key[kSelBlockUnroll];
#pragma unroll
    for (int u = 0; u < kSelBlockUnroll; ++u) {
      const int i = w0 + i0 + 32 * u + lane;
      key[u] = (i < ncand) ? float_to_key(__ldg(src + a.lo + i)) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kSelBlockUnroll; ++u) {
      const int i = w0 + i0 + 32 * u + lane;
      const bool is_gt = i < ncand && key[u] > thr, is_eq = i < ncand && key[u] == thr;
      const unsigned mg = __ballot_sync(0xffffffffu, is_gt), me = __ballot_sync(0xffffffffu, is_eq);
      const uint32_t gt_before = run_gt + __popc(mg & below), eq_before = run_eq + __popc(me & below);
      if (is_gt || (is_eq && eq_before < need_eq))
        out[a.lo + gt_before + (eq_before < need_eq ? eq_before : need_eq)] = a.lo + i;
      run_gt += __popc(mg);
      run_eq += __popc(me);
    }
  }
  for (int i = tid; i < a.lo; i += kSelThreads) out[i] = i;
  const int tail = a.n - a.hi;
  for (int i = tid; i < tail; i += kSelThreads) out[a.lo + a.m + i] = a.hi + i;
}

// Blocks of sel_fused_kernel that can be resident at once on this device (0 if unknown).
template <bool POOL>
inline int sel_fused_capacity(size_t smem) {
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sel_fused_kernel<POOL>, kSelThreads, smem) !=
      cudaSuccess)
    return 0;
  return sms * per_sm;
}

inline int launch_select(SelArgs a, int segs, const float* ts, float* pooled, int radius,
                         void* ws_base, const SelLayout& L, int32_t* dev_status, cudaStream_t st,
                         int pool_mode = 0) {
  if (segs == 0) return REFORM_OK;
  if (!ts && a.n <= kSelBlockMaxN && segs >= kSelBlockMinSegs) {
    g_last_path = REFORM_PATH_PER_SEGMENT;
    sel_block_kernel<<<segs, kSelThreads, 0, st>>>(a);
    count_launch();
    return check_launch();
  }
  dim3 grid(a.blocks_per_seg, segs);
  {
    const size_t smem = ts ? sizeof(float) * pool_tile_floats(kSelTile, radius) : 0;
    if (ts) cudaFuncSetAttribute(sel_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int capacity = ts ? sel_fused_capacity<true>(smem) : sel_fused_capacity<false>(smem);
    if ((long long)a.blocks_per_seg * segs <= capacity) {
      g_last_path = REFORM_PATH_COOPERATIVE;
      if (cudaMemsetAsync(ws_base, 0, L.zero_bytes, st) != cudaSuccess) return check_launch();
      SelFusedCtl* ctl = reinterpret_cast<SelFusedCtl*>(reinterpret_cast<char*>(ws_base) + L.ctl);
      void* args[] = {&a, &ctl, &ts, &pooled, &radius, &pool_mode, &dev_status};
      cudaError_t e = cudaLaunchCooperativeKernel(
          ts ? (const void*)sel_fused_kernel<true> : (const void*)sel_fused_kernel<false>, grid,
          dim3(kSelThreads), args, smem, st);
      if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return REFORM_ERR_CUDA;
      }
      count_launch();
      return check_launch();
    }
  }
  g_last_path = REFORM_PATH_PER_PASS;
  sel_init_kernel<<<segs, 256, 0, st>>>(a, segs);
  count_launch();
  if (ts) {
    size_t smem = sizeof(float) * pool_tile_floats(kSelTile, radius);
    cudaFuncSetAttribute(sel_hist_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    sel_hist_kernel<true><<<grid, kSelThreads, smem, st>>>(a, 0, ts, pooled, radius, pool_mode);
  } else {
    sel_hist_kernel<false><<<grid, kSelThreads, 0, st>>>(a, 0, nullptr, nullptr, 0, 0);
  }
  sel_hist_kernel<false><<<grid, kSelThreads, 0, st>>>(a, 1, nullptr, nullptr, 0, 0);
  sel_hist_kernel<false><<<grid, kSelThreads, 0, st>>>(a, 2, nullptr, nullptr, 0, 0);
  sel_count_kernel<<<grid, kSelThreads, 0, st>>>(a);
  sel_write_kernel<<<grid, kSelThreads, 0, st>>>(a);
  count_launch(5);
  return check_launch();
}

}  // namespace reform
