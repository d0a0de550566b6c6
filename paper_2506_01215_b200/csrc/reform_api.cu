// C ABI of the REFORM compress-and-gather core: argument validation, workspace
// carving and kernel dispatch.  Every entry point either returns an error
// before launching anything or enqueues its kernels on the caller's stream.
#include <atomic>
#include <chrono>
#include <random>

#include "common.cuh"
#include "rows.cuh"
#include "embed.cuh"
#include "rope.cuh"
#include "select.cuh"
#include "evict_fused.cuh"
#include "select_cluster.cuh"
#include "retrieve.cuh"
#include "chunk_simt.cuh"
#if !defined(REFORM_NO_SM100) && !__has_include("chunk_sm100.cuh")
#define REFORM_NO_SM100
#endif
#ifndef REFORM_NO_SM100
#include "chunk_sm100.cuh"
#include "decode.cuh"
#include "retrieve_sm100.cuh"
#endif

namespace reform {
thread_local int g_last_cuda_error = 0;
thread_local int g_last_path = REFORM_PATH_NONE;   // launch form of this thread's last selection (diagnostic)
static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

unsigned long long next_epoch() {
  static const unsigned long long salt = [] {
    unsigned long long x = (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count();
    try {
      std::random_device rd;
      x ^= ((unsigned long long)rd() << 32) ^ rd();
    } catch (...) {
    }
    return x;
  }();
  static std::atomic<unsigned long long> counter{1};
  unsigned long long e;
  do {
    e = (salt + counter.fetch_add(1, std::memory_order_relaxed)) << 3;
  } while (e == 0);
  return e;
}

static size_t elem_size(int dtype) { return dtype == REFORM_F32 ? 4 : 2; }
static bool dtype_ok(int dtype) { return dtype == REFORM_F32 || dtype == REFORM_BF16; }

static size_t chunk_lse_bytes(const reform_chunk_params* p) {
  return align_up(sizeof(float) * (size_t)p->B * p->Hq * p->Lc, 256);
}

// Decode-shaped steps (a few query rows per KV head) take the split-KV kernel.
static bool chunk_uses_decode(const reform_chunk_params* p) {
#ifndef REFORM_NO_SM100
  return p->Lc > 0 && decode_shape(p) && !(p->flags & REFORM_FORCE_SIMT);
#else
  (void)p;
  return false;
#endif
}

static size_t chunk_workspace_bytes(const reform_chunk_params* p);

static bool chunk_uses_sm100(const reform_chunk_params* p) {
#ifndef REFORM_NO_SM100
  return p->dtype == REFORM_BF16 && p->d == 128 && !(p->flags & REFORM_FORCE_SIMT);
#else
  (void)p;
  return false;
#endif
}

// (batch, head) pairs index gridDim.y of the chunk-step kernels
constexpr long long kMaxGridY = 65535;

// Shape checks shared by the workspace-size query and the launch.
static int validate_chunk_shape(const reform_chunk_params* p) {
  if (!p || p->struct_size != sizeof(reform_chunk_params)) return REFORM_ERR_INVALID_ARG;
  if (!dtype_ok(p->dtype)) return REFORM_ERR_UNSUPPORTED;
  if (p->B < 0 || p->Hq <= 0 || p->Hkv <= 0 || p->Hq % p->Hkv != 0) return REFORM_ERR_INVALID_ARG;
  if ((long long)p->B * p->Hq > kMaxGridY) return REFORM_ERR_INVALID_ARG;
  if (p->Lc < 0 || p->n_cache < 0 || (long long)p->n_cache + p->Lc > p->cap) return REFORM_ERR_INVALID_ARG;
  if (p->d != 64 && p->d != 128) return REFORM_ERR_UNSUPPORTED;
  return REFORM_OK;
}

static int validate_chunk(const reform_chunk_params* p) {
  int rc = validate_chunk_shape(p);
  if (rc != REFORM_OK) return rc;
  if (!(p->flags & REFORM_NO_SCORE)) {
    if (p->Lc > 0 && (p->score_window < 1 || p->score_window > p->Lc)) return REFORM_ERR_INVALID_ARG;
    if (!p->score) return REFORM_ERR_INVALID_ARG;
  }
  if (!(p->softmax_scale >= 0.f)) return REFORM_ERR_INVALID_ARG;
  if ((p->flags & REFORM_ROPE_INTERLEAVED) && !(p->flags & REFORM_ROPE)) return REFORM_ERR_INVALID_ARG;
  if ((p->flags & REFORM_ROPE) && !(p->rope_theta >= 0.f)) return REFORM_ERR_INVALID_ARG;
  if (!p->q || !p->k || !p->v || !p->out) return REFORM_ERR_INVALID_ARG;
  if (!aligned16(p->q) || !aligned16(p->k) || !aligned16(p->v) || !aligned16(p->out) ||
      !aligned16(p->score) || !aligned16(p->lse))
    return REFORM_ERR_INVALID_ARG;
  return REFORM_OK;
}
}  // namespace reform

namespace reform {
// Scratch of a REFORM_ROPE step: rotated keys [B*Hkv, cap, d] (the layout of k); rotated queries -- all rows, or on the
// tensor-core attention path (which rotates its query tiles at load) only the score window's rows;
// and on that path the (cos, sin) table [Lc][d/2].
struct RopeScratch {
  size_t k_bytes, q_bytes, table_bytes;
  int q_rows, q_first;   // rotated query rows kept, and the chunk row of the first
  bool at_load;          // the attention kernel rotates its query tiles itself
  size_t total() const { return k_bytes + q_bytes + table_bytes; }
};

static RopeScratch rope_scratch(const reform_chunk_params* p) {
  RopeScratch r{};
  if (!(p->flags & REFORM_ROPE)) return r;
  const size_t esz = elem_size(p->dtype);
  r.at_load = chunk_uses_sm100(p) && !chunk_uses_decode(p);
  if (r.at_load) {
    r.q_rows = (p->flags & REFORM_NO_SCORE) ? 0 : p->score_window;
    r.q_first = p->Lc - r.q_rows;
    r.table_bytes = align_up(sizeof(float2) * (size_t)p->Lc * (p->d / 2), 256);
  } else {
    r.q_rows = p->Lc;
    r.q_first = 0;
  }
  r.k_bytes = align_up((size_t)p->B * p->Hkv * p->cap * p->d * esz, 256);
  r.q_bytes = align_up((size_t)p->B * p->Hq * r.q_rows * p->d * esz, 256);
  return r;
}

static size_t chunk_workspace_bytes(const reform_chunk_params* p) {
  size_t bytes = p->lse ? 0 : chunk_lse_bytes(p);
#ifndef REFORM_NO_SM100
  if (chunk_uses_decode(p)) bytes += decode_workspace_bytes(p);
#endif
  bytes += rope_scratch(p).total();
  return bytes;
}
}  // namespace reform

using namespace reform;

extern "C" {

size_t reform_chunk_step_workspace_size(const reform_chunk_params* p) {
  if (validate_chunk_shape(p) != REFORM_OK) return 0;
  if (p->B == 0 || p->Lc == 0) return 0;
  return chunk_workspace_bytes(p);
}

int reform_chunk_step(const reform_chunk_params* p, reform_stream_t stream) {
  int rc = validate_chunk(p);
  if (rc != REFORM_OK) return rc;
  if (p->B == 0 || p->Lc == 0) return REFORM_OK;
  float* lse = p->lse;
  char* ws = reinterpret_cast<char*>(p->workspace);
  const size_t need = chunk_workspace_bytes(p);
  if (need && (!ws || p->workspace_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)))
    return REFORM_ERR_WORKSPACE;
  if (!lse) {
    lse = reinterpret_cast<float*>(ws);
    ws += chunk_lse_bytes(p);
  }
  float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->d);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
#ifndef REFORM_NO_SM100
  char* ws_decode = ws;
  if (chunk_uses_decode(p)) ws += decode_workspace_bytes(p);
#endif
  if (!(p->flags & REFORM_ROPE)) {
#ifndef REFORM_NO_SM100
    if (chunk_uses_decode(p)) {
      rc = launch_decode(p, lse, scale, ws_decode, st);
      if (rc != REFORM_OK || (p->flags & REFORM_NO_SCORE)) return rc;
      return launch_chunk_sm100(p, lse, scale, st, /*run_attention=*/false);
    }
    if (chunk_uses_sm100(p)) return launch_chunk_sm100(p, lse, scale, st);
#endif
    return launch_chunk_simt(p, lse, scale, st);
  }

  // REFORM_ROPE: rotate the keys (positions 0 .. n-1) and the queries that are not rotated at load
  // (positions n_cache + i) into the workspace, then run the same kernels on the rotated operands.
  const RopeScratch rs = rope_scratch(p);
  const int n = p->n_cache + p->Lc;
  const double base = p->rope_theta > 0.f ? (double)p->rope_theta : 10000.0;
  const bool inter = (p->flags & REFORM_ROPE_INTERLEAVED) != 0;
  if ((p->d * elem_size(p->dtype)) % 32 != 0) return REFORM_ERR_UNSUPPORTED;
  void* k_rot = ws;
  void* q_rot = ws + rs.k_bytes;
  float2* table = reinterpret_cast<float2*>(ws + rs.k_bytes + rs.q_bytes);
  if (p->dtype == REFORM_F32) {
    rc = launch_rope<float>(p->k, k_rot, p->B * p->Hkv, p->d, p->cap, 0, n, 0, base, inter, st);
    if (rc == REFORM_OK && rs.q_rows)
      rc = launch_rope<float>(p->q, q_rot, p->B * p->Hq, p->d, p->Lc, rs.q_first, rs.q_rows,
                              (long long)p->n_cache + rs.q_first, base, inter, st, rs.q_rows, 0);
  } else {
    rc = launch_rope<__nv_bfloat16>(p->k, k_rot, p->B * p->Hkv, p->d, p->cap, 0, n, 0, base, inter, st);
    if (rc == REFORM_OK && rs.q_rows)
      rc = launch_rope<__nv_bfloat16>(p->q, q_rot, p->B * p->Hq, p->d, p->Lc, rs.q_first, rs.q_rows,
                                      (long long)p->n_cache + rs.q_first, base, inter, st, rs.q_rows, 0);
  }
  if (rc != REFORM_OK) return rc;
#ifndef REFORM_NO_SM100
  if (rs.at_load) {
    rc = launch_rope_table(table, p->Lc, p->d, p->n_cache, base, st);
    if (rc != REFORM_OK) return rc;
    RopeOperands ro;
    ro.k_rot = k_rot;
    ro.q_score = q_rot;
    ro.q_score_rows = rs.q_rows;
    ro.q_score_first = rs.q_first;
    ro.table = table;
    ro.interleaved = inter ? 1 : 0;
    return launch_chunk_sm100(p, lse, scale, st, /*run_attention=*/true, &ro);
  }
#endif
  // every other path reads fully rotated copies: the same kernels on the rotated operands
  reform_chunk_params r = *p;
  r.flags &= ~(uint32_t)(REFORM_ROPE | REFORM_ROPE_INTERLEAVED);
  r.q = q_rot;
  r.k = k_rot;
#ifndef REFORM_NO_SM100
  if (chunk_uses_decode(p)) {
    rc = launch_decode(&r, lse, scale, ws_decode, st);
    if (rc != REFORM_OK || (p->flags & REFORM_NO_SCORE)) return rc;
    RopeOperands ro;
    ro.k_rot = k_rot;
    ro.q_score = q_rot;
    ro.q_score_rows = p->Lc;
    ro.q_score_first = 0;
    ro.q_attn = q_rot;
    return launch_chunk_sm100(p, lse, scale, st, /*run_attention=*/false, &ro);
  }
#endif
  return launch_chunk_simt(&r, lse, scale, st);
}

/* ---------------------------------------------------------------- evict */

static bool evict_in_place(const reform_evict_params* p) {
  return p->k_src == p->k_dst && p->v_src == p->v_dst && p->score_src == p->score_dst &&
         p->pos_src == p->pos_dst && p->cap_src == p->cap_dst;
}

static int validate_evict(const reform_evict_params* p) {
  if (!p || p->struct_size != sizeof(reform_evict_params)) return REFORM_ERR_INVALID_ARG;
  if (!dtype_ok(p->dtype)) return REFORM_ERR_UNSUPPORTED;
  if (p->B < 0 || p->Hkv <= 0 || p->d <= 0) return REFORM_ERR_INVALID_ARG;
  if ((long long)p->B * p->Hkv > kMaxGridY) return REFORM_ERR_INVALID_ARG;
  if (((size_t)p->d * elem_size(p->dtype)) % 16 != 0) return REFORM_ERR_UNSUPPORTED;
  if (p->n_keys < 0 || p->n_keys > p->cap_src || p->budget < 0) return REFORM_ERR_INVALID_ARG;
  if (p->n_sink < 0 || p->n_recent < 0 || (long long)p->n_sink + p->n_recent > p->budget)
    return REFORM_ERR_INVALID_ARG;
  int n_kept = p->n_keys < p->budget ? p->n_keys : p->budget;
  if (n_kept > p->cap_dst) return REFORM_ERR_INVALID_ARG;
  if (!p->k_src || !p->v_src || !p->score_src || !p->k_dst || !p->v_dst || !p->score_dst)
    return REFORM_ERR_INVALID_ARG;
  if ((p->pos_src == nullptr) != (p->pos_dst == nullptr)) return REFORM_ERR_INVALID_ARG;
  if (!aligned16(p->k_src) || !aligned16(p->v_src) || !aligned16(p->k_dst) || !aligned16(p->v_dst) ||
      !aligned16(p->score_src) || !aligned16(p->score_dst) || !aligned16(p->kept_idx))
    return REFORM_ERR_INVALID_ARG;
  // in place means all of K, V, score (and position) in place, with one capacity; otherwise none
  const bool any_same = p->k_src == p->k_dst || p->v_src == p->v_dst || p->score_src == p->score_dst ||
                        (p->pos_src && p->pos_src == p->pos_dst);
  if (any_same && !evict_in_place(p)) return REFORM_ERR_INVALID_ARG;
  return REFORM_OK;
}

static size_t evict_kept_bytes(const reform_evict_params* p) {
  return align_up(sizeof(int32_t) * (size_t)p->B * p->Hkv * (p->budget > 0 ? p->budget : 1), 256);
}

// Smallest workspace with which the call can run at all (the per-pass selection path).
static size_t evict_workspace_min(const reform_evict_params* p) {
  return sel_layout(p->B * p->Hkv, p->n_keys).total + (p->kept_idx ? 0 : evict_kept_bytes(p));
}

size_t reform_evict_topk_workspace_size(const reform_evict_params* p) {
  if (!p || p->struct_size != sizeof(reform_evict_params)) return 0;
  if (p->B <= 0 || p->Hkv <= 0 || p->n_keys < 0) return 0;
  const size_t fused = evict_fused_layout(p->B * p->Hkv, p->n_keys).total + (p->kept_idx ? 0 : evict_kept_bytes(p));
  const size_t basic = evict_workspace_min(p);
  return fused > basic ? fused : basic;
}

// need: the workspace size the entry point insists on.  wait_cycles / expect_extra: limits of the
// hand-off waits of the cooperative one-launch form (diagnostic entry point, which also rules out the
// cluster form, whose barriers are the hardware's; kEvWaitCycles and 0 otherwise).
static int evict_run(const reform_evict_params* p, cudaStream_t st, size_t need, long long wait_cycles,
                     int expect_extra) {
  const int n_kept = p->n_keys < p->budget ? p->n_keys : p->budget;
  if (p->n_kept_host) *p->n_kept_host = n_kept;
  const int segs = p->B * p->Hkv;
  g_last_path = REFORM_PATH_NONE;
  if (segs == 0 || n_kept == 0) return REFORM_OK;
  if (!p->workspace || p->workspace_bytes < need || (reinterpret_cast<uintptr_t>(p->workspace) & 255u))
    return REFORM_ERR_WORKSPACE;
  char* ws = reinterpret_cast<char*>(p->workspace);
  int lo, hi, m;
  if (p->n_keys <= p->budget) {  // keep everything: all rows are "forced"
    lo = hi = p->n_keys;
    m = 0;
  } else {
    lo = p->n_sink;
    hi = p->n_keys - p->n_recent;
    m = p->budget - p->n_sink - p->n_recent;
  }
  const int row_bytes = (int)(p->d * elem_size(p->dtype));
  const size_t kept_bytes = p->kept_idx ? 0 : evict_kept_bytes(p);
  const bool in_place = evict_in_place(p);
  const bool many_short = p->n_keys <= kSelBlockMaxN && segs >= kSelBlockMinSegs;  // one block per segment wins
  if (expect_extra == 0 && (in_place ? row_bytes <= 256 : !many_short)) {
    // one cluster per segment: selection and compaction in one launch, no workspace but the kept list.
    // Taken in place always, and otherwise when the clusters run in one wave on enough blocks to
    // stream the kept rows at the device's rate (the cooperative form below spreads the copy over
    // the whole device whatever the number of segments).
    const ClusterCapacity cap = cluster_select_capacity<1>(cluster_sel_smem_bytes(false, 0, 0));
    const int c = cluster_select_size(segs, p->n_keys, cap);
    if (c && (in_place || (cluster_select_one_wave(segs, c, cap) && segs * c >= kClMinBlocksForCopy))) {
      ClusterSelArgs a = {};
      a.vals = p->score_src;
      a.stride = p->cap_src;
      a.n = p->n_keys;
      a.lo = lo;
      a.hi = hi;
      a.m = m;
      a.out = p->kept_idx ? p->kept_idx : reinterpret_cast<int32_t*>(ws);
      a.out_stride = p->budget;
      a.k_src = (const uint4*)p->k_src;
      a.v_src = (const uint4*)p->v_src;
      a.k_dst = (uint4*)p->k_dst;
      a.v_dst = (uint4*)p->v_dst;
      a.score_src = p->score_src;
      a.score_dst = p->score_dst;
      a.pos_src = p->pos_src;
      a.pos_dst = p->pos_dst;
      a.n_kept = n_kept;
      a.cap_src = p->cap_src;
      a.cap_dst = p->cap_dst;
      a.vec = row_bytes / 16;
      a.in_place = in_place ? 1 : 0;
      g_last_path = REFORM_PATH_CLUSTER;
      return launch_cluster_select<1>(a, segs, c, st);
    }
  }
  if (in_place && !evict_fused_applies(segs, p->n_keys, p->workspace_bytes, kept_bytes))
    return REFORM_ERR_UNSUPPORTED;   // only the one-launch forms can move rows inside their own buffers
  if ((in_place || !many_short) && evict_fused_applies(segs, p->n_keys, p->workspace_bytes, kept_bytes)) {
    // one cooperative launch: selection with two hand-offs, then the compaction
    const EvictFusedLayout F = evict_fused_layout(segs, p->n_keys);
    EvictFusedArgs a;
    a.vals = p->score_src;
    a.stride = p->cap_src;
    a.n = p->n_keys;
    a.lo = lo;
    a.hi = hi;
    a.m = m;
    a.out = p->kept_idx ? p->kept_idx : reinterpret_cast<int32_t*>(ws + F.total);
    a.out_stride = p->budget;
    a.segs = segs;
    a.nb = F.nb;
    a.slices = reinterpret_cast<uint32_t*>(ws + F.slices);
    a.cand = reinterpret_cast<uint32_t*>(ws + F.cand);
    a.flags = reinterpret_cast<unsigned long long*>(ws + F.flags);
    a.expect_extra = expect_extra;
    a.epoch = next_epoch() << 5;
    a.in_place = in_place ? 1 : 0;
    a.wait_cycles = wait_cycles;
    a.k_src = (const uint4*)p->k_src;
    a.v_src = (const uint4*)p->v_src;
    a.k_dst = (uint4*)p->k_dst;
    a.v_dst = (uint4*)p->v_dst;
    a.score_src = p->score_src;
    a.score_dst = p->score_dst;
    a.pos_src = p->pos_src;
    a.pos_dst = p->pos_dst;
    a.n_kept = n_kept;
    a.cap_src = p->cap_src;
    a.cap_dst = p->cap_dst;
    a.vec = row_bytes / 16;
    a.dev_status = p->dev_status;
    g_last_path = REFORM_PATH_COOPERATIVE;
    return launch_evict_fused(a, st);
  }
  SelLayout L = sel_layout(segs, p->n_keys);
  int32_t* kept = p->kept_idx ? p->kept_idx : reinterpret_cast<int32_t*>(ws + L.total);
  SelArgs a;
  a.vals = p->score_src;
  a.stride = p->cap_src;
  a.n = p->n_keys;
  a.lo = lo;
  a.hi = hi;
  a.m = m;
  a.out = kept;
  a.out_stride = p->budget;
  a.state = reinterpret_cast<SelState*>(ws + L.state);
  a.hist = reinterpret_cast<uint32_t*>(ws + L.hist);
  a.blockcnt = reinterpret_cast<uint2*>(ws + L.blockcnt);
  a.blocks_per_seg = L.blocks_per_seg;
  int rc = launch_select(a, segs, nullptr, nullptr, 0, ws, L, p->dev_status, st);
  if (rc != REFORM_OK) return rc;
  return launch_evict_compact(p->k_src, p->v_src, p->k_dst, p->v_dst, p->score_src, p->score_dst,
                              p->pos_src, p->pos_dst, kept, p->budget, segs, n_kept, p->cap_src,
                              p->cap_dst, row_bytes, st);
}

int reform_evict_topk(const reform_evict_params* p, reform_stream_t stream) {
  int rc = validate_evict(p);
  if (rc != REFORM_OK) return rc;
  return evict_run(p, reinterpret_cast<cudaStream_t>(stream), reform_evict_topk_workspace_size(p), kEvWaitCycles, 0);
}

int reform_debug_evict_wait_expiry(const reform_evict_params* p, long long wait_cycles, reform_stream_t stream) {
  int rc = validate_evict(p);
  if (rc != REFORM_OK) return rc;
  if (wait_cycles <= 0 || wait_cycles > kEvWaitCycles) return REFORM_ERR_INVALID_ARG;
  const int segs = p->B * p->Hkv;
  const size_t kept_bytes = p->kept_idx ? 0 : evict_kept_bytes(p);
  const bool many_short = p->n_keys <= kSelBlockMaxN && segs >= kSelBlockMinSegs;
  if (segs == 0 || p->n_keys <= p->budget || p->budget == p->n_sink + p->n_recent || many_short ||
      !evict_fused_applies(segs, p->n_keys, p->workspace_bytes, kept_bytes))
    return REFORM_ERR_UNSUPPORTED;   // only the one-launch form has hand-off waits to run out
  return evict_run(p, reinterpret_cast<cudaStream_t>(stream), reform_evict_topk_workspace_size(p), wait_cycles, 1);
}

/* ------------------------------------------ evict without a workspace */

// Scratch of reform_evict_topk_static.  In host code this name is only a
// handle for cudaGetSymbolAddress; the kernels get the device address.
static __device__ __align__(256) unsigned char g_evict_static_scratch[REFORM_EVICT_STATIC_BYTES];

// Device address of the scratch array on the current device, looked up once per device.
static int evict_static_scratch(void** out) {
  constexpr int kMaxDevices = 64;
  static std::atomic<void*> cache[kMaxDevices];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    g_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidDevice);
    return REFORM_ERR_CUDA;
  }
  void* ptr = cache[dev].load(std::memory_order_acquire);
  if (!ptr) {
    e = cudaGetSymbolAddress(&ptr, g_evict_static_scratch);
    if (e != cudaSuccess || !ptr) {
      g_last_cuda_error = (int)e;
      return REFORM_ERR_CUDA;
    }
    cache[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return REFORM_OK;
}

int reform_evict_topk_static(const reform_evict_params* p, reform_stream_t stream) {
  int rc = validate_evict(p);
  if (rc != REFORM_OK) return rc;
  if ((long long)p->B * p->Hkv > REFORM_EVICT_STATIC_MAX_SEGS || p->n_keys > REFORM_EVICT_STATIC_MAX_KEYS ||
      p->budget > REFORM_EVICT_STATIC_MAX_BUDGET)
    return REFORM_ERR_TOO_LARGE;
  reform_evict_params q = *p;
  q.workspace = nullptr;
  q.workspace_bytes = 0;
  const size_t need = evict_workspace_min(&q);
  if (need > REFORM_EVICT_STATIC_BYTES) return REFORM_ERR_TOO_LARGE;
  void* scratch = nullptr;
  rc = evict_static_scratch(&scratch);
  if (rc != REFORM_OK) return rc;
  q.workspace = scratch;
  q.workspace_bytes = REFORM_EVICT_STATIC_BYTES;
  // the one-launch form is taken when its (larger) layout fits the array too
  return evict_run(&q, reinterpret_cast<cudaStream_t>(stream), need, kEvWaitCycles, 0);
}

/* ---------------------------------------------------------------- embed */

int reform_embed_append(const reform_embed_params* p, reform_stream_t stream) {
  if (!p || p->struct_size != sizeof(reform_embed_params)) return REFORM_ERR_INVALID_ARG;
  if (!dtype_ok(p->dtype)) return REFORM_ERR_UNSUPPORTED;
  if (p->B < 0 || p->Lc < 0 || p->d <= 0 || p->n_sel < 0 || p->n_sel > REFORM_MAX_SEL)
    return REFORM_ERR_INVALID_ARG;
  if (p->d % 4 != 0 || p->d > 4 * 32 * kEmbedMaxVec) return REFORM_ERR_UNSUPPORTED;
  if (p->E <= 0 || (p->E * elem_size(p->dtype)) % 16 != 0) return REFORM_ERR_UNSUPPORTED;
  if (p->token_offset < 0 || p->token_offset + p->Lc > p->N_cap) return REFORM_ERR_INVALID_ARG;
  if (!p->bank || !aligned16(p->bank) || (p->n_sel > 0 && !p->sel)) return REFORM_ERR_INVALID_ARG;
  if (!(p->eps >= 0.f)) return REFORM_ERR_INVALID_ARG;
  EmbedSel sel;
  sel.n_sel = p->n_sel;
  for (int s = 0; s < p->n_sel; ++s) {
    const reform_head_sel& e = p->sel[s];
    const void* src = nullptr;
    int H = 0;
    if (e.kind == REFORM_STATE_Q) { src = p->q_state; H = p->Hq; }
    else if (e.kind == REFORM_STATE_K) { src = p->k_state; H = p->Hkv; }
    else if (e.kind == REFORM_STATE_V) { src = p->v_state; H = p->Hkv; }
    else return REFORM_ERR_INVALID_ARG;
    if (!src || !aligned16(src) || e.head < 0 || e.head >= H || e.slot < 0 ||
        (long long)(e.slot + 1) * p->d > p->E)
      return REFORM_ERR_INVALID_ARG;
    sel.src[s] = src;
    sel.H[s] = H;
    sel.head[s] = e.head;
    sel.slot[s] = e.slot;
  }
  if (p->B == 0 || p->Lc == 0 || p->n_sel == 0) return REFORM_OK;
  float eps = p->eps > 0.f ? p->eps : 1e-12f;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (p->dtype == REFORM_F32)
    return launch_embed<float>(sel, p->bank, p->B, p->Lc, p->d, p->E, p->N_cap, p->token_offset, eps, st);
  return launch_embed<__nv_bfloat16>(sel, p->bank, p->B, p->Lc, p->d, p->E, p->N_cap, p->token_offset,
                                     eps, st);
}

/* ------------------------------------------------------------- retrieve */

static int validate_retrieve(const reform_retrieve_params* p) {
  if (!p || p->struct_size != sizeof(reform_retrieve_params)) return REFORM_ERR_INVALID_ARG;
  if (!dtype_ok(p->dtype)) return REFORM_ERR_UNSUPPORTED;
  if (p->B < 0 || p->B > kMaxGridY || p->N < 0 || p->N > p->N_cap || p->N > 0x7fffffffLL || p->E <= 0 ||
      p->nq < 1)
    return REFORM_ERR_INVALID_ARG;
  if ((p->E * elem_size(p->dtype)) % 16 != 0) return REFORM_ERR_UNSUPPORTED;
  if (p->pool_window < 1 || p->pool_window % 2 == 0) return REFORM_ERR_INVALID_ARG;
  if (p->pool_mode != REFORM_POOL_MAX && p->pool_mode != REFORM_POOL_MEAN) return REFORM_ERR_INVALID_ARG;
  if ((p->pool_window - 1) / 2 > kSelMaxRadius) return REFORM_ERR_UNSUPPORTED;
  if (p->k < 0 || p->n_keep_head < 0 || p->n_keep_tail < 0 ||
      (long long)p->n_keep_head + p->n_keep_tail > p->k)
    return REFORM_ERR_INVALID_ARG;
  if (!p->bank || !p->queries || !p->idx_out) return REFORM_ERR_INVALID_ARG;
  if (!aligned16(p->bank) || !aligned16(p->queries) || !aligned16(p->idx_out) ||
      !aligned16(p->token_score_out) || !aligned16(p->pooled_score_out))
    return REFORM_ERR_INVALID_ARG;
  return REFORM_OK;
}

static size_t retrieve_score_bytes(const reform_retrieve_params* p) {
  return align_up(sizeof(float) * (size_t)p->B * (size_t)p->N, 256);
}

size_t reform_retrieve_topk_workspace_size(const reform_retrieve_params* p) {
  if (!p || p->struct_size != sizeof(reform_retrieve_params)) return 0;
  if (p->B <= 0 || p->N <= 0) return 0;
  size_t total = sel_layout(p->B, p->N).total;
  if (!p->token_score_out) total += retrieve_score_bytes(p);
  if (!p->pooled_score_out) total += retrieve_score_bytes(p);
  return total;
}

int reform_retrieve_topk(const reform_retrieve_params* p, reform_stream_t stream) {
  int rc = validate_retrieve(p);
  if (rc != REFORM_OK) return rc;
  g_last_path = REFORM_PATH_NONE;
  if (p->B == 0 || p->N == 0 || p->k == 0) return REFORM_OK;
  size_t need = reform_retrieve_topk_workspace_size(p);
  if (!p->workspace || p->workspace_bytes < need || (reinterpret_cast<uintptr_t>(p->workspace) & 255u))
    return REFORM_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* ws = reinterpret_cast<char*>(p->workspace);
  SelLayout L = sel_layout(p->B, p->N);
  size_t off = L.total;
  float* ts = p->token_score_out;
  if (!ts) { ts = reinterpret_cast<float*>(ws + off); off += retrieve_score_bytes(p); }
  float* pooled = p->pooled_score_out;
  if (!pooled) { pooled = reinterpret_cast<float*>(ws + off); off += retrieve_score_bytes(p); }
  rc = REFORM_ERR_UNSUPPORTED;
#ifndef REFORM_NO_SM100
  if (p->dtype == REFORM_BF16)
    rc = launch_scan_sm100(p->bank, p->queries, ts, p->B, p->N, p->N_cap, p->E, p->nq, p->scale,
                           p->dev_status, st);
#endif
  if (rc == REFORM_ERR_UNSUPPORTED)
    rc = launch_scan(p->dtype, p->bank, p->queries, ts, p->B, p->N, p->N_cap, p->E, p->nq, p->scale, st);
  if (rc != REFORM_OK) return rc;
  SelArgs a;
  a.vals = pooled;
  a.stride = p->N;
  a.n = (int)p->N;
  if (p->N <= p->k) {
    a.lo = a.hi = (int)p->N;
    a.m = 0;
  } else {
    a.lo = p->n_keep_head;
    a.hi = (int)p->N - p->n_keep_tail;
    a.m = p->k - p->n_keep_head - p->n_keep_tail;
  }
  {
    // banks of up to 16 x 8192 tokens: pooling and selection by one cluster per sequence
    const int radius = (p->pool_window - 1) / 2;
    const ClusterCapacity cap = cluster_select_capacity<0>(cluster_sel_smem_bytes(true, kClTile, radius));
    const int c = cluster_select_size(p->B, p->N, cap);
    if (c && cluster_select_one_wave(p->B, c, cap)) {
      ClusterSelArgs ca = {};
      ca.vals = ts;
      ca.stride = p->N;
      ca.n = a.n;
      ca.lo = a.lo;
      ca.hi = a.hi;
      ca.m = a.m;
      ca.out = p->idx_out;
      ca.out_stride = p->k;
      ca.pooled_out = p->pooled_score_out;
      ca.radius = radius;
      ca.pool_mode = p->pool_mode;
      g_last_path = REFORM_PATH_CLUSTER;
      return launch_cluster_select<0>(ca, p->B, c, st);
    }
  }
  a.out = p->idx_out;
  a.out_stride = p->k;
  a.state = reinterpret_cast<SelState*>(ws + L.state);
  a.hist = reinterpret_cast<uint32_t*>(ws + L.hist);
  a.blockcnt = reinterpret_cast<uint2*>(ws + L.blockcnt);
  a.blocks_per_seg = L.blocks_per_seg;
  return launch_select(a, p->B, ts, pooled, (p->pool_window - 1) / 2, ws, L, p->dev_status, st, p->pool_mode);
}

/* --------------------------------------------------------------- gather */

int reform_gather(const reform_gather_params* p, reform_stream_t stream) {
  if (!p || p->struct_size != sizeof(reform_gather_params)) return REFORM_ERR_INVALID_ARG;
  if (p->B < 0 || p->k < 0 || p->n_rows < 0 || p->row_bytes <= 0) return REFORM_ERR_INVALID_ARG;
  if (p->row_bytes % 16 != 0) return REFORM_ERR_UNSUPPORTED;
  if (!p->src || !p->idx || !p->dst) return REFORM_ERR_INVALID_ARG;
  if (!aligned16(p->src) || !aligned16(p->dst) || (reinterpret_cast<uintptr_t>(p->idx) & 3u))
    return REFORM_ERR_INVALID_ARG;
  return launch_gather((const uint4*)p->src, p->idx, (uint4*)p->dst, p->B, p->k, p->n_rows,
                       p->row_bytes, p->dev_status, reinterpret_cast<cudaStream_t>(stream));
}

/* ----------------------------------------------------------------- rope */

int reform_rope(const reform_rope_params* p, reform_stream_t stream) {
  if (!p || p->struct_size != sizeof(reform_rope_params)) return REFORM_ERR_INVALID_ARG;
  if (!dtype_ok(p->dtype)) return REFORM_ERR_UNSUPPORTED;
  if (p->B < 0 || p->H < 0 || p->d <= 0 || p->cap < 0 || p->row_begin < 0 || p->rows < 0 ||
      p->row_begin + p->rows > p->cap || p->pos_begin < 0 || !(p->theta_base >= 0.f))
    return REFORM_ERR_INVALID_ARG;
  if ((p->d * elem_size(p->dtype)) % 32 != 0 || p->d / 2 > kRopeMaxPairs) return REFORM_ERR_UNSUPPORTED;
  if (!p->src || !p->dst || !aligned16(p->src) || !aligned16(p->dst)) return REFORM_ERR_INVALID_ARG;
  const double base = p->theta_base > 0.f ? (double)p->theta_base : 10000.0;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (p->dtype == REFORM_F32)
    return launch_rope<float>(p->src, p->dst, p->B * p->H, p->d, p->cap, p->row_begin, p->rows, p->pos_begin,
                              base, p->interleaved != 0, st);
  return launch_rope<__nv_bfloat16>(p->src, p->dst, p->B * p->H, p->d, p->cap, p->row_begin, p->rows,
                                    p->pos_begin, base, p->interleaved != 0, st);
}

/* ----------------------------------------------------------------- misc */

const char* reform_status_string(int status) {
  switch (status) {
    case REFORM_OK: return "ok";
    case REFORM_ERR_INVALID_ARG: return "invalid argument";
    case REFORM_ERR_UNSUPPORTED: return "unsupported dtype, head dimension or alignment";
    case REFORM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case REFORM_ERR_CUDA: return "CUDA call failed";
    case REFORM_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

int reform_last_cuda_error(void) { return g_last_cuda_error; }

int reform_device_error(int clear) {
  int32_t word = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&word, g_device_error, sizeof(word));
  if (e == cudaSuccess && clear && word) {
    const int32_t zero = 0;
    e = cudaMemcpyToSymbol(g_device_error, &zero, sizeof(zero));
  }
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return REFORM_ERR_CUDA;
  }
  return word;
}
int reform_version(void) { return 100; }
long long reform_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
int reform_debug_last_path(void) { return g_last_path; }

}  // extern "C"
