// TEST INFRASTRUCTURE ONLY -- slow, plain, fp64 CPU statement of the REFORM
// compress-and-gather core.  Nothing in the product path may call this file:
// it exists so that tests, the smoke check and the bench's cpu_baseline leg
// have something obviously correct to compare the CUDA kernels against.
//
// It shares no code, header, table or helper with the CUDA library.  Every
// input is converted exactly to double (bf16 -> double and fp32 -> double are
// exact), every sum runs in double in the order the definition states, and
// there is no tiling, fusion or reordering beyond splitting independent
// outputs across host threads.
//
// Operations (section / algorithm of the paper each one follows):
//   oracle_attention      Sec. 3.1 + Fig. 1 step (1): a chunk's queries attend
//                         causally over [compressed cache ; chunk].
//   oracle_key_scores     Sec. 3.1 (eviction by attention mass, the H2O
//                         criterion); Sec. 4 common setup (scores from the last
//                         128 queries of a chunk): attention mass per key.
//   oracle_evict_topk     Sec. 3.1 / Fig. 1 step (3): keep heavy hitters plus
//                         the initial and recent tokens; order preserved so
//                         position ids can be re-assigned consecutively.
//   oracle_embed_append   Sec. 3.2 "Combining multiple heads": e_comb =
//                         concat(e_i / ||e_i||).
//   oracle_retrieve_topk  Sec. 3.3 "Identification of significant inputs":
//                         cosine scan, max over query tokens, max-pool over
//                         adjacent tokens, top-k with first/last tokens kept.
//   oracle_gather         Sec. 3.3 / Alg. 1 GatherRelevant: row gather.
//   oracle_rope           Sec. 3.1, position re-assignment after compression: rotary
//                         embedding at consecutive positions.
//
// Readings of the paper that it does not fix (reduction over the GQA group is
// a sum, carried scores add, ties go to the lowest index, forced tokens count
// toward the budget) are parameters or documented where they apply.
// "parity unpinned" by the paper itself: the choice of sum over the GQA group
// and of accumulation across chunks (the paper only names the H2O criterion).

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_BF16 = 1 };

int g_threads = 0;

inline double load_elem(const void* base, int dtype, size_t i) {
  if (dtype == DT_F32) {
    return (double)((const float*)base)[i];
  }
  uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16;
  float f;
  std::memcpy(&f, &bits, 4);
  return (double)f;
}

inline size_t elem_size(int dtype) { return dtype == DT_F32 ? 4 : 2; }

// Round a double to the nearest bf16 (ties to even) without passing through
// fp32, so there is no double rounding.
inline uint16_t double_to_bf16_bits(double x) {
  if (x != x) return 0x7FC0;
  if (x == 0.0) return std::signbit(x) ? 0x8000 : 0x0000;
  if (std::isinf(x)) return x > 0 ? 0x7F80 : 0xFF80;
  int e;
  double m = std::frexp(x, &e);  // x = m * 2^e, |m| in [0.5, 1)
  double y;
  if (e < -125) {                // bf16 subnormal range: fixed quantum 2^-133
    y = std::ldexp(std::nearbyint(std::ldexp(x, 133)), -133);
  } else {
    y = std::ldexp(std::nearbyint(m * 256.0), e - 8);  // 8 significant bits
  }
  float f = (float)y;            // exact unless it overflowed to inf
  uint32_t bits;
  std::memcpy(&bits, &f, 4);
  return (uint16_t)(bits >> 16);
}

inline void store_elem(void* base, int dtype, size_t i, double x) {
  if (dtype == DT_F32) {
    ((float*)base)[i] = (float)x;  // one rounding, nearest-even
  } else {
    ((uint16_t*)base)[i] = double_to_bf16_bits(x);
  }
}

int num_threads() {
  if (g_threads > 0) return g_threads;
  unsigned n = std::thread::hardware_concurrency();
  return n ? (int)n : 1;
}

// Run f(i) for i in [0, n) on the host threads; each i is an independent
// output so the split changes no arithmetic.
template <class F>
void parallel_for(size_t n, F f) {
  int nt = std::min<size_t>((size_t)num_threads(), n ? n : 1);
  if (nt <= 1) {
    for (size_t i = 0; i < n; ++i) f(i);
    return;
  }
  std::atomic<size_t> next(0);
  std::vector<std::thread> pool;
  for (int t = 0; t < nt; ++t) {
    pool.emplace_back([&]() {
      for (;;) {
        size_t i = next.fetch_add(1);
        if (i >= n) break;
        f(i);
      }
    });
  }
  for (auto& th : pool) th.join();
}

// Logits of chunk row i of q-head h against its visible keys, then the row's
// max and log-sum-exp.  Visible set: cache rows [0, n_cache) and chunk rows
// [n_cache, n_cache + i]; with causal == 0 every one of the n keys is visible.
struct RowSoftmax {
  std::vector<double> s;  // logits, length nvis
  double m;               // max logit
  double l;               // sum of exp(s - m)
  int nvis;
};

void row_logits(int dtype, int d, int Lc, int n_cache, double scale, int causal,
                const void* q, size_t q_off, const void* k, size_t k_off, int i,
                RowSoftmax& r) {
  int n = n_cache + Lc;
  r.nvis = causal ? (n_cache + i + 1) : n;
  r.s.resize(r.nvis);
  double m = -std::numeric_limits<double>::infinity();
  for (int j = 0; j < r.nvis; ++j) {
    double acc = 0.0;
    for (int e = 0; e < d; ++e) {
      acc += load_elem(q, dtype, q_off + e) * load_elem(k, dtype, k_off + (size_t)j * d + e);
    }
    acc *= scale;
    r.s[j] = acc;
    if (acc > m) m = acc;
  }
  double l = 0.0;
  for (int j = 0; j < r.nvis; ++j) l += std::exp(r.s[j] - m);
  r.m = m;
  r.l = l;
}

// Total order used by both top-k selections: larger value first, then lower
// index.  -0.0 compares equal to +0.0 under '<', which is the canonical form
// the selection wants.
struct Cand {
  double v;
  int32_t idx;
};
inline bool cand_before(const Cand& a, const Cand& b) {
  if (a.v > b.v) return true;
  if (a.v < b.v) return false;
  return a.idx < b.idx;
}

}  // namespace

extern "C" {

int oracle_set_threads(int n) {
  g_threads = n;
  return num_threads();
}

int oracle_get_threads(void) { return num_threads(); }

// Attention output and log-sum-exp for the listed chunk rows.
//   q [B,Hq,Lc,d]; k, v [B,Hkv,cap,d] with rows [0,n_cache) the compressed
//   cache and rows [n_cache, n_cache+Lc) this chunk.  q-head h reads kv-head
//   h / (Hq/Hkv).  rows: n_rows chunk-row indices, or NULL for all Lc rows.
//   out [B,Hq,n_rows,d], lse [B,Hq,n_rows] (natural log).
int oracle_attention(int dtype, int B, int Hq, int Hkv, int d, int Lc, int n_cache, int cap,
                     double scale, int causal, const void* q, const void* k, const void* v,
                     const int32_t* rows, int n_rows, double* out, double* lse) {
  if (Hkv <= 0 || Hq % Hkv != 0 || n_cache + Lc > cap) return -1;
  int G = Hq / Hkv;
  if (!rows) n_rows = Lc;
  size_t tasks = (size_t)B * Hq * n_rows;
  parallel_for(tasks, [&](size_t t) {
    int r = (int)(t % n_rows);
    int h = (int)((t / n_rows) % Hq);
    int b = (int)(t / ((size_t)n_rows * Hq));
    int i = rows ? rows[r] : r;
    int g = h / G;
    size_t q_off = (((size_t)b * Hq + h) * Lc + i) * d;
    size_t kv_off = ((size_t)b * Hkv + g) * (size_t)cap * d;
    RowSoftmax rs;
    row_logits(dtype, d, Lc, n_cache, scale, causal, q, q_off, k, kv_off, i, rs);
    double* o = out + t * d;
    for (int e = 0; e < d; ++e) o[e] = 0.0;
    for (int j = 0; j < rs.nvis; ++j) {
      double p = std::exp(rs.s[j] - rs.m) / rs.l;
      for (int e = 0; e < d; ++e) o[e] += p * load_elem(v, dtype, kv_off + (size_t)j * d + e);
    }
    if (lse) lse[t] = rs.m + std::log(rs.l);
  });
  return 0;
}

// Per-key attention mass.  score_new[b,g,j] = sum over the G q-heads of group
// g and over the last W chunk rows i of p^h_ij (0 where j is masked for i).
// score_out[b,g,j] = (accumulate && j < n_cache ? score_in[b,g,j] : 0) + score_new.
// score_in / score_out are [B,Hkv,cap]; only rows [0, n_cache+Lc) are written.
int oracle_key_scores(int dtype, int B, int Hq, int Hkv, int d, int Lc, int n_cache, int cap,
                      int W, double scale, int causal, int accumulate, const void* q,
                      const void* k, const double* score_in, double* score_out) {
  if (Hkv <= 0 || Hq % Hkv != 0 || n_cache + Lc > cap || W < 1 || W > Lc) return -1;
  int G = Hq / Hkv;
  int n = n_cache + Lc;
  int i0 = Lc - W;
  // Row normalisers first: the mass a key receives is defined with the final
  // softmax denominator of each query row.
  std::vector<double> lse((size_t)B * Hq * W);
  parallel_for(lse.size(), [&](size_t t) {
    int w = (int)(t % W);
    int h = (int)((t / W) % Hq);
    int b = (int)(t / ((size_t)W * Hq));
    int g = h / G;
    size_t q_off = (((size_t)b * Hq + h) * Lc + (i0 + w)) * d;
    size_t kv_off = ((size_t)b * Hkv + g) * (size_t)cap * d;
    RowSoftmax rs;
    row_logits(dtype, d, Lc, n_cache, scale, causal, q, q_off, k, kv_off, i0 + w, rs);
    lse[t] = rs.m + std::log(rs.l);
  });
  size_t tasks = (size_t)B * Hkv * n;
  parallel_for(tasks, [&](size_t t) {
    int j = (int)(t % n);
    int g = (int)((t / n) % Hkv);
    int b = (int)(t / ((size_t)n * Hkv));
    size_t k_off = (((size_t)b * Hkv + g) * (size_t)cap + j) * d;
    double acc = 0.0;
    for (int hh = 0; hh < G; ++hh) {
      int h = g * G + hh;
      for (int w = 0; w < W; ++w) {
        int i = i0 + w;
        if (causal && j > n_cache + i) continue;  // key not visible to this query
        size_t q_off = (((size_t)b * Hq + h) * Lc + i) * d;
        double s = 0.0;
        for (int e = 0; e < d; ++e) s += load_elem(q, dtype, q_off + e) * load_elem(k, dtype, k_off + e);
        s *= scale;
        acc += std::exp(s - lse[((size_t)b * Hq + h) * W + w]);
      }
    }
    size_t o = ((size_t)b * Hkv + g) * (size_t)cap + j;
    double carry = (accumulate && j < n_cache && score_in) ? score_in[o] : 0.0;
    score_out[o] = carry + acc;
  });
  return 0;
}

// Cache compression for every (b, kv-head): if n_keys <= budget keep all;
// otherwise keep the first n_sink and last n_recent rows and, of the rows in
// between, the (budget - n_sink - n_recent) with the largest score (full sort,
// ties to the lower index).  Kept rows are copied in ascending source order.
// Returns the number of rows kept per head, or < 0 on bad arguments.
int oracle_evict_topk(int B, int Hkv, int n_keys, int cap_src, int cap_dst, int budget, int n_sink,
                      int n_recent, long long row_bytes, const void* k_src, const void* v_src,
                      const double* score_src, const int32_t* pos_src, void* k_dst, void* v_dst,
                      double* score_dst, int32_t* pos_dst, int32_t* kept_idx) {
  if (n_keys > cap_src || n_sink < 0 || n_recent < 0 || n_sink + n_recent > budget) return -1;
  int n_kept = std::min(n_keys, budget);
  if (n_kept > cap_dst) return -1;
  size_t heads = (size_t)B * Hkv;
  parallel_for(heads, [&](size_t hh) {
    const double* sc = score_src + hh * (size_t)cap_src;
    std::vector<int32_t> kept;
    if (n_keys <= budget) {
      for (int j = 0; j < n_keys; ++j) kept.push_back(j);
    } else {
      int lo = n_sink, hi = n_keys - n_recent;  // candidates are [lo, hi)
      std::vector<Cand> c;
      for (int j = lo; j < hi; ++j) c.push_back({sc[j], j});
      std::sort(c.begin(), c.end(), cand_before);
      int m = budget - n_sink - n_recent;
      for (int j = 0; j < n_sink; ++j) kept.push_back(j);
      for (int r = 0; r < m; ++r) kept.push_back(c[r].idx);
      for (int j = hi; j < n_keys; ++j) kept.push_back(j);
      std::sort(kept.begin(), kept.end());
    }
    for (int r = 0; r < n_kept; ++r) {
      int32_t j = kept[r];
      size_t src = (hh * (size_t)cap_src + j) * (size_t)row_bytes;
      size_t dst = (hh * (size_t)cap_dst + r) * (size_t)row_bytes;
      if (k_src && k_dst) std::memcpy((char*)k_dst + dst, (const char*)k_src + src, row_bytes);
      if (v_src && v_dst) std::memcpy((char*)v_dst + dst, (const char*)v_src + src, row_bytes);
      if (score_dst) score_dst[hh * (size_t)cap_dst + r] = sc[j];
      if (pos_src && pos_dst) pos_dst[hh * (size_t)cap_dst + r] = pos_src[hh * (size_t)cap_src + j];
      if (kept_idx) kept_idx[hh * (size_t)budget + r] = j;
    }
  });
  return n_kept;
}

// Context-embedding rows.  For token t of the chunk and each selected
// (kind, head, slot): bank[b, token_offset + t, slot*d : (slot+1)*d] =
// x / max(||x||_2, eps), x that head's state for the token; the quotient is
// rounded once to the bank dtype.  sel holds n_sel triples (kind, head, slot),
// kind 0 = query state [B,Hq,Lc,d], 1 = key state, 2 = value state [B,Hkv,Lc,d].
// bank_f64 (optional, same shape) receives the unrounded values.
int oracle_embed_append(int dtype, int B, int Lc, int d, int Hq, int Hkv, const void* q_state,
                        const void* k_state, const void* v_state, int n_sel, const int32_t* sel,
                        void* bank, double* bank_f64, long long N_cap, int E,
                        long long token_offset, double eps) {
  if (token_offset < 0 || token_offset + Lc > N_cap) return -1;
  for (int s = 0; s < n_sel; ++s) {
    int kind = sel[3 * s], head = sel[3 * s + 1], slot = sel[3 * s + 2];
    const void* src = kind == 0 ? q_state : kind == 1 ? k_state : kind == 2 ? v_state : nullptr;
    int H = kind == 0 ? Hq : Hkv;
    if (!src || head < 0 || head >= H || slot < 0 || (slot + 1) * d > E) return -1;
  }
  if (eps <= 0.0) eps = 1e-12;
  size_t tasks = (size_t)B * Lc;
  parallel_for(tasks, [&](size_t t) {
    int tok = (int)(t % Lc);
    int b = (int)(t / Lc);
    for (int s = 0; s < n_sel; ++s) {
      int kind = sel[3 * s], head = sel[3 * s + 1], slot = sel[3 * s + 2];
      const void* src = kind == 0 ? q_state : kind == 1 ? k_state : v_state;
      int H = kind == 0 ? Hq : Hkv;
      size_t off = (((size_t)b * H + head) * Lc + tok) * d;
      double ss = 0.0;
      for (int e = 0; e < d; ++e) {
        double x = load_elem(src, dtype, off + e);
        ss += x * x;
      }
      double nrm = std::max(std::sqrt(ss), eps);
      size_t o = ((size_t)b * N_cap + token_offset + tok) * (size_t)E + (size_t)slot * d;
      for (int e = 0; e < d; ++e) {
        double y = load_elem(src, dtype, off + e) / nrm;
        if (bank) store_elem(bank, dtype, o + e, y);
        if (bank_f64) bank_f64[o + e] = y;
      }
    }
  });
  return 0;
}

// Token selection.  sim[q][t] = scale * <queries[q], bank[t]>; ts[t] = max_q
// sim; pooled[t] = max of ts over [t-r, t+r] clipped to [0, N), r =
// (pool_window-1)/2 (Sec. 3.3), or with pool_mode == 1 the mean of ts over that
// clipped window (the smoothing used when heads are ranked, Appendix "Detailed
// head selection process", Step 3: the window is the token and its neighbours,
// and at the ends the mean runs over the tokens that exist);
// tokens [0, n_keep_head) and [N-n_keep_tail, N) are
// always selected; the remaining k - forced come from the other tokens in
// order (pooled desc, index asc) by a full sort; output ascending.
// Returns the number selected (min(k, N)) or < 0 on bad arguments.
int oracle_retrieve_topk(int dtype, int B, long long N, long long N_cap, int E, const void* bank,
                         int nq, const void* queries, double scale, int pool_window,
                         int n_keep_head, int n_keep_tail, int k, int32_t* idx_out,
                         double* ts_out, double* pooled_out, int pool_mode) {
  if (N > N_cap || nq < 1 || pool_window < 1 || pool_window % 2 == 0) return -1;
  if (pool_mode != 0 && pool_mode != 1) return -1;
  if (n_keep_head < 0 || n_keep_tail < 0 || n_keep_head + n_keep_tail > k) return -1;
  int n_out = (int)std::min<long long>(k, N);
  int r = (pool_window - 1) / 2;
  for (int b = 0; b < B; ++b) {
    std::vector<double> ts((size_t)N), pooled((size_t)N);
    parallel_for((size_t)N, [&](size_t t) {
      double best = -std::numeric_limits<double>::infinity();
      size_t row = ((size_t)b * N_cap + t) * (size_t)E;
      for (int qi = 0; qi < nq; ++qi) {
        size_t qo = ((size_t)b * nq + qi) * (size_t)E;
        double acc = 0.0;
        for (int e = 0; e < E; ++e) acc += load_elem(queries, dtype, qo + e) * load_elem(bank, dtype, row + e);
        acc *= scale;
        if (acc > best) best = acc;
      }
      ts[t] = best;
    });
    parallel_for((size_t)N, [&](size_t t) {
      long long lo = std::max<long long>(0, (long long)t - r);
      long long hi = std::min<long long>(N - 1, (long long)t + r);
      if (pool_mode == 0) {
        double best = ts[lo];
        for (long long u = lo + 1; u <= hi; ++u) best = std::max(best, ts[u]);
        pooled[t] = best;
      } else {
        double sum = 0.0;
        for (long long u = lo; u <= hi; ++u) sum += ts[u];
        pooled[t] = sum / (double)(hi - lo + 1);
      }
    });
    if (ts_out) std::memcpy(ts_out + (size_t)b * N, ts.data(), sizeof(double) * (size_t)N);
    if (pooled_out) std::memcpy(pooled_out + (size_t)b * N, pooled.data(), sizeof(double) * (size_t)N);
    std::vector<int32_t> sel;
    if (N <= k) {
      for (long long t = 0; t < N; ++t) sel.push_back((int32_t)t);
    } else {
      long long lo = n_keep_head, hi = N - n_keep_tail;
      std::vector<Cand> c;
      for (long long t = lo; t < hi; ++t) c.push_back({pooled[t], (int32_t)t});
      std::sort(c.begin(), c.end(), cand_before);
      int m = k - n_keep_head - n_keep_tail;
      for (long long t = 0; t < lo; ++t) sel.push_back((int32_t)t);
      for (int i = 0; i < m; ++i) sel.push_back(c[i].idx);
      for (long long t = hi; t < N; ++t) sel.push_back((int32_t)t);
      std::sort(sel.begin(), sel.end());
    }
    std::memcpy(idx_out + (size_t)b * k, sel.data(), sizeof(int32_t) * (size_t)n_out);
  }
  return n_out;
}

// Rotary position embedding with consecutive position ids (Sec. 3.1: after compression the
// cache rows are re-assigned consecutive ids, so row r of [cache ; chunk] sits at position
// pos_begin + (r - row_begin)).  For rows [row_begin, row_begin + rows) of x [B,H,cap,d]:
// pair (a, b) of a row is rotated by angle pos * base^(-2 i / d), i the pair index:
//   a' = a cos - b sin,  b' = b cos + a sin
// with the pair (x[i], x[i + d/2]) if interleaved == 0 ("rotate-half" layout of the Llama /
// Mistral family) or (x[2i], x[2i+1]) if interleaved != 0.  One rounding to the tensor dtype.
int oracle_rope(int dtype, int B, int H, int d, long long cap, long long row_begin, long long rows,
                long long pos_begin, double base, int interleaved, const void* src, void* dst) {
  if (d % 2 != 0 || row_begin < 0 || rows < 0 || row_begin + rows > cap || base <= 0.0) return -1;
  const int half = d / 2;
  size_t tasks = (size_t)B * H * (size_t)rows;
  parallel_for(tasks, [&](size_t t) {
    long long r = (long long)(t % (size_t)rows);
    size_t bh = t / (size_t)rows;
    size_t off = (bh * (size_t)cap + (size_t)(row_begin + r)) * (size_t)d;
    double pos = (double)(pos_begin + r);
    std::vector<double> y(d);
    for (int i = 0; i < half; ++i) {
      double ang = pos * std::pow(base, -2.0 * i / d);
      double c = std::cos(ang), s = std::sin(ang);
      int ia = interleaved ? 2 * i : i, ib = interleaved ? 2 * i + 1 : i + half;
      double a = load_elem(src, dtype, off + ia), b = load_elem(src, dtype, off + ib);
      y[ia] = a * c - b * s;
      y[ib] = b * c + a * s;
    }
    for (int e = 0; e < d; ++e) store_elem(dst, dtype, off + e, y[e]);
  });
  return 0;
}

// dst[b, r, :] = src[b, idx[b, r], :], rows of row_bytes bytes.
int oracle_gather(int B, long long n_rows, long long row_bytes, const void* src, const int32_t* idx,
                  int k, void* dst) {
  for (int b = 0; b < B; ++b) {
    for (int r = 0; r < k; ++r) {
      long long j = idx[(size_t)b * k + r];
      if (j < 0 || j >= n_rows) return -1;
      std::memcpy((char*)dst + ((size_t)b * k + r) * (size_t)row_bytes,
                  (const char*)src + ((size_t)b * n_rows + j) * (size_t)row_bytes, (size_t)row_bytes);
    }
  }
  return 0;
}

}  // extern "C"
