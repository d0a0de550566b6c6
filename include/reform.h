/*
 * reform.h -- C ABI of the REFORM compress-and-gather core for NVIDIA B200
 * (sm_100a).
 *
 * Five operations, in the order the method calls them while it walks a long
 * input chunk by chunk (Alg. 1, procedures ForwardChunk and REFORM):
 *
 *   reform_chunk_step     attention of one chunk over [compressed KV cache ;
 *                         chunk KV] that also emits the per-key eviction score
 *   reform_embed_append   per-head L2-normalised QKV states appended to the
 *                         cross-layer context-embedding bank
 *   reform_evict_topk     compacts each KV head's cache back to its budget
 *   reform_retrieve_topk  cosine scan of the bank against the query
 *                         embeddings, pooling, top-k token selection
 *   reform_gather         copies the selected rows into a contiguous buffer
 * and, beside the path, reform_rope (rotary embedding at the consecutive
 * position ids the compression re-assigns).
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers unless a field says "host".
 *     The caller owns every buffer; the library allocates nothing and keeps
 *     no pointer after the call returns.  Its global state is: a per-thread
 *     record of the last CUDA error and of the last selection's launch form
 *     (reform_debug_last_path), a launch counter, one error word per
 *     device (reform_device_error) and, per device, the fixed scratch array
 *     of reform_evict_topk_static (REFORM_EVICT_STATIC_BYTES).
 *   - Work is enqueued on the caller's stream and the call returns without
 *     synchronising.  Results are valid once the stream reaches that point.
 *   - Tensors are dense, row-major, innermost dimension contiguous; device
 *     pointers must be 16-byte aligned.
 *   - Every params struct starts with struct_size = sizeof(the struct); a
 *     mismatch returns REFORM_ERR_INVALID_ARG (guards against ABI drift).
 *   - dev_status (optional, device int32): a kernel that gives up on a bounded
 *     wait, or meets an out-of-range index, ORs a REFORM_DEV_* bit into it
 *     instead of trapping; the context stays usable.  The caller zeroes and
 *     reads it.  The same bits are also kept in a per-device word inside the
 *     library (reform_device_error), so a failure is visible without it.
 *   - workspace: scratch device memory, at least reform_*_workspace_size()
 *     bytes, 256-byte aligned, private to the call while it is in flight.
 *   - Return value: REFORM_OK or a negative REFORM_ERR_* code.  On any error
 *     nothing has been launched.
 *   - Indices are int32.  NaN inputs are outside the contract.  Batched
 *     calls take at most 65,535 (sequence, head) pairs: B * Hq for the chunk
 *     step, B * Hkv for the eviction, B for the retrieval; more is
 *     REFORM_ERR_INVALID_ARG.  A workspace-size query returns 0 for arguments
 *     the call itself would reject.
 */
#ifndef REFORM_H_
#define REFORM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* reform_stream_t; /* a cudaStream_t */

enum {
  REFORM_OK = 0,
  REFORM_ERR_INVALID_ARG = -1, /* NULL pointer, bad size, bad struct_size, misaligned pointer */
  REFORM_ERR_UNSUPPORTED = -2, /* dtype / head dimension the kernels do not cover */
  REFORM_ERR_WORKSPACE = -3,   /* workspace missing or too small */
  REFORM_ERR_CUDA = -4,        /* a CUDA call failed; see reform_last_cuda_error() */
  REFORM_ERR_TOO_LARGE = -5    /* problem exceeds the built-in scratch of a *_static entry point */
};

enum { REFORM_F32 = 0, REFORM_BF16 = 1 };

/* bits a kernel may OR into *dev_status */
enum {
  REFORM_DEV_TIMEOUT = 1,     /* a bounded wait inside a kernel expired */
  REFORM_DEV_BAD_INDEX = 2    /* an index outside its range was skipped */
};

/* flags of reform_chunk_step */
enum {
  REFORM_SCORE_ACCUMULATE = 1u, /* score[j] += carried score for cache rows j < n_cache */
  REFORM_NO_SCORE = 2u,         /* skip the key-score pass (plain prefill attention) */
  REFORM_FORCE_SIMT = 4u,       /* use the CUDA-core kernels even where a tensor-core path exists */
  REFORM_ROPE = 8u,             /* q and k are un-rotated: apply the rotary embedding inside the call */
  REFORM_ROPE_INTERLEAVED = 16u /* with REFORM_ROPE: pairs are (x[2i], x[2i+1]) instead of (x[i], x[i+d/2]) */
};

/* pooling of the token scores in reform_retrieve_topk */
enum { REFORM_POOL_MAX = 0, REFORM_POOL_MEAN = 1 };

/* kinds of state a context-embedding slot can come from */
enum { REFORM_STATE_Q = 0, REFORM_STATE_K = 1, REFORM_STATE_V = 2 };

/* ------------------------------------------------------------------------
 * reform_chunk_step -- Sec. 3.1 "recurrent chunked forwarding" (Fig. 1 step 1)
 * fused with the H2O eviction score of Sec. 3.1 / Sec. 4 "Common setup".
 *
 * For every batch b, query head h (KV head g = h / (Hq/Hkv)) and chunk row i:
 *   visible keys j: cache rows [0, n_cache) and chunk rows [n_cache, n_cache+i]
 *   s_ij = softmax_scale * <q_i, k_j>;  p_ij = softmax over visible j
 *   out_i = sum_j p_ij v_j;  lse_i = log sum_j exp(s_ij)   (natural log)
 * and, unless REFORM_NO_SCORE, for every KV head g and key j < n_cache+Lc:
 *   score[g][j] = (ACCUMULATE && j < n_cache ? score[g][j] : 0)
 *                 + sum_{h in group g} sum_{i >= Lc - score_window} p_ij
 *
 *   q      [B,Hq,Lc,d]    in
 *   k, v   [B,Hkv,cap,d]  in; rows [0,n_cache) hold the compressed cache and
 *                         rows [n_cache, n_cache+Lc) this chunk (caller wrote them)
 *   out    [B,Hq,Lc,d]    out, same dtype as q
 *   lse    [B,Hq,Lc]      fp32 out; may be NULL if the workspace holds room for it
 *   score  [B,Hkv,cap]    fp32 in/out; rows [0, n_cache+Lc) are written
 * d is 64 or 128.  dtype REFORM_BF16 with d == 128 runs on the tensor cores
 * (fp32 accumulate); REFORM_F32, and bf16 with d == 64, run on CUDA cores.
 * Decode-shaped steps (bf16, d == 128, Lc * Hq / Hkv <= 16: a few new tokens
 * over the recomputed cache) take a split-key kernel that needs workspace for
 * its partial results even when lse is given: always size the workspace with
 * reform_chunk_step_workspace_size().
 * softmax_scale 0 means 1/sqrt(d).  score_window in [1, Lc].
 *
 * REFORM_ROPE (Sec. 3.1, position re-assignment after compression): the cache
 * keeps un-rotated keys because every eviction renumbers its rows, so q and k
 * are passed un-rotated and the call rotates them at the ids of the moment --
 * row r of [cache ; chunk] at position r, chunk query i at n_cache + i, angle
 * pos * rope_theta^(-2 pair / d) as in reform_rope -- and computes out, lse and
 * score from the rotated operands.  q and k themselves are not modified.  On
 * the tensor-core path each query tile is rotated in shared memory right after
 * it is loaded; the keys, which every block re-reads, are rotated once per call
 * into the workspace (as are the score window's query rows), so size the
 * workspace with reform_chunk_step_workspace_size().  rope_theta 0 means 10000.
 * ------------------------------------------------------------------------ */
typedef struct reform_chunk_params {
  size_t struct_size;
  int32_t dtype;
  int32_t B, Hq, Hkv, d;
  int32_t Lc, n_cache, cap;
  int32_t score_window;
  float softmax_scale;
  uint32_t flags;
  float rope_theta;
  const void* q;
  const void* k;
  const void* v;
  void* out;
  float* lse;
  float* score;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
} reform_chunk_params;

size_t reform_chunk_step_workspace_size(const reform_chunk_params* p);
int reform_chunk_step(const reform_chunk_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_evict_topk -- Sec. 3.1 cache compression (Fig. 1 step 3); the initial
 * and the most recent rows are never evicted (Sec. 4, common setup).
 *
 * Independently for every (b, KV head): if n_keys <= budget all rows are
 * kept.  Otherwise the first n_sink and last n_recent rows are kept, plus the
 * budget - n_sink - n_recent rows of [n_sink, n_keys - n_recent) with the
 * largest score; equal scores go to the lower index (-0 counts as +0).  Kept
 * rows are written in ascending source order, so cache row r can take
 * position id r (the consecutive re-assignment of Sec. 3.1).
 *
 *   k_src, v_src [B,Hkv,cap_src,d] in;   score_src [B,Hkv,cap_src] fp32 in
 *   pos_src      [B,Hkv,cap_src] int32 in, optional (NULL)
 *   k_dst, v_dst [B,Hkv,cap_dst,d] out;  score_dst [B,Hkv,cap_dst] fp32 out
 *   pos_dst      optional; kept_idx [B,Hkv,budget] int32 out, optional
 * Rows [0, n_kept) of the destinations are written, n_kept = min(n_keys,
 * budget), also stored to *n_kept_host (host int32, optional) before return.
 * n_sink + n_recent > budget, or n_kept > cap_dst, is REFORM_ERR_INVALID_ARG.
 *
 * In place: the destinations may BE the sources -- k_dst == k_src, v_dst ==
 * v_src, score_dst == score_src, pos_dst == pos_src, cap_dst == cap_src, all
 * of them or none (a mixture, or any other overlap, is outside the contract;
 * equal pointers in a mixture are REFORM_ERR_INVALID_ARG).  The kept rows then
 * move down inside their own buffers and a layer needs one K/V buffer instead
 * of two.  In place needs rows of at most 256 bytes and either segments of
 * at most 131,072 keys (one thread-block cluster per segment, any number of
 * segments) or a shape whose selection blocks fit the device at once (segments
 * up to 262,144 keys, about a device's worth of 8,192-key blocks per call);
 * otherwise the call returns REFORM_ERR_UNSUPPORTED and nothing is launched.
 * The workspace needs no clearing between calls.
 * ------------------------------------------------------------------------ */
typedef struct reform_evict_params {
  size_t struct_size;
  int32_t dtype;
  int32_t B, Hkv, d;
  int32_t n_keys, cap_src, cap_dst;
  int32_t budget, n_sink, n_recent;
  const void* k_src;
  const void* v_src;
  const float* score_src;
  const int32_t* pos_src;
  void* k_dst;
  void* v_dst;
  float* score_dst;
  int32_t* pos_dst;
  int32_t* kept_idx;
  int32_t* n_kept_host;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
} reform_evict_params;

size_t reform_evict_topk_workspace_size(const reform_evict_params* p);
int reform_evict_topk(const reform_evict_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_evict_topk_static -- the paper has no counterpart; this is a
 * packaging variant of reform_evict_topk for callers that cannot allocate
 * device memory and so have no workspace to pass: for example a serving
 * process that handed all of HBM to its KV-cache pool at start-up (a later
 * cudaMalloc would simply fail), or a latency-critical loop in which the
 * device-wide synchronisation that cudaMalloc / cudaFree imply is not allowed.
 *
 * Same arguments, same results and same kernels as reform_evict_topk, except
 * that p->workspace and p->workspace_bytes are ignored: the scratch (the
 * selection histograms and counters, and the kept-index list when p->kept_idx
 * is NULL) lives in a fixed array inside the library, REFORM_EVICT_STATIC_BYTES
 * large, that every GPU which loads the library holds until the process exits.
 * The call allocates nothing and frees nothing.
 *
 * Limits: B * Hkv <= REFORM_EVICT_STATIC_MAX_SEGS, n_keys <=
 * REFORM_EVICT_STATIC_MAX_KEYS, budget <= REFORM_EVICT_STATIC_MAX_BUDGET;
 * anything larger returns REFORM_ERR_TOO_LARGE and launches nothing.
 *
 * The first call on each device looks up the array's device address (with
 * that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps the previous call's
 * contents (the call clears what must start at zero): two calls that overlap
 * on the GPU -- different streams, or different host threads -- race on it.
 * Calls on one stream are safe.
 * ------------------------------------------------------------------------ */
#define REFORM_EVICT_STATIC_MAX_SEGS 32
#define REFORM_EVICT_STATIC_MAX_KEYS 65536
#define REFORM_EVICT_STATIC_MAX_BUDGET 16384
#define REFORM_EVICT_STATIC_BYTES (3u << 20)

int reform_evict_topk_static(const reform_evict_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_debug_evict_wait_expiry -- diagnostic, no counterpart in the paper.
 * The kernels of this library never spin without a limit: a block that polls
 * for another block, for a copy or for the tensor cores gives up after a
 * bounded time, raises REFORM_DEV_TIMEOUT and lets the launch wind down with
 * the context intact (the blocks of a thread-block cluster meet at the
 * hardware's cluster barrier instead, which involves no polling loop).  This
 * entry point lets a test see that happen without faulting anything: it runs
 * reform_evict_topk's cooperative one-launch form with the
 * hand-off waits limited to wait_cycles SM clock cycles and with every
 * selection block waiting for one block more than the launch has -- a flag
 * that nothing ever sets.  Every block's first wait therefore runs out; the
 * kernel returns, REFORM_DEV_TIMEOUT is set in *p->dev_status and in the
 * per-device error word, and the outputs are unspecified.  The call after it
 * behaves as if this one had not happened.
 * Arguments as for reform_evict_topk.  wait_cycles in (0, 400,000,000].
 * REFORM_ERR_UNSUPPORTED if the shape cannot take that form
 * (nothing to choose, 48 or more short segments, more blocks than fit the
 * device at once).
 * ------------------------------------------------------------------------ */
int reform_debug_evict_wait_expiry(const reform_evict_params* p, long long wait_cycles,
                                   reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_embed_append -- Sec. 3.2 "Combining multiple heads":
 *   e_comb = concat_i ( e_i / ||e_i|| ).
 *
 * For every b, chunk token t and selected (kind, head, slot):
 *   bank[b, token_offset + t, slot*d : (slot+1)*d] = x / max(||x||_2, eps)
 * with x the d-vector of that head's Q, K or V state for token t.  Norm and
 * quotient are computed in fp32 for a bf16 bank and in fp64 for an fp32 bank,
 * then rounded once (nearest-even) to the bank dtype: every element is within
 * one unit in the last place of the exact quotient.
 *
 *   q_state [B,Hq,Lc,d]; k_state, v_state [B,Hkv,Lc,d]  in; a kind that no
 *                         selection uses may be NULL
 *   sel     host array of n_sel (<= REFORM_MAX_SEL) entries, read during the call
 *   bank    [B,N_cap,E]   in/out, same dtype as the states; (slot+1)*d <= E
 * eps 0 means 1e-12.  token_offset + Lc <= N_cap.
 * ------------------------------------------------------------------------ */
#define REFORM_MAX_SEL 16

typedef struct reform_head_sel {
  int32_t kind; /* REFORM_STATE_Q / _K / _V */
  int32_t head;
  int32_t slot;
} reform_head_sel;

typedef struct reform_embed_params {
  size_t struct_size;
  int32_t dtype;
  int32_t B, Lc, d, Hq, Hkv;
  int32_t n_sel;
  int32_t E;
  int64_t N_cap;
  int64_t token_offset;
  float eps;
  const reform_head_sel* sel; /* host */
  const void* q_state;
  const void* k_state;
  const void* v_state;
  void* bank;
  int32_t* dev_status;
} reform_embed_params;

int reform_embed_append(const reform_embed_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_retrieve_topk -- Sec. 3.3 "Identification of significant inputs".
 *
 * Independently for every b:
 *   ts[t]     = max_q  scale * <queries[q], bank[t]>          t in [0, N)
 *   pooled[t] = max of ts over [t-r, t+r] clipped to [0, N),  r = (pool_window-1)/2
 *   selected  = tokens [0, n_keep_head) and [N - n_keep_tail, N), plus the
 *               k - n_keep_head - n_keep_tail other tokens with the largest
 *               pooled score (ties to the lower index), ascending.
 * With pool_mode == REFORM_POOL_MEAN, pooled[t] is instead the mean of ts over
 * the same clipped window (divided by the number of tokens in it): the
 * smoothing the paper applies when it ranks heads (Appendix, detailed head
 * selection, Step 3: mean over a token and its 20 neighbours is pool_window =
 * 21).  The window is summed directly, so this mode costs O(pool_window) per
 * token.
 * Bank rows are stored per-head normalised (reform_embed_append), so the
 * cosine of Sec. 3.2 is this dot product with scale = 1 / n_slots.
 *
 *   bank     [B,N_cap,E] in;  queries [B,nq,E] in, same dtype
 *   idx_out  [B,k] int32 out; the first n_out = min(k, N) entries of each row are written
 *   token_score_out, pooled_score_out [B,N] fp32 out, optional (NULL)
 * pool_window odd >= 1.  n_keep_head + n_keep_tail > k is REFORM_ERR_INVALID_ARG.
 * ------------------------------------------------------------------------ */
typedef struct reform_retrieve_params {
  size_t struct_size;
  int32_t dtype;
  int32_t B;
  int64_t N, N_cap;
  int32_t E, nq;
  float scale;
  int32_t pool_window;
  int32_t n_keep_head, n_keep_tail;
  int32_t k;
  int32_t pool_mode; /* REFORM_POOL_MAX or REFORM_POOL_MEAN */
  const void* bank;
  const void* queries;
  int32_t* idx_out;
  float* token_score_out;
  float* pooled_score_out;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
} reform_retrieve_params;

size_t reform_retrieve_topk_workspace_size(const reform_retrieve_params* p);
int reform_retrieve_topk(const reform_retrieve_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_gather -- Sec. 3.3, collecting the input embeddings of the selected
 * tokens (Alg. 1, GatherRelevant).
 *
 *   dst[b, r, :] = src[b, idx[b, r], :]      r in [0, k)
 *   src [B,n_rows,row_bytes] in; idx [B,k] int32 in; dst [B,k,row_bytes] out
 * row_bytes is a multiple of 16.  An index outside [0, n_rows) zero-fills its
 * row and sets REFORM_DEV_BAD_INDEX in *dev_status; no out-of-range access
 * is made.
 * src is any address the device can read: device memory, or page-locked host
 * memory under unified addressing (cudaHostAlloc, cudaHostRegister).  In the
 * second case only the k selected rows of each sequence cross the bus, which
 * is what a caller wants whose input embeddings of a million-token context
 * stay in host memory.  idx and dst are device memory.
 * ------------------------------------------------------------------------ */
typedef struct reform_gather_params {
  size_t struct_size;
  int32_t B;
  int32_t k;
  int64_t n_rows;
  int64_t row_bytes;
  const void* src;
  const int32_t* idx;
  void* dst;
  int32_t* dev_status;
} reform_gather_params;

int reform_gather(const reform_gather_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------
 * reform_rope -- Sec. 3.1, position re-assignment after compression: the rows
 * that survive an eviction are renumbered 0, 1, 2, ... in cache order.
 * The cache therefore keeps un-rotated keys, and a step rotates its operands
 * with the ids of the moment: cache row r at position r, chunk row i at
 * n_cache + i (queries likewise).  This call applies the rotary embedding to
 * rows [row_begin, row_begin + rows) of every (b, head) at consecutive
 * positions pos_begin, pos_begin + 1, ...:
 *   angle = pos * theta_base^(-2 i / d)           i = pair index in [0, d/2)
 *   a' = a cos(angle) - b sin(angle);   b' = b cos(angle) + a sin(angle)
 * with pair i = (x[i], x[i + d/2]) (interleaved == 0, the rotate-half layout
 * of the Llama / Mistral family) or (x[2i], x[2i+1]) (interleaved != 0).
 * Angles are reduced to [-pi, pi] in fp64 and their sine and cosine evaluated
 * in fp32 (absolute error about 1e-7), the rotation in fp32, one rounding to
 * dtype.
 *
 *   src [B,H,cap,d] in;  dst [B,H,cap,d] out (may be src: in place); rows
 *   outside the range are not touched.  theta_base 0 means 10000.
 * d * sizeof(dtype) must be a multiple of 32 and d at most 512
 * (REFORM_ERR_UNSUPPORTED otherwise).
 * ------------------------------------------------------------------------ */
typedef struct reform_rope_params {
  size_t struct_size;
  int32_t dtype;
  int32_t B, H, d;
  int32_t interleaved;
  int64_t cap;
  int64_t row_begin, rows;
  int64_t pos_begin;
  float theta_base;
  const void* src;
  void* dst;
  int32_t* dev_status;
} reform_rope_params;

int reform_rope(const reform_rope_params* p, reform_stream_t stream);

/* ------------------------------------------------------------------------ */
const char* reform_status_string(int status);
/* cudaError_t of the last failed CUDA call made by this thread (0 if none). */
int reform_last_cuda_error(void);
/* REFORM_DEV_* bits that kernels of this library have raised on the current device since the last
 * clear (whether or not the failing call was given a dev_status word), or REFORM_ERR_CUDA.  Reads
 * device memory with a blocking copy: synchronise the streams of interest first.  clear != 0
 * resets the word. */
int reform_device_error(int clear);
/* major * 10000 + minor * 100 + patch */
int reform_version(void);
/* Number of kernels this library has launched from the calling process since
 * load (monotonic; for accounting in benchmarks). */
long long reform_kernel_launch_count(void);
/* Which launch form the last reform_evict_topk (or _static) or reform_retrieve_topk call made by
 * this thread chose for its selection (diagnostic; the results do not depend on it). */
enum {
  REFORM_PATH_NONE = 0,        /* no such call yet, or nothing to select */
  REFORM_PATH_CLUSTER = 1,     /* one thread-block cluster per segment, one launch */
  REFORM_PATH_COOPERATIVE = 2, /* one cooperative launch over global-memory hand-offs */
  REFORM_PATH_PER_SEGMENT = 3, /* one block per segment (many short segments), then the row copy */
  REFORM_PATH_PER_PASS = 4     /* one launch per radix pass, then the row copy */
};
int reform_debug_last_path(void);

#ifdef __cplusplus
}
#endif
#endif /* REFORM_H_ */
