/*
 * s4r.h - C ABI of the B200 (sm_100a) library for the S4R decode hot path
 * (arXiv 2608.00528: low-rank KV-cache compression with latent-space scoring
 * and sparse reconstruction).
 *
 * Citations name the paper's sections; equations of Sec. 3 are unnumbered in
 * the paper, so "Eq. n" is the n-th displayed equation of Sec. 3 in order of
 * appearance (Eq. 3: C = S B; Eq. 5: per-step projection; Eq. 6: append;
 * Eq. 8: latent logits; Eq. 9: softmax; Eq. 11: pooling; Eq. 12: group
 * aggregation; Eq. 13-15: local window, top-k, union; Eq. 16: sparse
 * reconstruction; Eq. 17: sink concatenation; Eq. 18: attention with RoPE).
 *
 * General rules
 *   - Unless an argument is documented as HOST memory, every data pointer is a
 *     DEVICE pointer owned by the caller.  The library never allocates or
 *     frees device memory, keeps no state between calls (except the opt-in
 *     stage timing below) and never synchronises the stream (except
 *     s4r_decode_step_host, s4r_append_decode_step_host and s4r_stage_times,
 *     see there).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *     work of a call is enqueued on it, in order.  The device-pointer calls
 *     may be captured into a CUDA graph (after one uncaptured call on the
 *     device): while the stream is capturing, the decode step projects the
 *     query in a kernel of its own instead of inside the scoring kernel, so
 *     that nothing in the captured arguments is specific to one call.
 *   - On sm_100 with bf16 storage the scoring kernel's CTAs of one sequence
 *     exchange partial sums of the per-step projections and wait for one
 *     another (bounded).  The launch is sized to one CTA per SM and the host
 *     checks that the device can hold all of them; if other work keeps them
 *     apart for more than a second the call ends with S4R_DEV_TIMEOUT.
 *   - Every entry point returns S4R_OK or a negative s4r_status_t.  Misuse
 *     that the host can see is rejected before anything is launched.
 *   - `dev_status` (may be NULL) is a device int32 the kernels OR flags into
 *     (S4R_DEV_*); kernels never trap and never spin without a bound.
 *   - Tensors are dense, row-major, last index fastest.  Storage type
 *     (`dtype`) applies to K, V, q, sinks, bases and coefficients alike.
 *   - There is no CPU fallback and no other GPU architecture: on a device that
 *     is not compute capability 10.x the calls return S4R_ERR_ARCH.
 *
 * Notation (paper, App. A): B batch, H_q query heads, h_kv KV heads,
 * G = H_q / h_kv, d_h head dimension, D' = h_kv * d_h, r rank, s sink count,
 * L non-sink cache length INCLUDING the current token (Sec. 3.2.2), W local
 * window, k global top-k budget.
 */
#ifndef S4R_H_
#define S4R_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  S4R_OK = 0,
  S4R_ERR_INVALID_ARG = -1, /* NULL pointer, negative size, inconsistent geometry          */
  S4R_ERR_UNSUPPORTED = -2, /* valid in the paper, not built here (see each call)           */
  S4R_ERR_WORKSPACE = -3,   /* workspace missing, misaligned (256 B) or too small           */
  S4R_ERR_CUDA = -4,        /* a CUDA runtime call failed (launch error, bad stream, ...)   */
  S4R_ERR_ARCH = -5         /* current device is not sm_100                                 */
} s4r_status_t;

/* flags OR-ed into *dev_status by kernels */
#define S4R_DEV_TIMEOUT 1  /* a bounded wait (mbarrier) expired; results of that call are invalid */
#define S4R_DEV_BOUNDS 2   /* coef_len[b] outside [0, max_len] or cache full on append; clamped   */
#define S4R_DEV_NUMERIC 4  /* s4r_build_basis met a pivot that was not positive (rank-deficient sample) */

#define S4R_F32 0
#define S4R_BF16 1

#define S4R_POOL_MAX 0
#define S4R_POOL_AVG 1
#define S4R_GROUP_MEAN 0
#define S4R_GROUP_MAX 1
#define S4R_VALUE_AUTO 0
#define S4R_VALUE_RECONSTRUCT 1

/* Layer geometry, validated on every call.
 * Supported: head_dim 128 (also 64), G <= 8, rank_k and rank_v multiples of 8 in [8, 512],
 * rank_k == rank_v not required. */
typedef struct {
  int32_t batch;         /* B >= 1                                                        */
  int32_t n_q_heads;     /* H_q, multiple of n_kv_heads                                    */
  int32_t n_kv_heads;    /* h_kv                                                           */
  int32_t head_dim;      /* d_h                                                            */
  int32_t rank_k;        /* r of the key subspace                                          */
  int32_t rank_v;        /* r of the value subspace                                        */
  int32_t sink_count;    /* s >= 0 (Sec. 3.1.1; s = 0 is the "without sinks" ablation)     */
  int32_t dtype;         /* S4R_BF16 or S4R_F32                                            */
  int64_t coef_capacity; /* rows allocated per sequence in coef_k and coef_v               */
} s4r_layer_t;

/* Switches of the relevance estimate (Eq. 9-12); the paper's defaults are
 * pool_kernel 7, max pooling, mean aggregation. */
typedef struct {
  int32_t score_window; /* W_q, query-coefficient rows scored (Eq. 7, 9, 10): 1 = the current query alone; more
                           than 1 only through s4r_decode_step_windowed */
  int32_t pool_kernel;  /* kappa, odd, 1 = no pooling, <= 31                              */
  int32_t pool_mode;    /* S4R_POOL_MAX | S4R_POOL_AVG                                    */
  int32_t group_mode;   /* S4R_GROUP_MEAN | S4R_GROUP_MAX                                 */
  int32_t value_path;   /* S4R_VALUE_AUTO (0) | S4R_VALUE_RECONSTRUCT: how Eq. 16-18 treat the values.
                         * RECONSTRUCT forms V^ = C^V[sel] (B^V)^T on chip and then P V^, literally Eq. 16.
                         * AUTO lets the library evaluate the same product as (P C^V[sel]) (B^V)^T where that is
                         * faster (bf16, head_dim 128); the two agree up to fp32 rounding order.             */
} s4r_score_t;

/* RoPE of Eq. 18: rotate-half pairing (i, i + d_h/2), inv_freq_i = theta^(-2i/d_h), no scaling.
 * Sink j sits at position j, non-sink row l at s + l, the query at s + L - 1.  theta <= 0: off. */
typedef struct {
  float theta;
  int32_t reserved; /* must be 0 */
} s4r_rope_t;

/* Bytes of scratch s4r_decode_step / s4r_compress need for this geometry when no sequence is longer
 * than max_len non-sink rows (compress: max_len = T - s).  0 on invalid arguments.  The workspace
 * must be 256-byte aligned; its contents are undefined between calls. */
size_t s4r_workspace_bytes(const s4r_layer_t *layer, int64_t max_len, int32_t window, int32_t top_k);

/* The same for s4r_decode_step_windowed with W_q = score_window (1 <= W_q <= S4R_MAX_SCORE_WINDOW, else 0). */
#define S4R_MAX_SCORE_WINDOW 128
size_t s4r_workspace_bytes_windowed(const s4r_layer_t *layer, int64_t max_len, int32_t window, int32_t top_k,
                                    int32_t score_window);

/* Subspace construction (Sec. 3.1.2; Eq. 1: sampled rows L2-normalised along the feature dimension, Eq. 2: the
 * top-r right singular vectors of the normalised sample), per sequence b and for ONE tensor (call it for the keys
 * with rank_k and for the values with rank_v):
 *   S_n[t]   = X[b, s + sample_idx[b, t]] / ||X[b, s + sample_idx[b, t]]||        t = 0 .. n_samples - 1
 *   basis[b] = [D', rank] the rank leading right singular vectors of S_n, column i scaled by the sign that makes
 *              its largest-magnitude entry positive (lowest index on ties), rounded to the layer dtype
 *   sigma[b] = [rank] fp32 singular values (optional, may be NULL)
 * X          [B, T, D'] pre-RoPE rows INCLUDING the s sink rows (device, layer dtype)
 * sample_idx [B, n_samples] int32 NON-SINK indices in [0, T - s) (device); out-of-range entries set
 *            S4R_DEV_BOUNDS and are clamped.  s4r_hybrid_sample_indices writes the paper's sampling pattern.
 * Method: block power iteration with r + 32 vectors on the Gram matrix S_n^T S_n, n_iter iterations (<= 0: 24; more
 * than 4096: S4R_ERR_INVALID_ARG),
 * Rayleigh-Ritz at the end; vector i converges like (sigma_{r+33} / sigma_i)^(2 n_iter), so the result is the
 * SVD's up to that error and fp32 rounding.  Singular vectors whose singular values are closer than that are
 * determined only as a subspace (by this routine as by any SVD in finite precision).
 * Requirements: rank % 8 == 0, rank + 32 <= min(D', n_samples), rank <= 200 (S4R_ERR_UNSUPPORTED otherwise).
 * workspace_bytes >= s4r_basis_workspace_bytes(...).  Asynchronous on `stream`.  A rank-deficient sample sets
 * S4R_DEV_NUMERIC (the basis is then not orthonormal). */
size_t s4r_basis_workspace_bytes(const s4r_layer_t *layer, int32_t rank, int32_t n_samples);
int s4r_build_basis(const s4r_layer_t *layer, const void *X, int64_t T, const int32_t *sample_idx, int32_t n_samples,
                    int32_t rank, int32_t n_iter, void *basis, float *sigma, void *workspace, size_t workspace_bytes,
                    int32_t *dev_status, void *stream);

/* Host helper: the paper's hybrid sampling (Sec. 3.1.2) over n_nonsink positions: a contiguous block of the
 * ceil(recent_frac * n_samples) most recent positions plus evenly spread early positions floor(j * early / n_u)
 * (duplicates removed).  Writes ascending indices to out (HOST, room for n_samples) and returns how many. */
int32_t s4r_hybrid_sample_indices(int64_t n_nonsink, int32_t n_samples, double recent_frac, int32_t *out);

/* Prefill-side projection (Sec. 3.1.1 sink split + Eq. 3), per sequence b:
 *   sink_k[b] = K[b, 0:s], sink_v[b] = V[b, 0:s]            (verbatim copies)
 *   coef_k[b, 0:T-s] = K[b, s:T] * key_basis[b]              (fp32 accumulate, one rounding to dtype)
 *   coef_v[b, 0:T-s] = V[b, s:T] * value_basis[b]
 *   coef_len[b] = T - s
 * K, V          [B, T, D'] pre-RoPE keys / values of the prompt, T >= s, T - s <= coef_capacity
 * key_basis     [B, D', rank_k], value_basis [B, D', rank_v]   (Eq. 2; computed by the caller)
 * norm_stats    reserved, must be NULL: the paper normalises only the sampled rows that build the
 *               bases (Eq. 1) and projects the raw rows (Eq. 3)
 * sink_k/v out  [B, s, D'];  coef_k out [B, coef_capacity, rank_k];  coef_v likewise;  coef_len out [B]
 */
int s4r_compress(const s4r_layer_t *layer, const void *K, const void *V, int64_t T, const void *key_basis,
                 const void *value_basis, const void *norm_stats, void *sink_k, void *sink_v, void *coef_k,
                 void *coef_v, int32_t *coef_len, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                 void *stream);

/* Decode-time cache update (Eq. 5 for K and V, Eq. 6), per sequence b:
 *   coef_k[b, coef_len[b]] = k_t[b] * key_basis[b];  coef_v likewise;  coef_len[b] += 1
 * k_t, v_t [B, D'] pre-RoPE.  A full cache (coef_len[b] == coef_capacity) sets S4R_DEV_BOUNDS and
 * leaves that sequence unchanged. */
int s4r_append(const s4r_layer_t *layer, const void *k_t, const void *v_t, const void *key_basis,
               const void *value_basis, void *coef_k, void *coef_v, int32_t *coef_len, int32_t *dev_status,
               void *stream);

/* One decode step of one layer for the whole batch (Sec. 3.2.2-3.2.3), per sequence b with L = coef_len[b]
 * (the current token already appended):
 *   1. c^Q[g] = Q~[g] key_basis, Q~[g] = concat over KV heads kv of query head kv*G+g        (Eq. 5)
 *   2. Z[g, l] = <c^Q[g], coef_k[l]> / sqrt(rank_k), l in [0, L)                              (Eq. 8)
 *   3. A[g, :] = softmax over l; pooled over kappa neighbours; aggregated over g -> score[l]   (Eq. 9-12)
 *   4. W_eff = min(window, L); local = [L - W_eff, L); k_eff = min(top_k, L - W_eff);
 *      global = the k_eff best of score[0 : L - W_eff], ties to the lower index                (Eq. 13-15)
 *   5. selected rows are reconstructed on chip, K^ = coef_k[sel] key_basis^T, V^ likewise     (Eq. 16),
 *      joined with the sinks (Eq. 17), rotated (RoPE, if on) and attended                      (Eq. 18)
 * q             [B, H_q, d_h] pre-RoPE
 * max_len       host-known upper bound of every coef_len[b] (<= coef_capacity); sizes grids and scratch
 * window, top_k W >= 0 and k >= 0
 * out           [B, H_q, d_h], type out_dtype (S4R_F32 or S4R_BF16)
 * sel_idx       [B, window + top_k] int32: global picks ascending, then the local window ascending, as
 *               non-sink indices (absolute position = s + index); unused tail = -1.  Sinks are always
 *               attended and never listed.
 * sel_count     [B] int32 = W_eff + k_eff
 * Returns S4R_ERR_UNSUPPORTED for score->score_window != 1 (see s4r_decode_step_windowed). */
int s4r_decode_step(const s4r_layer_t *layer, const void *q, const void *sink_k, const void *sink_v,
                    const void *coef_k, const void *coef_v, const int32_t *coef_len, const void *key_basis,
                    const void *value_basis, int64_t max_len, int32_t window, int32_t top_k,
                    const s4r_score_t *score, const s4r_rope_t *rope, void *out, int32_t out_dtype,
                    int32_t *sel_idx, int32_t *sel_count, void *workspace, size_t workspace_bytes,
                    int32_t *dev_status, void *stream);

/* The decode step with the paper's full relevance estimator (Sec. 3.2.2): a FIFO of the W_q = score->score_window
 * most recent projected queries scores the cache instead of the current query alone.
 *   Eq. 7   the window drops its oldest row and appends c^Q of the current query (so it always holds W_q rows)
 *   Eq. 8-9 window row i (0 = oldest) belongs to the token at non-sink index L - W_q + i; its latent logits are
 *           softmax-normalised over the rows l <= L - W_q + i it may see (causal mask); rows with a negative
 *           index see nothing
 *   Eq. 10  the W_q probability rows of a query group are averaged (divided by W_q)
 * followed by pooling, group aggregation, selection, reconstruction and attention exactly as in s4r_decode_step.
 * query_window  [B, W_q, G, rank_k] fp32, caller-owned per-layer state, oldest row first; updated in place.  Before
 *               the first step the caller fills rows 1..W_q-1 with the coefficients of the W_q - 1 preceding
 *               queries (Eq. 4: C^Q = Q~ B^K; zeros if there are none) - row 0 is dropped by that step.
 * Built for bf16 caches with rank_k a multiple of 64 (at most 320) on sm_100; S4R_ERR_UNSUPPORTED otherwise and
 * for W_q > S4R_MAX_SCORE_WINDOW.  Whole query groups with at most 128 window rows together are scored by one
 * pair of passes over C^K (row normalisers, then the window mean): one pair for G * W_q <= 128, ceil(G /
 * floor(128 / W_q)) pairs otherwise.  The window rows enter the tensor-core product as two bf16 terms (16
 * mantissa bits), so a logit carries a relative error of about 2^-17.
 * workspace_bytes >= s4r_workspace_bytes_windowed(...).  All other arguments as in s4r_decode_step. */
int s4r_decode_step_windowed(const s4r_layer_t *layer, const void *q, const void *sink_k, const void *sink_v,
                             const void *coef_k, const void *coef_v, const int32_t *coef_len, const void *key_basis,
                             const void *value_basis, int64_t max_len, int32_t window, int32_t top_k,
                             const s4r_score_t *score, const s4r_rope_t *rope, float *query_window, void *out,
                             int32_t out_dtype, int32_t *sel_idx, int32_t *sel_count, void *workspace,
                             size_t workspace_bytes, int32_t *dev_status, void *stream);

/* s4r_append followed by s4r_decode_step_windowed as one call: the projection kernel that produces c^Q also projects
 * and appends the new token's rows (Eq. 5-6) and bumps coef_len, then the windowed step runs on the grown cache.
 * k_t, v_t [B, D'] pre-RoPE; coef_k, coef_v, coef_len are updated; max_len must bound coef_len[b] + 1. */
int s4r_append_decode_step_windowed(const s4r_layer_t *layer, const void *k_t, const void *v_t, const void *q,
                                    const void *sink_k, const void *sink_v, void *coef_k, void *coef_v,
                                    int32_t *coef_len, const void *key_basis, const void *value_basis, int64_t max_len,
                                    int32_t window, int32_t top_k, const s4r_score_t *score, const s4r_rope_t *rope,
                                    float *query_window, void *out, int32_t out_dtype, int32_t *sel_idx,
                                    int32_t *sel_count, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                    void *stream);

/* Initial query-coefficient window (Eq. 4: C^Q = Q~ B^K for the last prompt queries).
 * queries       [B, n_queries, H_q, d_h] (device, layer dtype), oldest first, pre-RoPE; 0 <= n_queries <= W_q
 * query_window  [B, W_q, G, rank_k] fp32 (device): rows W_q - n_queries .. W_q - 1 receive the coefficients of the
 *               queries, the rows before them zeros.  The first s4r_decode_step_windowed then drops row 0 and
 *               appends the first generated token's query.
 * Any geometry s4r_decode_step accepts.  Errors as s4r_append. */
int s4r_window_init(const s4r_layer_t *layer, const void *queries, int32_t n_queries, const void *key_basis,
                    float *query_window, int32_t score_window, void *stream);

/* s4r_append followed by s4r_decode_step as one call (Sec. 3.2.1 then 3.2.2-3.2.3): the new token's key and
 * value rows are projected in the same pass over the bases that projects the query (Eq. 5), appended
 * (Eq. 6), and the step then runs on the grown cache.  The new rows may differ from those of s4r_append by one
 * rounding of the storage type (the D' products are added in a different, equally fixed order).
 * k_t, v_t [B, D'] pre-RoPE; coef_k, coef_v, coef_len are updated; max_len must bound coef_len[b] + 1. */
int s4r_append_decode_step(const s4r_layer_t *layer, const void *k_t, const void *v_t, const void *q,
                           const void *sink_k, const void *sink_v, void *coef_k, void *coef_v, int32_t *coef_len,
                           const void *key_basis, const void *value_basis, int64_t max_len, int32_t window,
                           int32_t top_k, const s4r_score_t *score, const s4r_rope_t *rope, void *out,
                           int32_t out_dtype, int32_t *sel_idx, int32_t *sel_count, void *workspace,
                           size_t workspace_bytes, int32_t *dev_status, void *stream);

/* Same step for callers whose per-step data lives in HOST memory: q_host, out_host, sel_idx_host and
 * sel_count_host are host buffers (pinned memory makes the copies asynchronous); q_dev, out_dev,
 * sel_idx_dev, sel_count_dev are device staging buffers of the same shapes.  The call copies q to the
 * device, runs s4r_decode_step, copies out / sel_idx / sel_count back and waits for the stream, so the
 * host buffers are valid on return.  The cache itself (sinks, coefficients, bases) stays on the device:
 * it is the persistent state of Sec. 3.3, not a per-step input. */
int s4r_decode_step_host(const s4r_layer_t *layer, const void *q_host, void *q_dev, const void *sink_k,
                         const void *sink_v, const void *coef_k, const void *coef_v, const int32_t *coef_len,
                         const void *key_basis, const void *value_basis, int64_t max_len, int32_t window,
                         int32_t top_k, const s4r_score_t *score, const s4r_rope_t *rope, void *out_host,
                         void *out_dev, int32_t out_dtype, int32_t *sel_idx_host, int32_t *sel_idx_dev,
                         int32_t *sel_count_host, int32_t *sel_count_dev, void *workspace,
                         size_t workspace_bytes, int32_t *dev_status, void *stream);

/* The fused step (s4r_append_decode_step) for callers whose per-step data lives in HOST memory, with ONE copy
 * in each direction.  The inputs of a step are packed in one block {q, k_t, v_t} and the results in one block
 * {out, sel_idx, sel_count}; s4r_host_step_layout gives the byte offsets (each a multiple of 16):
 *   in_off [4] = offsets of q [B, H_q, d_h], k_t [B, D'], v_t [B, D'] (layer dtype) and the block size
 *   out_off[4] = offsets of out [B, H_q, d_h] (out_dtype), sel_idx [B, W + k] int32, sel_count [B] int32 and
 *                the block size
 * in_host / out_host are HOST blocks (pinned memory makes the copies asynchronous), in_dev / out_dev device
 * staging blocks of the same sizes, 16-byte aligned.  The call copies in_host to in_dev, runs the step, copies
 * out_dev to out_host and waits for the stream, so out_host is valid on return.  Errors as
 * s4r_append_decode_step. */
int s4r_host_step_layout(const s4r_layer_t *layer, int32_t window, int32_t top_k, int32_t out_dtype, size_t *in_off,
                         size_t *out_off);
int s4r_append_decode_step_host(const s4r_layer_t *layer, const void *in_host, void *in_dev, const void *sink_k,
                                const void *sink_v, void *coef_k, void *coef_v, int32_t *coef_len,
                                const void *key_basis, const void *value_basis, int64_t max_len, int32_t window,
                                int32_t top_k, const s4r_score_t *score, const s4r_rope_t *rope, void *out_host,
                                void *out_dev, int32_t out_dtype, void *workspace, size_t workspace_bytes,
                                int32_t *dev_status, void *stream);

/* The decode step for callers that cannot allocate device memory.  (The paper has no counterpart; this is
 * a property of the library, not of the method.)  Some callers have nowhere to get a workspace from: code
 * that runs where cudaMalloc is forbidden or would stall - inside a latency-critical serving loop whose
 * memory pool is already carved up, a plugin that is handed tensors but no allocator, a process that must
 * not touch the allocator after start-up.  For them the scratch of s4r_decode_step lives in a fixed array
 * inside the library (S4R_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library, held
 * until the process exits).  Arguments and results are exactly those of s4r_decode_step without
 * `workspace` / `workspace_bytes`; the call itself allocates and frees nothing.
 *   - Geometries whose s4r_workspace_bytes(...) exceeds S4R_STATIC_SCRATCH_BYTES are rejected with
 *     S4R_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address (a one-off query that also makes
 *     sure the module is loaded).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left in it; the step
 *     overwrites every scratch location before reading it, so nothing needs clearing - but two calls that
 *     overlap on the GPU (different streams, no ordering between them) race on it and corrupt each other.
 *     Keep calls on one device ordered. */
#define S4R_STATIC_SCRATCH_BYTES (16u << 20)
int s4r_decode_step_static(const s4r_layer_t *layer, const void *q, const void *sink_k, const void *sink_v,
                           const void *coef_k, const void *coef_v, const int32_t *coef_len,
                           const void *key_basis, const void *value_basis, int64_t max_len, int32_t window,
                           int32_t top_k, const s4r_score_t *score, const s4r_rope_t *rope, void *out,
                           int32_t out_dtype, int32_t *sel_idx, int32_t *sel_count, int32_t *dev_status,
                           void *stream);

/* Host helpers (no GPU work). */
/* Eq. 14: k = max(floor(rho * L) - W, 0). */
int64_t s4r_top_k_from_ratio(double rho, int64_t L, int32_t window);
/* Largest rank r (multiple of `multiple`) whose persistent memory ratio of Sec. 3.3,
 * (s D' + L r + G W r / 2 + D' r) / ((s + L) D'), does not exceed eta; 0 if none. */
int32_t s4r_rank_for_ratio(double eta, int64_t L, int32_t sink_count, int32_t d_kv, int32_t group,
                           int32_t query_window, int32_t multiple);
/* Number of kernel launches the last s4r_decode_step / s4r_compress / s4r_append call on this thread made. */
int32_t s4r_last_launch_count(void);

/* Opt-in per-stage timing for benchmarks (the only state the library keeps; off by default).
 * s4r_stage_timing(1) makes every later s4r_decode_step on this host thread record CUDA events on its
 * stream around its stages; s4r_stage_timing(0) switches it off again.  s4r_stage_times waits for the events
 * of the last step and writes up to n elapsed times in milliseconds, in stage order: 0 query projection
 * (Eq. 5), 1 latent scoring (Eq. 8), 2 relevance + selection (Eq. 9-15), 3 sparse reconstruction +
 * attention over the selected rows (Eq. 16-18), 4 merge with the sinks (Eq. 17-18).  Returns the number of
 * stages written, or a negative s4r_status_t. */
#define S4R_N_STAGES 5
int s4r_stage_timing(int enable);
int s4r_stage_times(float *ms_out, int n);

const char *s4r_strerror(int status);
/* Text of the last CUDA runtime error that made a call on this host thread return S4R_ERR_CUDA. */
const char *s4r_last_cuda_error(void);
int s4r_version(void);

#ifdef __cplusplus
}
#endif
#endif /* S4R_H_ */
