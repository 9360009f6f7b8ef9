/*
 * compactor.h - C ABI of the B200 (sm_100a) implementation of Compactor's prefill-time KV-cache
 * compression pass: approximate leverage scoring of the keys (Algorithm 1), optional blend with
 * a caller-supplied attention score (Eq. 6), per-head top-ceil(r N) selection (Section 3.4) and
 * compaction of the retained K/V rows into a dense per-head cache.
 *
 * Conventions
 *   - Every function returns an int status: COMPACTOR_OK (0) or a negative COMPACTOR_E_* code.
 *     Nothing throws.  Argument errors are detected before any work is enqueued.
 *   - "device" pointers are CUDA device pointers of the current device; "host" pointers are
 *     ordinary host memory, read before the call returns.  The library never allocates or frees
 *     device memory: every buffer, including the workspace, belongs to the caller.
 *   - Device work is enqueued on the caller's stream (`stream` is a cudaStream_t passed as
 *     void*; NULL is the default stream) and the call returns without synchronising.  Everything
 *     enqueued is a kernel or a memset (the prefix tables travel as kernel arguments, 239
 *     sequences per small launch), so the call can be recorded into a CUDA graph and replayed on
 *     new contents of the same buffers.
 *   - Keys/values are bf16 with the d channels of a token contiguous; the other three strides
 *     (layer, KV head, token) are given in ELEMENTS and must be multiples of 8 (16 bytes); base
 *     pointers must be 16-byte aligned.  d must be 128.  1 <= m <= 128.
 *   - Sequences are packed back to back along the token axis: sequence b owns tokens
 *     [cu_seqlens[b], cu_seqlens[b+1]) of every (layer, head).  A "unit" is one
 *     (layer, head, sequence) triple; unit id = (layer * heads + head) * batch + b.
 *     Units are scored and selected independently (Section 3, Notation: heads are treated
 *     one by one).
 *   - Kept rows of sequence b occupy rows [cu_keep[b], cu_keep[b+1]) of every (layer, head)
 *     block of the outputs, cu_keep = prefix sums of keep_counts; total_keep = cu_keep[batch].
 *   - Outputs must not alias inputs or the workspace.
 *   - `status` (device, int32 [layers*heads*batch], may be NULL) receives per-unit flags once the
 *     stream has run: bit 0 = the unit's Gram matrix held a non-finite value (scores of the unit
 *     are unspecified), bit 1 = the sketched Gram matrix was numerically rank deficient (the
 *     singular directions contribute nothing, as a pseudo-inverse would), bit 2 = a bounded
 *     device-side wait ran out.
 *   - On problems with at most 600 MB of keys the kernels of a call are launched as a chain of
 *     programmatic dependent launches (each may set up while its predecessor drains); results do
 *     not depend on it.  The library reads a few environment variables at every call, none of which
 *     changes a result: COMPACTOR_NO_PDL=1 (no chained launches), COMPACTOR_PDL_MASK,
 *     COMPACTOR_GRAM_BLOCK / COMPACTOR_SCORE_BLOCK (block lengths of the two sweeps, a power of two
 *     from 256 to 65536 tokens), COMPACTOR_FUSED_SWEEP and its companions (an experimental
 *     one-kernel sweep).  They are measuring aids; leave them unset.
 */
#ifndef COMPACTOR_H_
#define COMPACTOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define COMPACTOR_OK                  0
#define COMPACTOR_E_INVALID_ARGUMENT -1   /* null pointer, bad size, bad stride or alignment      */
#define COMPACTOR_E_UNSUPPORTED      -2   /* d != 128 or m outside [1, 128]                      */
#define COMPACTOR_E_WORKSPACE        -3   /* workspace smaller than compactor_workspace_bytes()  */
#define COMPACTOR_E_CUDA             -4   /* a CUDA runtime call failed (see cudaGetLastError)   */
#define COMPACTOR_E_TOO_LARGE        -5   /* problem exceeds the library's built-in scratch      */

#define COMPACTOR_STATUS_NONFINITE   1
#define COMPACTOR_STATUS_RANK        2
#define COMPACTOR_STATUS_TIMEOUT     4

/* Small factorisations for compactor_score_variant (Appendix C). */
#define COMPACTOR_FACTOR_CHOLESKY    0    /* G = L L^T: the R factor of the QR route          */
#define COMPACTOR_FACTOR_EIG         1    /* G = V Lambda V^T with a floor on the eigenvalues */

/* A strided bf16 tensor [layers][heads][total_tokens][d] in device memory. */
typedef struct compactor_mat {
    const void* ptr;          /* device, 16-byte aligned                           */
    int64_t stride_layer;     /* elements between consecutive layers               */
    int64_t stride_head;      /* elements between consecutive KV heads             */
    int64_t stride_token;     /* elements between consecutive tokens (>= d)        */
} compactor_mat;

/* Problem shape.  cu_seqlens is a HOST array of batch+1 non-decreasing offsets starting at 0. */
typedef struct compactor_shape {
    int32_t layers;
    int32_t heads;
    int32_t d;                /* head dimension; must be 128                       */
    int32_t m;                /* sketch dimension, 1..128 (the paper uses 48)      */
    int32_t batch;            /* number of packed sequences                        */
    const int32_t* cu_seqlens;/* host, [batch+1]                                   */
} compactor_shape;

/* Library version (major*10000 + minor*100 + patch). */
int compactor_version(void);

/* Static description of a status code. */
const char* compactor_error_string(int code);

/*
 * Algorithm 1, line 1: a Gaussian sketch Phi [d][m] (row-major fp32, HOST memory) with iid
 * N(0, 1/m) entries from a counter-based generator, so that any caller can reproduce it:
 * word i = splitmix64 finaliser of seed + (i+1)*0x9E3779B97F4A7C15; words (2p, 2p+1) give
 * u1 = ((x>>11)+1) 2^-53 and u2 = (x>>11) 2^-53; Box-Muller (sqrt(-2 ln u1) cos/sin(2 pi u2))
 * gives row-major entries 2p and 2p+1, each divided by sqrt(m) in double and rounded to fp32.
 * Any other Phi may be passed to the scoring calls instead; scores do not depend on its scale.
 */
int compactor_make_sketch(uint64_t seed, int32_t d, int32_t m, float* phi_host);

/*
 * Appendix D: a subsampled randomised Hadamard sketch, written out as a matrix Phi [d][m] (HOST,
 * row-major fp32) that the scoring calls take like any other sketch: Phi = (1/sqrt(m)) D H R^T with
 * D random signs, H the Sylvester-Walsh-Hadamard matrix of order d (d a power of two) and R a
 * choice of m columns without replacement.  Random bits come from the splitmix64 stream of
 * compactor_make_sketch: word i (i < d) gives the sign of row i (bit 0 set = minus); word d + j
 * drives step j of a Fisher-Yates shuffle of 0..d-1 (swap position j with j + word mod (d - j)),
 * whose first m entries are the chosen columns.
 */
int compactor_make_sketch_srht(uint64_t seed, int32_t d, int32_t m, float* phi_host);

/*
 * Number of retained tokens for a sequence of n tokens at retention ratio r (Section 3,
 * Preliminaries: k = ceil(r N)): ceil evaluated on the double product, clamped to [1, n];
 * 0 when n <= 0.  Returns the count (never an error code).
 */
int64_t compactor_keep_count(int64_t n, double r);

/*
 * Context-calibrated retention (Section 3.5): with b = alpha*nll + beta and the fitted curve
 * f(r) = (exp(rb-b) - exp(-b)) / (1 - exp(-b)), writes the r with f(r) = tau, i.e.
 * r* = log(1 + tau*(e^b - 1)) / b (r* = tau when b = 0).  tau must lie in (0, 1].
 */
int compactor_calibrated_ratio(double nll, double alpha, double beta, double tau, double* r_out);

/*
 * Fit of the calibration curve (Section 3.5): finds (alpha, beta) minimising the asymmetric mean
 * squared error sum_i w_i (f_{alpha,beta}(r_i, nll_i) - y_i)^2 / n over n training triples, where
 * f is the curve of compactor_calibrated_ratio with b = alpha*nll_i + beta, y_i is the measured
 * NLL ratio at retention r_i, and w_i = under_weight (>= 1) when the curve predicts more quality
 * than was measured (which would make r* too small), else 1; the paper weights those errors
 * higher without giving the weight.  Host arrays, host computation (Levenberg-Marquardt from a
 * grid of starting points); loss_out may be NULL.
 */
int compactor_fit_calibration(int64_t n, const double* r, const double* nll, const double* y,
                              double under_weight, double* alpha_out, double* beta_out, double* loss_out);

/*
 * Token-averaged negative log-likelihood (Section 3.5): for each of `batch` sequences, the mean
 * over its scored rows of -log softmax(logits_i)[targets_i].  This is the context statistic NLL(c)
 * that compactor_calibrated_ratio turns into a retention ratio.
 *   logits       device, [rows][vocab] with `row_stride` elements between rows; bf16
 *                (logits_dtype COMPACTOR_DTYPE_BF16) or fp32 (COMPACTOR_DTYPE_F32); 16-byte aligned,
 *                row_stride * element size a multiple of 16.
 *   targets      device int32 [rows]: the token each row is scored on; a negative id (or one
 *                >= vocab) leaves the row unscored: its row result is 0 and it does not count in
 *                the average.
 *   cu_rows      HOST int32 [batch+1], non-decreasing from 0 to rows: the rows of each sequence.
 *   row_nll_out  device fp32 [rows], required: the per-row terms (also the kernel's scratch).
 *   nll_out      device fp64 [batch]: the averages (0 for a sequence with no scored row).
 * Arithmetic: one streaming pass in fp32 (running maximum, base-2 exponentials), averages in fp64
 * in a fixed order.  No workspace.  Errors: COMPACTOR_E_INVALID_ARGUMENT for null pointers, bad
 * alignment, vocab < 1, an unknown dtype or an inconsistent cu_rows.
 */
#define COMPACTOR_DTYPE_BF16 0
#define COMPACTOR_DTYPE_F32  1
int compactor_nll(const void* logits, int32_t logits_dtype, int64_t rows, int32_t vocab, int64_t row_stride,
                  const int32_t* targets, int32_t batch, const int32_t* cu_rows,
                  float* row_nll_out, double* nll_out, void* stream);

/*
 * Bytes of device workspace that compactor_score and compactor_compress need for this shape.
 * compactor_select and compactor_compact only need a small table at its start and accept any
 * workspace of at least 16*(batch+1) bytes rounded up to 256 (compactor_select uses whatever
 * follows the table as scratch, see there).  The workspace must be 256-byte aligned; its
 * contents need not be preserved between calls.  Returns 0 for an invalid shape.
 */
size_t compactor_workspace_bytes(const compactor_shape* shape);

/*
 * Approximate leverage scores of every unit (Algorithm 1, lines 2-6) and the blend of Eq. 6.
 *   k_score      keys to score (the paper scores the keys before positional encoding).
 *   phi          device, fp32 [d][m] row-major: the sketch, shared by all units.
 *   attn_scores  device fp32 [layers][heads][total_tokens] or NULL.  If given, the output is
 *                s = z(attn) + lambda * z(o) per unit (population std; a term with zero std
 *                contributes 0); if NULL the output is the outlier score o itself.
 *   scores_out   device fp32 [layers][heads][total_tokens].
 * With m = d and any invertible phi (the identity, say) the result is the exact leverage score
 * of Definition 1 / Eq. 1, the paper's "exact" ablation; sketches wider than 64 columns run in a
 * slower configuration of the same kernels.
 * The small factorisation is a Cholesky factorisation of G = (K Phi)^T (K Phi) in fp64 - one of
 * the algebraically equal routes the paper allows (Section 3.2, Appendix C); Gram sums are fp32
 * within runs of 512 tokens and fp64 beyond.
 */
int compactor_score(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                    const float* attn_scores, float lambda, float* scores_out,
                    int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * compactor_score with the small factorisation chosen by the caller (Appendix C).
 *   factorization  COMPACTOR_FACTOR_CHOLESKY: exactly compactor_score.  Cholesky of G is the R
 *                  factor of the appendix's QR route (K Phi = Q R, score = squared row norm of Q).
 *                  COMPACTOR_FACTOR_EIG: the appendix's eigendecomposition route.  G = V Lambda V^T
 *                  (cyclic Jacobi, fp64), every eigenvalue raised to at least eig_floor,
 *                  score_i = || k_i Phi V Lambda^-1/2 ||^2.  Unlike the other routes the result
 *                  depends on the scale of Phi once the floor is active; the status bit
 *                  COMPACTOR_STATUS_RANK then reports that some eigenvalue was below the floor.
 *   eig_floor      the floor (the paper suggests about 1e-6); must be positive and finite;
 *                  ignored for COMPACTOR_FACTOR_CHOLESKY.
 * The eigendecomposition route takes m <= 64 (COMPACTOR_E_UNSUPPORTED beyond).
 * All other arguments, the workspace and the error behaviour are those of compactor_score.
 */
int compactor_score_variant(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                            int32_t factorization, double eig_floor,
                            const float* attn_scores, float lambda, float* scores_out,
                            int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Per-unit top-k (Section 3.4: the ceil(r N) highest-scoring tokens are kept, here per head).
 *   scores       device fp32 [layers][heads][total_tokens].
 *   keep_counts  host int32 [batch]: tokens kept per sequence (0 <= keep <= length), the same
 *                for every layer and head.
 *   idx_out      device int32 [layers][heads][total_keep]: for each unit the indices (local to
 *                the sequence, 0-based) of its keep_counts[b] largest scores, ascending.  Equal
 *                scores are ranked by lower index first.  NaN scores rank above +inf.
 * One CTA selects a unit.  Where that would leave most of the GPU idle (fewer units than SMs and
 * sequences of 10^5 tokens or more) and the workspace is the size compactor_workspace_bytes()
 * gives, every score vector is cut into slices that share a histogram and a candidate list in the
 * workspace; the indices are the same either way.
 */
int compactor_select(const compactor_shape* shape, const float* scores,
                     const int32_t* keep_counts, int32_t* idx_out,
                     int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Compaction: k_out[l][h][cu_keep[b]+j][:] = k_cache[l][h][cu_seqlens[b]+idx[l][h][cu_keep[b]+j]][:]
 * and likewise for v, as bit copies.  k_out / v_out are dense bf16 [layers][heads][total_keep][d].
 * Indices outside [0, length) are skipped (their output rows are left untouched).
 */
int compactor_compact(const compactor_shape* shape, compactor_mat k_cache, compactor_mat v_cache,
                      const int32_t* idx, const int32_t* keep_counts,
                      void* k_out, void* v_out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole pass: score k_score, select, and gather rows of k_cache / v_cache.
 * k_score may be the same tensor as k_cache.  scores_out may be NULL (scores then live only in
 * the workspace); idx_out, k_out, v_out as above.
 */
int compactor_compress(const compactor_shape* shape, compactor_mat k_score, compactor_mat k_cache,
                       compactor_mat v_cache, const float* phi, const float* attn_scores,
                       float lambda, const int32_t* keep_counts,
                       float* scores_out, int32_t* idx_out, void* k_out, void* v_out,
                       int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * compactor_compress with stage markers, for measurement (the paper reports one wall-clock
 * number per context length, Fig. 1; this splits ours by stage).  stage_events is a HOST array of
 * n_events cudaEvent_t handles created by the caller (NULL entries are skipped).  They are
 * recorded on the stream: [0] before the first kernel, [1] after the Gram pass, [2] after the
 * factorisation, [3] after the scoring pass, [4] after the blend (recorded even when there is
 * none), [5] after selection, [6] after compaction.  Results are identical to compactor_compress.
 */
#define COMPACTOR_N_STAGE_EVENTS 7
int compactor_compress_profiled(const compactor_shape* shape, compactor_mat k_score, compactor_mat k_cache,
                                compactor_mat v_cache, const float* phi, const float* attn_scores,
                                float lambda, const int32_t* keep_counts,
                                float* scores_out, int32_t* idx_out, void* k_out, void* v_out,
                                int32_t* status, void* workspace, size_t workspace_bytes, void* stream,
                                void* const* stage_events, int32_t n_events);

/*
 * Attention term of the score (Eq. 5): for every unit, a = concat_i 1^T softmax(scale * Q[i] K[i]^T)
 * over chunks i of `chunk` consecutive tokens of the sequence (no causal mask), summed over the
 * q_per_kv query heads that share the KV head, then mean-pooled.  The result is what
 * compactor_score / compactor_compress take as attn_scores.
 *   q        bf16 [layers][heads * q_per_kv][total_tokens][d]; query head j of KV head h is
 *            head index h * q_per_kv + j.  Same stride and alignment rules as the keys.
 *   chunk    must be 256 (the paper's setting).
 *   scale    > 0; the paper's equation prints no scale, attention layers use 1/sqrt(d).
 *   pool     odd window of the mean pooling (1 = none): centred, zero beyond the ends of the
 *            sequence, divided by `pool` (the paper pools but does not give the window).
 *   attn_out device fp32 [layers][heads][total_tokens].
 * The last, shorter chunk of a sequence is a softmax over its own keys.  Exponentials are
 * rounded to fp16 before they are summed over the query rows on the tensor cores (fp32
 * accumulation).  Workspace: compactor_workspace_bytes() suffices (16*(batch+1) bytes rounded up
 * to 256, plus 4 bytes per output element when pool > 1).
 */
int compactor_attention_scores(const compactor_shape* shape, compactor_mat q, compactor_mat k,
                               int32_t q_per_kv, int32_t chunk, float scale, int32_t pool,
                               float* attn_out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * compactor_attention_scores (Eq. 5) with the per-unit status word of the other device calls:
 * `status` (device int32 [layers*heads*batch], may be NULL) is cleared when the call starts and
 * receives COMPACTOR_STATUS_TIMEOUT for every unit of a CTA one of whose bounded device-side waits
 * ran out (the attention term of such a unit is unspecified).  Everything else as above.
 */
int compactor_attention_scores_status(const compactor_shape* shape, compactor_mat q, compactor_mat k,
                                      int32_t q_per_kv, int32_t chunk, float scale, int32_t pool,
                                      float* attn_out, int32_t* status, void* workspace, size_t workspace_bytes,
                                      void* stream);

/*
 * Selection across the heads of a layer (Section 3.4 allows the top scores to be taken over all
 * heads instead of within each head; the paper's experiments use such head-adaptive budgets).
 * For every (layer, sequence b) the heads * keep_counts[b] largest scores over all heads are kept,
 * ranked by (score descending, head ascending, index ascending), so heads keep different numbers
 * of tokens while the layer keeps as many as per-head selection would.
 *   idx_out           device int32 [layers][heads * total_keep]: layer l, sequence b owns entries
 *                     [heads * cu_keep[b], heads * cu_keep[b+1]); inside that block head h owns
 *                     [off[h], off[h+1]) with off = head_offsets_out[l][b][0 .. heads]; indices are
 *                     local to the sequence and ascending within a head.
 *   head_offsets_out  device int32 [layers][batch][heads + 1], off[0] = 0, off[heads] = heads * keep_counts[b].
 * heads must not exceed 64.  Workspace: compactor_across_heads_workspace_bytes() (the tables, and
 * per (layer, sequence) a histogram, a candidate list and per-slice counts: every head's scores are
 * cut into slices that are counted and emitted by CTAs of their own).
 * compactor_compact_across_heads gathers K/V rows in exactly that order into
 * k_out / v_out [layers][heads * total_keep][d] (bit copies; out-of-range indices are skipped).
 */
size_t compactor_across_heads_workspace_bytes(const compactor_shape* shape);
int compactor_select_across_heads(const compactor_shape* shape, const float* scores,
                                  const int32_t* keep_counts, int32_t* idx_out, int32_t* head_offsets_out,
                                  void* workspace, size_t workspace_bytes, void* stream);
int compactor_compact_across_heads(const compactor_shape* shape, compactor_mat k_cache, compactor_mat v_cache,
                                   const int32_t* idx, const int32_t* head_offsets,
                                   const int32_t* keep_counts, void* k_out, void* v_out,
                                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * The paper's whole method in one call: attention term (Eq. 5) -> leverage scores (Algorithm 1)
 * -> blend (Eq. 6) -> selection within each head or across the heads of a layer (Section 3.4) ->
 * gather.  The experiments of Section 4 use chunk 256, lambda 0.3, m 48 and selection across heads.
 *   options      HOST struct:
 *     selection      COMPACTOR_SELECT_PER_HEAD or COMPACTOR_SELECT_ACROSS_HEADS.
 *     factorization  COMPACTOR_FACTOR_CHOLESKY or COMPACTOR_FACTOR_EIG (with eig_floor), as in
 *                    compactor_score_variant.
 *     lambda         weight of the leverage term in Eq. 6 (ignored without an attention term).
 *     q_per_kv       query heads per KV head; 0 = no attention term: the score is the leverage
 *                    score alone and q is ignored.
 *     chunk, scale, pool   as in compactor_attention_scores (chunk must be 256).
 *   q            queries, bf16 [layers][heads * q_per_kv][total_tokens][d] (ignored if q_per_kv = 0).
 *   k_score      keys scored by Algorithm 1 (the paper: before positional encoding);
 *   k_cache      keys the attention term is taken against and the rows are gathered from (may be
 *                the same tensor as k_score);  v_cache likewise for the values.
 *   scores_out   device fp32 [layers][heads][total_tokens] or NULL: the final (blended) score.
 *   idx_out, k_out, v_out
 *                per-head selection: the layouts of compactor_select / compactor_compact;
 *                across heads: those of compactor_select_across_heads / compactor_compact_across_heads.
 *   head_offsets_out  device int32 [layers][batch][heads + 1]; across heads only (else may be NULL).
 *   status       device int32 [layers*heads*batch] or NULL; cleared once, then collects the flags of
 *                the attention and the scoring kernels.
 * Workspace: compactor_compress_full_workspace_bytes(shape, options), 256-byte aligned.  Errors as for
 * the calls it is made of; everything is checked before anything is enqueued.
 */
#define COMPACTOR_SELECT_PER_HEAD      0
#define COMPACTOR_SELECT_ACROSS_HEADS  1
typedef struct compactor_options {
    int32_t selection;
    int32_t factorization;
    double  eig_floor;
    float   lambda;
    int32_t q_per_kv;
    int32_t chunk;
    float   scale;
    int32_t pool;
} compactor_options;
size_t compactor_compress_full_workspace_bytes(const compactor_shape* shape, const compactor_options* options);
int compactor_compress_full(const compactor_shape* shape, const compactor_options* options, compactor_mat q,
                            compactor_mat k_score, compactor_mat k_cache, compactor_mat v_cache,
                            const float* phi, const int32_t* keep_counts, float* scores_out,
                            int32_t* idx_out, int32_t* head_offsets_out, void* k_out, void* v_out,
                            int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * compactor_score for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience).  Same inputs, outputs and results as compactor_score, but
 * no workspace argument: the scratch is a fixed array of compactor_builtin_scratch_bytes()
 * (32 MiB) inside the library, resident on every device the process uses from the first use of
 * the library on that device until the process exits.  The call allocates and frees nothing.
 *   - Size limit: the scratch must hold 16*(batch+1) bytes of tables, about 72 KiB per unit
 *     (at m = 48) and 128 KiB per Gram block (blocks are lengthened up to 65536 tokens to make it
 *     fit, i.e. down to 2 bytes per token per (layer, head)).  A larger problem is refused with
 *     COMPACTOR_E_TOO_LARGE before anything is enqueued; split it by layers or use
 *     compactor_score.
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls share the one array and it keeps whatever the previous call left there (nothing
 *     in it needs clearing: every call rewrites what it reads).  Two calls whose device work
 *     can overlap - different streams, or different host threads on the same device - race on
 *     it; order them on one stream or with events.
 */
size_t compactor_builtin_scratch_bytes(void);
int compactor_score_builtin_scratch(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                                    const float* attn_scores, float lambda, float* scores_out,
                                    int32_t* status, void* stream);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper).  Enqueues a one-warp
 * kernel that waits, with a limit of about a millisecond, once on a barrier that completes and
 * once on a barrier that nothing completes, through the same wait routine the streaming kernels
 * use.  status_out (device int32[1]) receives COMPACTOR_STATUS_TIMEOUT (4) when the first wait
 * succeeded and the second gave up as designed; any other value is a defect.  The context stays
 * usable: nothing traps or hangs.
 */
int compactor_wait_selftest(int32_t* status_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* COMPACTOR_H_ */
