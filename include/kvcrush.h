/*
 * kvcrush.h - C ABI of the B200 (sm_100a) KVCrush KV-cache compression pass.
 *
 * One pass over the prompt of every (layer, sequence) runs four stages:
 *
 *   kvcrush_score      per-token, per-head attention importance: column sums of
 *                      the softmax attention matrix          (Algorithm 1, Sec. 3.1)
 *   kvcrush_signature  per-head thresholds and the packed binary head-behaviour
 *                      signature of every token              (Algorithm 1, Sec. 3.1)
 *   kvcrush_select     B_important tokens by cumulative attention (H2O) plus one
 *                      representative per Hamming bucket of the remaining tokens
 *                                                            (Algorithm 2, Sec. 3, Sec. 3.2)
 *   kvcrush_compact    gather of the kept K/V rows into the reduced cache (Sec. 3.2)
 *
 * Conventions for every entry point unless stated otherwise
 *   - Pointers named *_dev (and every tensor / output pointer) are DEVICE pointers
 *     owned by the caller; pointers named *_host are host pointers read during the
 *     call only.  The library allocates and frees no memory and keeps no state
 *     between calls apart from two process-wide, write-once caches (the driver's
 *     tensor-map encoder entry point; for kvcrush_signature_static the device address
 *     of its array); scratch memory is the caller's `workspace` (device, 256-byte
 *     aligned, size from kvcrush_workspace_size).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and the call returns without synchronising.  Inputs are never written.
 *   - Return value: KVCRUSH_OK, or a negative KVCRUSH_ERR_* code, in which case
 *     nothing was enqueued.  Problems found on the device (a bounded wait that ran
 *     out) are reported through `status_dev` (int32[4], zeroed by the caller before
 *     the first call): status[0] = 0 when fine, else a KVCRUSH_DEV_* code,
 *     status[1] = kernel id, status[2..3] = detail.  A kernel that reports an
 *     error leaves its outputs unspecified.
 *   - Token-major tensors: element (layer l, token t, head h, channel d) lives at
 *     ptr + l*stride_layer + t*stride_token + h*stride_head + d (strides in
 *     elements, channel stride 1).  Tokens of all sequences are packed along the
 *     token axis: sequence s owns tokens [cu_seqlens[s], cu_seqlens[s+1]).
 *   - Per-head score arrays are [n_layers][n_q_heads][total_tokens] float32;
 *     signatures are [n_layers][total_tokens][W] uint32, W = ceil(n_q_heads/32),
 *     head h in bit (h mod 32) of word (h div 32), unused bits zero.
 */
#ifndef KVCRUSH_H_
#define KVCRUSH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* return codes */
#define KVCRUSH_OK                 0
#define KVCRUSH_ERR_INVALID_ARG   (-1)   /* NULL pointer, negative size, inconsistent shapes */
#define KVCRUSH_ERR_UNSUPPORTED   (-2)   /* shape or type outside what the kernels handle   */
#define KVCRUSH_ERR_MISALIGNED    (-3)   /* pointer or stride breaks an alignment rule       */
#define KVCRUSH_ERR_WORKSPACE     (-4)   /* workspace NULL or too small                      */
#define KVCRUSH_ERR_CUDA          (-5)   /* a CUDA runtime / driver call failed              */
#define KVCRUSH_ERR_STATIC_LIMIT  (-6)   /* problem larger than a built-in scratch array     */

/* status_dev[0] values */
#define KVCRUSH_DEV_OK             0
#define KVCRUSH_DEV_TIMEOUT        1     /* a bounded wait on a barrier ran out */
#define KVCRUSH_DEV_BUDGET         2     /* kvcrush_kmeans_select: a budget_rep above max_budget_rep (status[2] = segment) */

/* element types */
#define KVCRUSH_BF16  0
#define KVCRUSH_FP16  1
#define KVCRUSH_FP32  2

/* stages, for kvcrush_workspace_size */
#define KVCRUSH_STAGE_SCORE      0
#define KVCRUSH_STAGE_SIGNATURE  1
#define KVCRUSH_STAGE_SELECT     2
#define KVCRUSH_STAGE_COMPACT    3

/* anchor strategies of Algorithm 2 */
#define KVCRUSH_ANCHOR_ALTERNATE 0   /* bit h = h mod 2 (head 0 -> 0)                         */
#define KVCRUSH_ANCHOR_MEAN      1   /* per-bit majority of the grouped tokens, ties -> 1     */
#define KVCRUSH_ANCHOR_EXPLICIT  2   /* caller's bits (a seeded random anchor is drawn on the host) */

/* score kernels */
#define KVCRUSH_SCORE_AUTO       0   /* tensor-core kernels when type, shape and strides allow, else SIMT;
                                        never a silent drop to SIMT because the driver lacks something  */
#define KVCRUSH_SCORE_SIMT       1   /* fp32 CUDA-core kernels (any supported shape and type) */
#define KVCRUSH_SCORE_TENSOR     2   /* tcgen05 kernels, error if the shape is not supported  */

/* Shape of one compression problem; shared by all four stages. */
typedef struct kvcrush_problem {
  int32_t n_layers;               /* >= 1 */
  int32_t n_seqs;                 /* sequences in the packed batch, >= 1 */
  int32_t n_q_heads;              /* 1..128 */
  int32_t n_kv_heads;             /* divides n_q_heads; query head h reads KV head h / (n_q_heads/n_kv_heads) */
  int32_t head_dim;               /* D */
  int32_t total_tokens;           /* T = cu_seqlens[n_seqs] */
  int32_t max_seqlen;             /* longest sequence */
  int32_t causal;                 /* 1: query j attends keys t <= j of its own sequence; 0: all keys of the sequence */
  float   softmax_scale;          /* 0 => 1/sqrt(head_dim) (Algorithm 1) */
  int32_t query_window;           /* 0: every query votes; w > 0: only the last w queries of each sequence
                                     (observation window, Sec. 2.3) - kvcrush_score only */
  const int32_t* cu_seqlens_host; /* [n_seqs+1] ascending from 0; HOST copy (grid sizing) */
  const int32_t* cu_seqlens_dev;  /* the same array in device memory */
} kvcrush_problem_t;

/* A token-major tensor [n_layers][total_tokens][heads][head_dim]. */
typedef struct kvcrush_tensor {
  const void* ptr_dev;            /* 16-byte aligned */
  int32_t dtype;                  /* KVCRUSH_BF16 | KVCRUSH_FP16 | KVCRUSH_FP32 */
  int32_t reserved;               /* set to 0 */
  int64_t stride_layer;           /* in elements; every stride * element size must be a multiple of 16 bytes */
  int64_t stride_token;
  int64_t stride_head;
} kvcrush_tensor_t;

/* Bytes of device workspace `stage` needs for this problem (0 is a valid answer). */
int kvcrush_workspace_size(const kvcrush_problem_t* problem, int stage, size_t* bytes);

/*
 * Stage 1 - attention-importance scores (Algorithm 1, first two steps).
 *   A_h = softmax(Q_h K_h^T * softmax_scale) per sequence (causal if problem->causal),
 *   scores[l][h][t] = sum over the queries j of t's sequence of A_h(j, t)
 * i.e. the attention key t receives.  (Algorithm 1 prints the sum with A_h's indices
 * in the other order, which is identically 1; the column sum is what is computed.)
 * With normalize != 0 the result is divided by the number of voting queries (the paper's 1/S).
 * With problem->query_window = w > 0 only the last w queries of each sequence are summed (the
 * observation window of SnapKV, Sec. 2.3): work drops from O(S^2) to O(S*w); the row log-sum-exp
 * is then computed (and lse_out_dev written) for those queries only.
 * The S x S matrix is never stored: a first sweep computes the log-sum-exp of every
 * query row, a second sweep recomputes the logits and accumulates exp(s - lse).
 *   Q, K        token-major tensors with n_q_heads / n_kv_heads heads, same dtype
 *               (BF16, FP16 or FP32).  Tensor-core kernels: BF16 or FP16, head_dim a
 *               multiple of 8 up to 128 (full speed at 64 and 128).
 *   lse_in_dev  optional [n_layers][n_q_heads][T] float32 natural-log row
 *               log-sum-exp of the scaled logits (as a prefill attention kernel
 *               returns it); when given the first sweep is skipped.
 *   scores_dev  out [n_layers][n_q_heads][T] float32
 *   lse_out_dev optional out, same shape: the row log-sum-exp (natural log);
 *               not written when lse_in_dev is given
 *   impl        KVCRUSH_SCORE_AUTO takes the tensor-core kernels when Q and K are BF16 or FP16, head_dim is a
 *               multiple of 8 up to 128 and the strides can be described to the TMA unit (a stride of 0 along an
 *               axis longer than 1, or beyond the tensor map's limits, cannot), otherwise the CUDA-core kernels.
 *               When the problem qualifies but the driver does not provide the tensor-map encoder, AUTO returns
 *               KVCRUSH_ERR_UNSUPPORTED rather than running the (about 100 times slower) CUDA-core kernels
 *               unnoticed; ask for KVCRUSH_SCORE_SIMT explicitly in that case.  KVCRUSH_SCORE_TENSOR returns
 *               KVCRUSH_ERR_UNSUPPORTED for anything the tensor-core kernels cannot take.
 *   workspace   kvcrush_workspace_size(.., KVCRUSH_STAGE_SCORE, ..) bytes; with lse_in_dev given only the first
 *               256 bytes are used (the kernels' work counters) and a 256-byte workspace is enough
 */
int kvcrush_score(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q, const kvcrush_tensor_t* K,
                  const float* lse_in_dev, float* scores_dev, float* lse_out_dev, int normalize, int impl,
                  void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Decode step of stage 1 (Sec. 2.3 / 4.1.1: H2O goes on summing attention weights while tokens are generated, and
 * the paper's paged experiments evict during decoding).  Every sequence has exactly one new query - the query of its
 * last token - and
 *     scores[l][h][t] += softmax over the sequence's tokens of (q_new[l][seq(t)][h] . k[l][t][h div G] * scale)
 * for every token t of the sequence, the new token included.  Feed the running scores to kvcrush_signature /
 * kvcrush_select(_pages) whenever the cache has outgrown its budget.
 *   problem     describes the cached tokens as they are now (cu_seqlens include each sequence's new token);
 *               causal and query_window are ignored
 *   Q_new       [n_layers][n_seqs][n_q_heads][head_dim]: stride_token steps from one sequence to the next
 *   K           the cached keys, token-major, same dtype as Q_new (BF16, FP16 or FP32), head_dim <= 256, multiple of 8
 *   scores_dev  in/out [n_layers][n_q_heads][T] float32 running column sums
 * Runs on the CUDA cores (one block per layer, sequence and KV head, which serves the query heads of its group);
 * bound by reading K twice.
 */
int kvcrush_score_decode(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q_new, const kvcrush_tensor_t* K,
                         float* scores_dev, int32_t* status_dev, void* stream);

/*
 * Stage 2 - per-head thresholds and packed signatures (Algorithm 1, Sec. 3.1).
 *   theta[l][s][h] = the keep-th largest value of scores[l][h][tokens of s]
 *                    (keep >= length: -inf, all ones; keep <= 0: +inf, all zeros)
 *   bit h of sigs[l][t] = scores[l][h][t] >= theta[l][seq(t)][h]
 *   sig_keep_dev   [n_layers][n_seqs] int32 rank per (layer, sequence); ignored when
 *                  theta_in_dev is given
 *   theta_in_dev   optional [n_layers][n_seqs][n_q_heads] float32 explicit thresholds
 *                  (the input form of Algorithm 1)
 *   sigs_dev       out [n_layers][T][W] uint32
 *   theta_out_dev  optional out [n_layers][n_seqs][n_q_heads] float32
 *   importance_out_dev  optional out [n_layers][T] float64: the token importance I(t) that stage 3 ranks (the
 *                  sum of the token's per-head scores in the order kvcrush_select states), written from the
 *                  loads this stage does anyway; hand it to kvcrush_select / kvcrush_select_pages as
 *                  importance_dev and they skip their own pass over the scores
 *   workspace      holds the thresholds when theta_out_dev is NULL
 */
int kvcrush_signature(const kvcrush_problem_t* problem, const float* scores_dev, const int32_t* sig_keep_dev,
                      const float* theta_in_dev, uint32_t* sigs_dev, float* theta_out_dev, double* importance_out_dev,
                      void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Stage 3 - the kept set of every (layer, sequence) (Sec. 3, Algorithm 2, Sec. 3.2).
 *   I(t)  = sum of the per-head scores of t: float64, heads added in ascending order
 *           inside each KV group, then the group sums in ascending order
 *   Imp   = the budget_imp tokens of largest I (ties: lower token index)       [H2O]
 *   C     = the other tokens, N = |C|; anchor a; d_t = popcount(sig_t xor a)
 *   sort C by (d_t, t); bucket i = sorted positions [floor(i*N/R), floor((i+1)*N/R)),
 *           R = budget_rep
 *   rep_i = member of bucket i closest to the bucket's per-bit mean (L1; ties: lower t)
 *   kept  = Imp U {rep_i}, ascending token index.  budget_imp + budget_rep >= length
 *           keeps every token.
 *   scores_dev         [n_layers][n_q_heads][T] float32; may be NULL when importance_dev is given
 *   importance_dev     optional [n_layers][T] float64: I(t) as kvcrush_signature writes it (importance_out_dev);
 *                      NULL: computed here from scores_dev
 *   budget_imp_dev, budget_rep_dev  [n_layers][n_seqs] int32, >= 0
 *   anchor_mode        KVCRUSH_ANCHOR_*
 *   anchor_bits_dev    [W] uint32 (anchor_per_segment == 0) or [n_layers][n_seqs][W];
 *                      read only for KVCRUSH_ANCHOR_EXPLICIT; bits above n_q_heads ignored
 *   keep_initial,      >= 0: the first keep_initial and the last keep_recent tokens of every sequence count
 *   keep_recent        as infinitely important (Table 1 of the paper reserves initial and recent parts of the
 *                      budget; SnapKV keeps its observation window); they take places of budget_imp,
 *                      lowest index first if there are more of them
 *   cu_kept_dev        [n_layers*n_seqs + 1] int32: where each segment's kept list starts
 *                      in idx_dev, segment = layer*n_seqs + seq; the caller sets it to the
 *                      prefix sums of min(budget_imp + budget_rep, length)
 *   idx_dev            out [cu_kept[last]] int32 token index inside its sequence
 *   kind_dev           optional out, same length, uint8: 0 important, 1 representative
 *   n_kept_dev         optional out [n_layers][n_seqs] int32: tokens kept of every segment,
 *                      min(budget_imp + budget_rep, length) - what cu_kept's differences must be
 * Sequences longer than 262144 tokens are not supported.
 */
int kvcrush_select(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                   const uint32_t* sigs_dev, const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                   int anchor_mode, const uint32_t* anchor_bits_dev, int anchor_per_segment,
                   int keep_initial, int keep_recent,
                   const int32_t* cu_kept_dev, int32_t* idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                   void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Max pooling of per-head scores along the token axis (Sec. 2.3 / 4.1.1: SnapKV keeps the
 * neighbours of high-scoring tokens by max pooling): out[l][h][t] = max of in[l][h][t-r .. t+r]
 * clipped to t's sequence, r = (kernel - 1) / 2.  kernel must be odd and >= 1; in and out must not
 * alias.  Feed the result to kvcrush_signature / kvcrush_select in place of the raw scores.
 */
int kvcrush_pool_scores(const kvcrush_problem_t* problem, const float* scores_in_dev, int kernel,
                        float* scores_out_dev, int32_t* status_dev, void* stream);

/*
 * Stage 4 - reduced cache (Sec. 3.2: the kept tokens form the final cache).
 *   out[l][cu_kept[l*n_seqs+s] - cu_kept[l*n_seqs] + i][h][:] =
 *        in[l][cu_seqlens[s] + idx[cu_kept[l*n_seqs+s] + i]][h][:]        for K and for V
 *   K, V           token-major caches with n_kv_heads heads (any element type; bytes are copied)
 *   total_kept     cu_kept[n_layers*n_seqs] (host value, for grid sizing)
 *   K_out, V_out   token-major outputs; ptr_dev is written; same dtype as the inputs;
 *                  head_dim * element size must be a multiple of 16 bytes
 * V (and V_out) may be NULL to gather one tensor only.
 */
int kvcrush_compact(const kvcrush_problem_t* problem, const kvcrush_tensor_t* K, const kvcrush_tensor_t* V,
                    const int32_t* cu_kept_dev, const int32_t* idx_dev, int64_t total_kept,
                    const kvcrush_tensor_t* K_out, const kvcrush_tensor_t* V_out,
                    int32_t* status_dev, void* stream);

/*
 * Stage 3 at page (or chunk) granularity (Sec. 4.3.4: chunks of 8 tokens; Sec. 4.3.5: pages of 32 tokens, where
 * the baseline sums the attention weights over a page and the binary vector of a page is the concatenation of the
 * head vectors of its tokens).  A page is page_size consecutive tokens of one sequence, page p = tokens
 * [p*page_size, (p+1)*page_size); the last page may be short: its missing tokens count as all-zero vectors of zero
 * importance.  Budgets, cu_kept and the output count PAGES.
 *   J(p)  = sum of I(t) over the tokens of p (I as in kvcrush_select), float64, tokens in ascending order
 *   Imp   = the budget_imp pages of largest J (ties: lower page)
 *   v_p   = sigs of the page's tokens one after the other (page_size * W words); anchor: the token anchor in
 *           every slot (ALTERNATE, EXPLICIT) or the per-bit majority of the grouped pages (MEAN, ties to 1)
 *   then exactly the steps of kvcrush_select on the other pages: d_p = popcount(v_p xor anchor), (d_p, p) order,
 *   budget_rep equal-frequency buckets, per bucket the page closest to the per-bit mean (L1; ties: lower page),
 *   kept = Imp U representatives, ascending.  budget_imp + budget_rep >= number of pages keeps every page.
 *   scores_dev,        as for kvcrush_select: the token importance comes from importance_dev when given, else from
 *   importance_dev     the scores
 *   page_size          >= 1; page_size * W <= 128 words and at most 8192 pages per sequence, otherwise
 *                      KVCRUSH_ERR_UNSUPPORTED.  page_size 1 gives the result of kvcrush_select.
 *   anchor_bits_dev    [W] or [n_layers][n_seqs][W] token anchor (EXPLICIT only)
 *   keep_initial,      >= 0, in pages: the first / last pages of every sequence are important by decree (Table 1:
 *   keep_recent        a 672-token budget = 32 initial + 512 middle + 128 recent tokens at page size 32)
 *   cu_kept_dev        [n_layers*n_seqs + 1] prefix sums of min(budget_imp + budget_rep, pages of the sequence)
 *   page_idx_dev       out [cu_kept[last]] int32 page number inside its sequence
 *   kind_dev           optional out: 0 important, 1 representative
 *   n_kept_dev         optional out [n_layers][n_seqs] int32: pages kept of every segment
 *   workspace          kvcrush_workspace_size(.., KVCRUSH_STAGE_SELECT, ..) bytes
 */
int kvcrush_select_pages(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                         const uint32_t* sigs_dev, int page_size,
                         const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                         int anchor_mode, const uint32_t* anchor_bits_dev, int anchor_per_segment,
                         int keep_initial, int keep_recent,
                         const int32_t* cu_kept_dev, int32_t* page_idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                         void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Stage 4 at page granularity (Sec. 4.3.5): the kept pages form the reduced paged cache.
 *   out[l][(cu_kept[l*n_seqs+s] - cu_kept[l*n_seqs] + i) * page_size + j][h][:] =
 *        in[l][cu_seqlens[s] + page_idx[cu_kept[l*n_seqs+s] + i] * page_size + j][h][:]     j < page_size
 *   and zeros for the slots j of a short last page that lie past the end of the sequence.
 *   total_kept_pages   cu_kept[n_layers*n_seqs] (host value)
 * Other arguments as for kvcrush_compact; the outputs hold total kept pages * page_size token rows per layer.
 */
int kvcrush_compact_pages(const kvcrush_problem_t* problem, const kvcrush_tensor_t* K, const kvcrush_tensor_t* V,
                          int page_size, const int32_t* cu_kept_dev, const int32_t* page_idx_dev,
                          int64_t total_kept_pages, const kvcrush_tensor_t* K_out, const kvcrush_tensor_t* V_out,
                          int32_t* status_dev, void* stream);

/*
 * The running scores of a decode-time loop follow the cache through an eviction (Sec. 2.3 / 4.1.1: the cumulative
 * attention of the kept tokens goes on accumulating):
 *   out[l][h][(cu_kept[l*n_seqs+s] - cu_kept[l*n_seqs] + i) * P + j] = in[l][h][cu_seqlens[s] + idx[cu_kept[..] + i] * P + j]
 * with P = 1 and j = 0 for kept tokens (page_size 0), P = page_size and j < P for kept pages; slots of a short last
 * page that lie past the end of the sequence get 0.  The arrangement along the token axis is that of
 * kvcrush_compact / kvcrush_compact_pages.
 *   scores_in_dev   [n_layers][n_q_heads][T] float32
 *   scores_out_dev  out [n_layers][n_q_heads][out_tokens] float32; must not alias the input
 *   out_tokens      token stride of the output (>= the kept rows of any layer)
 */
int kvcrush_compact_scores(const kvcrush_problem_t* problem, const float* scores_in_dev, int page_size,
                           const int32_t* cu_kept_dev, const int32_t* idx_dev, int64_t total_kept,
                           float* scores_out_dev, int64_t out_tokens, int32_t* status_dev, void* stream);

/*
 * Clustering baseline of the ablation "KMeans vs KVCrush" (Experiments, Ablation Study, Fig. 3: k-means with 100
 * iterations in the place of Algorithm 2's grouping, about 200 % more inference latency than H2O against less than
 * 0.5 % for KVCrush).  Not a stage of the pass: it is here so that a conventional clustering of the same binary head
 * vectors can be timed beside kvcrush_select.  Same arguments, outputs and important set as kvcrush_select; the
 * other tokens (ascending, N of them) are grouped by Lloyd's algorithm instead of by Hamming distance to an anchor:
 *   k = budget_rep clusters; initial centroids = the vectors at ranks floor(i*N/k) of the grouped tokens;
 *   an iteration assigns every vector to the centroid at the smallest squared Euclidean distance (compared exactly,
 *   as integer fractions; ties: lower cluster) and replaces every centroid by the per-bit mean of its members (a
 *   cluster without members keeps its centroid); after `iterations` iterations one more assignment fixes the members;
 *   every cluster with members gives the member closest to its centroid (ties: lower token), kind 1;
 *   budget that empty clusters leave unused goes to the most important of the remaining tokens, kind 0.
 * The paper gives the method's name and iteration count only; initialisation, tie rules and the treatment of empty
 * clusters are this library's.
 *   max_budget_rep   host value: no budget_rep of the call exceeds it (sizes the workspace); a larger budget is
 *                    reported as KVCRUSH_DEV_BUDGET through status_dev and that segment is left unwritten
 *   iterations       >= 0 (the paper's figure uses 100)
 *   workspace        kvcrush_kmeans_workspace_size(problem, max_budget_rep) bytes
 * Sequences longer than 32768 tokens, or with n_q_heads * max_seqlen^4 >= 2^66 (the exact comparison works in 64-bit
 * integers), return KVCRUSH_ERR_UNSUPPORTED.
 */
int kvcrush_kmeans_workspace_size(const kvcrush_problem_t* problem, int max_budget_rep, size_t* bytes);
int kvcrush_kmeans_select(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                          const uint32_t* sigs_dev, const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                          int max_budget_rep, int iterations, int keep_initial, int keep_recent,
                          const int32_t* cu_kept_dev, int32_t* idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                          void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream);

/*
 * Stage 2 without caller-provided scratch (the paper has no counterpart; this is a packaging
 * variant of kvcrush_signature for hosts that cannot hand over device memory).
 *
 * Who needs it: code that runs where device allocation is off the table - a plug-in inside a
 * serving engine that owns the whole memory pool and forbids cudaMalloc in its hot path, a
 * callback that must not trigger the implicit device synchronisation an allocation causes, or an
 * embedding that simply has no allocator to offer for the thresholds' scratch.
 *
 * Same computation and outputs as kvcrush_signature with sig_keep_dev (no explicit thresholds,
 * no theta output): the per-head thresholds live in a scratch array that is part of the library
 * image (file-scope __device__ memory, KVCRUSH_STATIC_THETA_MAX floats = 256 KiB, resident on every
 * GPU that loads the library until the process exits).  The call allocates nothing and frees nothing.
 *   - n_layers * n_seqs * n_q_heads must not exceed KVCRUSH_STATIC_THETA_MAX, otherwise
 *     KVCRUSH_ERR_STATIC_LIMIT is returned and nothing runs.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current); make that first call outside any stream
 *     capture.  Later calls reuse the address.
 *   - All calls share the one array per device and it keeps whatever the previous call left.  Nothing
 *     in it has to start at zero: every threshold a call reads is written earlier in that same call.
 *     Two calls that overlap on the GPU (different streams, no ordering) race on it; serialise them.
 */
#define KVCRUSH_STATIC_THETA_MAX 65536
int kvcrush_signature_static(const kvcrush_problem_t* problem, const float* scores_dev,
                             const int32_t* sig_keep_dev, uint32_t* sigs_dev,
                             int32_t* status_dev, void* stream);

/* Text for a return code. */
const char* kvcrush_strerror(int code);

/* Library version, major*10000 + minor*100 + patch. */
int kvcrush_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KVCRUSH_H_ */
