/*
 * vitcop.h -- C ABI of the B200 (sm_100a) visual-token pruning operator chain of ViTCoP
 * (arXiv 2601.17818, "Visual and Textual Semantic Collaborative Pruning").
 *
 * Conventions that hold for every entry point
 *   - Plain C linkage, plain pointers and sizes.  Unless a parameter says "host", every tensor
 *     pointer is a DEVICE pointer owned by the caller.  The library never allocates or frees
 *     caller-visible memory and keeps no state between calls; scratch memory comes from a
 *     caller-provided `workspace` whose size `vitcop_workspace_bytes` reports.
 *   - Tensors are dense, row-major, last dimension contiguous.  bf16 tensors are passed as
 *     `const void*` (2-byte elements).  Base pointers of bf16 tensors must be 16-byte aligned and
 *     their row lengths (d, Dh, D) multiples of 8 elements; otherwise VITCOP_ERR_UNSUPPORTED.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *     enqueue work on that stream and return without synchronising; outputs are valid once the
 *     stream has reached the end of the call's work.
 *   - The visual tokens of a sequence occupy the contiguous span [vis_start, vis_start + vis_len);
 *     everything outside the span is text and is never scored, selected or dropped.
 *     `vis_len` may be given per sample as a device array (`vis_len`, int32 [B]) or, when that
 *     pointer is NULL, as one host integer (`vis_len_uniform`) for all samples.
 *   - Return value: a VITCOP_* status.  Conditions that only the device can see (see
 *     VITCOP_ERR_BUDGET, VITCOP_ERR_TIMEOUT) are recorded in a status word at the start of the
 *     call's workspace and read back with `vitcop_poll_status`.  Nothing traps or aborts.
 */
#ifndef VITCOP_H_
#define VITCOP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---------------------------------------------------------------- status codes */
#define VITCOP_OK               0
#define VITCOP_ERR_INVALID_ARG  1   /* NULL required pointer, negative size, span outside the sequence, aliasing */
#define VITCOP_ERR_UNSUPPORTED  2   /* alignment / divisibility / size limit not met */
#define VITCOP_ERR_WORKSPACE    3   /* workspace NULL or smaller than vitcop_workspace_bytes reports */
#define VITCOP_ERR_BUDGET       4   /* quota mode with budget < number of clusters (device-side, via poll) */
#define VITCOP_ERR_CUDA         5   /* a CUDA runtime call failed; see vitcop_last_cuda_error */
#define VITCOP_ERR_TIMEOUT      6   /* a bounded device-side wait expired (device-side, via poll) */

/* Largest visual span one sequence may have in vitcop_select / vitcop_prune_step / the filter. */
#define VITCOP_MAX_VISUAL_TOKENS 16384

/* ---------------------------------------------------------------- operations (for workspace sizing) */
#define VITCOP_OP_FILTER      0
#define VITCOP_OP_KNORM       1
#define VITCOP_OP_SELECT      2
#define VITCOP_OP_COMPACT     3
#define VITCOP_OP_PRUNE_STEP  4
#define VITCOP_OP_SIMILARITY  5
#define VITCOP_OP_SALIENCY    6   /* vitcop_cls_saliency: B = images, H = heads, N = keys per head (M) */
#define VITCOP_OP_MERGE       7   /* vitcop_merge_clusters: Nv = Nv_cap, N = Mcap */
#define VITCOP_OP_COLLAB_STEP 8   /* vitcop_collaborative_step */
#define VITCOP_OP_KPROJ       9   /* vitcop_kproj_knorm: B, H, N, d */

/* Human-readable name of a status code (static storage, never NULL). */
const char* vitcop_status_string(int status);

/* cudaError_t value of the most recent failing CUDA runtime call made by this library on the
 * calling thread (0 if none).  Meaningful after a call returned VITCOP_ERR_CUDA. */
int vitcop_last_cuda_error(void);

/* Bytes of device workspace `op` needs for the given problem (arguments an op does not use are
 * ignored; pass 0).  Nv is the capacity of the visual span (max over samples), n == Nv for the
 * filter.  `bytes` is a host pointer.  The workspace must be 256-byte aligned. */
int vitcop_workspace_bytes(int op, int B, int H, int N, int d, int Nv, int D, int Dh, size_t* bytes);

/* Synchronises `stream`, copies the device status word of `workspace` to `*device_status`
 * (host pointer; VITCOP_OK, VITCOP_ERR_BUDGET or VITCOP_ERR_TIMEOUT) and returns VITCOP_OK, or
 * VITCOP_ERR_CUDA if the synchronisation or the copy failed.  Every entry point that takes a
 * workspace resets the word when it starts, so poll after the call of interest. */
int vitcop_poll_status(const void* workspace, void* stream, int* device_status);

/* ---------------------------------------------------------------- diagnostic: bounded device waits
 * The paper has no counterpart.  Kernels whose CTAs wait for one another or for asynchronous copies (the Gram
 * sweeps of the redundancy filter) bound every wait; when a wait runs out, the CTA abandons its work, lets its
 * copies and tensor-core operations in flight finish, frees its tensor memory and records VITCOP_ERR_TIMEOUT in
 * the status word (read it with vitcop_poll_status; the call's outputs are then undefined, the workspace and the
 * library remain usable).  This call sets the limit for launches made after it, process-wide:
 *   limit_ns      time after which a wait gives up; 0 restores the default of 2 s
 *   expire_roles  for failure-handling tests: waits of the named roles give up at once, whatever their state
 *                 (1 load warp, 2 tensor-core issue warp, 4 epilogue warps; 0 = none)
 * Always returns VITCOP_OK. */
int vitcop_set_wait_limit(unsigned long long limit_ns, int expire_roles);

/* ---------------------------------------------------------------- diagnostic: per-kernel device times
 * The paper has no counterpart; this exists so that a benchmark can attribute the time of a multi-kernel
 * call to its kernels.  Between vitcop_kernel_timing_begin and vitcop_kernel_timing_end every kernel the
 * library launches (process-wide) is bracketed by two CUDA events on its stream, and kernels of one call
 * no longer overlap (programmatic dependent launch is switched off), so a call runs slower than normal.
 * vitcop_kernel_timing_end waits for the recorded events, sums launches and milliseconds per kernel name
 * into out[0 .. *count) (host memory, at most `capacity` distinct names) and switches timing off.
 * Not for use during stream capture.  Errors: INVALID_ARG, CUDA. */
typedef struct {
    char  name[48];     /* kernel name, NUL-terminated */
    int   launches;
    float total_ms;
} vitcop_kernel_time;

int vitcop_kernel_timing_begin(void);
int vitcop_kernel_timing_end(vitcop_kernel_time* out, int capacity, int* count);

/* ---------------------------------------------------------------- redundancy filter (VIC)
 * Visual Information Clustering, Algorithm 2 of the paper (Section "Visual Semantic Guidance",
 * Eq. 2 and Eq. 3): pairwise feature distance d_ij, local density
 * rho_i = sum_{j != i} exp(-(d_ij/d_c)^2), delta_i = min d_ij over denser tokens j within spatial
 * distance tau, gamma = rho * delta, the n_centers largest gamma become cluster centres and every
 * other token inherits the label of its nearest denser neighbour.  Near-duplicate tokens fall into
 * one cluster; vitcop_select in quota mode then keeps only each cluster's quota of them.
 *
 * Readings where the paper is silent: "denser" is the total order (rho desc, index asc); a token
 * without admissible denser neighbour is an orphan (delta = +inf, parent = -1), ranks first among
 * centre candidates and, if not chosen, joins the nearest centre by feature distance; a label is
 * the token index of the cluster's centre.
 *
 *   metric 0 (cosine): d_ij^2 = 2 - 2 s_ij, s_ij the cosine similarity -- the Euclidean distance
 *                      between L2-normalised features (Gram matrix on the tensor cores, raw bf16
 *                      inputs, normalisation applied in fp32 afterwards)
 *   metric 1 (euclid): d_ij^2 = |f_i|^2 + |f_j|^2 - 2 f_i.f_j
 */
typedef struct {
    int   metric;      /* 0 cosine, 1 euclid */
    float d_c;         /* cutoff distance of Eq. 2 (> 0) */
    float tau;         /* spatial threshold of Eq. 3 on the coordinates in `pos`; < 0 disables the test */
    double alpha;      /* centre ratio: n_centers = ceil(n * alpha) evaluated in double (a float 0.05 would make
                          200 * alpha exceed 10 and round up to 11); used when n_centers <= 0 */
    int   n_centers;   /* > 0 overrides alpha; clamped to n */
} vitcop_filter_params;

/*   feat       bf16 [B, n, D]          token features (D multiple of 64, n <= VITCOP_MAX_VISUAL_TOKENS)
 *   pos        fp32 [B, n, 2] or NULL  token coordinates (8-byte aligned); NULL disables the spatial test
 *   p          host pointer
 *   label      int32 [B, n]   out      token index of the centre of each token's cluster
 *   n_clusters int32 [B]      out      number of centres (same for every sample)
 *   rho        fp32 [B, n]    out, optional (NULL)   density, Eq. 2
 *   delta2     fp32 [B, n]    out, optional          delta_i^2, +inf for orphans
 *   parent     int32 [B, n]   out, optional          nearest denser neighbour N_i, -1 for orphans
 * Errors: INVALID_ARG (NULL feat/label/p, B or n or D < 0, d_c <= 0, metric not 0/1),
 * UNSUPPORTED (D % 64 != 0, n too large, misaligned feat), WORKSPACE, CUDA.  B == 0 or n == 0 is a no-op. */
int vitcop_redundancy_filter(const void* feat, const float* pos, int B, int n, int D,
                             const vitcop_filter_params* p, int32_t* label, int32_t* n_clusters,
                             float* rho, float* delta2, int32_t* parent,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Rows [row_begin, row_end) of the pairwise similarity matrix the filter works from (Algorithm 2,
 * step 1): cosine similarity s_ij for metric 0, the raw Gram value f_i.f_j for metric 1.  Produced by
 * the same tensor-core path as the filter; exported so that the similarity scores themselves can be
 * checked.   out: fp32 [B, row_end - row_begin, n]. */
int vitcop_similarity_rows(const void* feat, int B, int n, int D, int metric, int row_begin, int row_end,
                           float* out, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- K-norm saliency
 * Eq. 4 of the paper: score_i = sqrt( sum_h |K_i^(h)|_2^2 ) for every token i of the visual span; a
 * SMALLER norm means a MORE important token (Key Insight 2).  H is the number of K/V heads stored.
 *   K      bf16, element (b,h,t,e) at K + b*stride_b + h*stride_h + t*stride_n + e  (strides in elements,
 *          multiples of 8; d multiple of 8)
 *   score  fp32 [B, Nv_cap] out; entry (b, i) is token vis_start + i; entries at i >= vis_len[b] are untouched
 * Errors: INVALID_ARG (NULL K/score, negative sizes, vis_start + vis_len > N, vis_len > Nv_cap), UNSUPPORTED, CUDA. */
int vitcop_knorm_score(const void* K, int B, int H, int N, int d,
                       int64_t stride_b, int64_t stride_h, int64_t stride_n,
                       int vis_start, const int32_t* vis_len, int vis_len_uniform,
                       float* score, int Nv_cap, void* stream);

/* ---------------------------------------------------------------- budgeted selection
 * mode 0 (plain): Algorithm 1, Stage III -- keep the min(budget, vis_len) tokens with the smallest
 *   score (largest != 0: the largest, as Stage I does with Eq. 1); ties go to the lower index.
 * mode 1 (quota): Eq. 5 / Algorithm 3 up to the elite set -- with N_c distinct labels and n = vis_len,
 *   cluster c keeps its q_c = floor(|C_c| / n * (budget - N_c)) smallest-score tokens (integer
 *   arithmetic, ties -> lower index).  budget < N_c keeps nothing for that sample and records
 *   VITCOP_ERR_BUDGET in the workspace status word.  Merging of the rest (Eq. 6) is not done here.
 * NaN scores order after every number.
 *   score      fp32 [B, Nv_cap]
 *   label      int32 [B, Nv_cap], values in [0, vis_len); required in quota mode, ignored otherwise
 *   p          host pointer
 *   keep_idx   int32 [B, keep_stride] out: kept token indices relative to the span, ascending;
 *              keep_stride >= min(budget, Nv_cap); entries past n_keep[b] are untouched
 *   n_keep     int32 [B] out
 *   keep_mask  uint8 [B, Nv_cap] out, optional: 1 = kept
 * Errors: INVALID_ARG, UNSUPPORTED (Nv_cap > VITCOP_MAX_VISUAL_TOKENS), WORKSPACE, CUDA. */
typedef struct {
    int mode;      /* 0 plain, 1 quota */
    int largest;   /* plain mode only: 0 keep the smallest scores, 1 keep the largest */
    int budget;    /* k (plain) or the total budget B of Algorithm 3 (quota); >= 0 */
} vitcop_select_params;

int vitcop_select(const float* score, const int32_t* label, int B,
                  const int32_t* vis_len, int vis_len_uniform, int Nv_cap,
                  const vitcop_select_params* p,
                  int32_t* keep_idx, int keep_stride, int32_t* n_keep, uint8_t* keep_mask,
                  void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- order-preserving compaction
 * Materialises the shortened sequence the following layers run on (Algorithm 1: "process the token
 * sequence through layer l" after V_current shrank): output row r of sample b is the input row at
 *   r                                   for r <  vis_start                        (text before the span)
 *   vis_start + keep_idx[b][r-vis_start] for r <  vis_start + n_keep[b]            (kept visual tokens)
 *   r - n_keep[b] + vis_len[b]          for r <  out_len[b]                       (text after the span)
 * with out_len[b] = seq_len[b] - vis_len[b] + n_keep[b].  Rows are copied bit for bit.
 *   hidden      bf16 [B, N, Dh]      (any of hidden / K / V may be NULL together with its output)
 *   K, V        bf16 [B, H, N, d]
 *   seq_len     int32 [B] or NULL (= N for every sample)
 *   keep_idx    int32 [B, keep_stride], ascending, as written by vitcop_select;  n_keep int32 [B]
 *   hidden_out  bf16 [B, Ncap, Dh];  K_out, V_out bf16 [B, H, Ncap, d]; must not overlap the inputs
 *   kept_pos    int32 [B, Ncap] out, optional: input position of each output row, -1 past out_len
 *   out_len     int32 [B] out
 * Rows at r >= Ncap are not written (out_len still reports the full length, so the caller can tell).
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int vitcop_compact_kv(const void* hidden, const void* K, const void* V,
                      int B, int H, int N, int d, int Dh, const int32_t* seq_len,
                      int vis_start, const int32_t* vis_len, int vis_len_uniform,
                      const int32_t* keep_idx, int keep_stride, const int32_t* n_keep,
                      void* hidden_out, void* K_out, void* V_out, int Ncap,
                      int32_t* kept_pos, int32_t* out_len, void* stream);

/* ---------------------------------------------------------------- fused pruning step
 * One in-LLM pruning step of Algorithm 1 without host synchronisation: K-norm (Eq. 4) of the visual
 * span, selection under `budget` (label == NULL: plain top-k of Stage III; label != NULL: the
 * cluster quota of Stage II), and compaction of hidden states, K and V.
 * Arguments as in the three calls above (K, V dense [B, H, N, d]).  Optional outputs (NULL to skip):
 *   score_out fp32 [B, Nv_cap], keep_idx_out int32 [B, Nv_cap], n_keep_out int32 [B].
 * Nv_cap is the capacity of the visual span (>= every vis_len).  out_len and n_keep_out can feed the
 * next step's seq_len and vis_len directly. */
int vitcop_prune_step(const void* hidden, const void* K, const void* V,
                      int B, int H, int N, int d, int Dh, const int32_t* seq_len,
                      int vis_start, const int32_t* vis_len, int vis_len_uniform, int Nv_cap,
                      const int32_t* label, int budget,
                      void* hidden_out, void* K_out, void* V_out, int Ncap,
                      int32_t* kept_pos, int32_t* out_len,
                      float* score_out, int32_t* keep_idx_out, int32_t* n_keep_out,
                      void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- Stage II in one call
 * Algorithm 1 at layer l_s: VIC(F, P) -> cluster labels, K-norms (Eq. 4), collaborative pruning under the budget
 * (Eq. 5, Algorithm 3 up to the elite set) and compaction of hidden states, K and V -- the work of
 * vitcop_redundancy_filter followed by vitcop_prune_step with those labels, with identical results.  Being one
 * call, it may run the K-norm, which does not depend on the clustering, beside the clustering's sweep instead of
 * after it.  Every sample has the same Nv visual tokens at [vis_start, vis_start + Nv).
 *   feat bf16 [B, Nv, D], pos fp32 [B, Nv, 2] or NULL, fp (host) as in vitcop_redundancy_filter
 *   hidden, K, V, the outputs, kept_pos, out_len as in vitcop_prune_step (Nv_cap = Nv)
 *   label_out int32 [B, Nv] and n_clusters_out int32 [B]: required outputs (the labels the selection used)
 *   rho_out, delta2_out fp32 [B, Nv], parent_out int32 [B, Nv]: optional, as in vitcop_redundancy_filter
 *   score_out, keep_idx_out [B, Nv], n_keep_out [B]: optional
 *   workspace: vitcop_workspace_bytes(VITCOP_OP_COLLAB_STEP, B, 0, 0, 0, Nv, D, 0) bytes; one status word
 * Errors: as the two calls it replaces. */
int vitcop_collaborative_step(const void* feat, const float* pos, int D, const vitcop_filter_params* fp,
                              const void* hidden, const void* K, const void* V,
                              int B, int H, int N, int d, int Dh, int vis_start, int Nv, int budget,
                              void* hidden_out, void* K_out, void* V_out, int Ncap,
                              int32_t* kept_pos, int32_t* out_len,
                              int32_t* label_out, int32_t* n_clusters_out,
                              float* rho_out, float* delta2_out, int32_t* parent_out,
                              float* score_out, int32_t* keep_idx_out, int32_t* n_keep_out,
                              void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- cluster merge
 * Eq. 6 of the paper (second half of Algorithm 3): in every cluster the tokens that were NOT kept as elites are
 * averaged into one representative token, t_c = (1 / |R_c|) * sum_{i in R_c} t_i, so that a pruning step returns
 * the elites plus one merged token per cluster.  Rows are summed in fp32 in ascending token order.
 * Readings where the paper is silent: the merged tokens are hidden-state rows; they come out as a separate
 * tensor, one row per cluster that has non-elite tokens, in ascending order of the cluster's label (Algorithm 3
 * returns an unordered union, so where they go in the sequence is the caller's choice); a cluster whose tokens
 * were all kept yields no row.
 *   hidden        bf16 [B, N, Dh]   (Dh multiple of 8)
 *   label         int32 [B, Nv_cap]  cluster labels of the span, as written by vitcop_redundancy_filter
 *   keep_mask     uint8 [B, Nv_cap]  1 = elite (kept), as written by vitcop_select
 *   merged        bf16 [B, Mcap, Dh] out, optional: the averages rounded to nearest even
 *   merged_f32    fp32 [B, Mcap, Dh] out, optional: the averages before that rounding
 *   merged_label  int32 [B, Mcap] out: label of each merged row;  merged_count int32 [B, Mcap] out: |R_c|
 *   n_merged      int32 [B] out: number of clusters with non-elite tokens (rows past Mcap are not written)
 *   workspace     vitcop_workspace_bytes(VITCOP_OP_MERGE, B, 0, Mcap, 0, Nv_cap, 0, 0) bytes
 * Errors: INVALID_ARG, UNSUPPORTED (Dh % 8, alignment, Nv_cap > VITCOP_MAX_VISUAL_TOKENS), WORKSPACE, CUDA. */
int vitcop_merge_clusters(const void* hidden, int B, int N, int Dh,
                          int vis_start, const int32_t* vis_len, int vis_len_uniform, int Nv_cap,
                          const int32_t* label, const uint8_t* keep_mask,
                          void* merged, float* merged_f32, int32_t* merged_label, int32_t* merged_count,
                          int32_t* n_merged, int Mcap, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- Stage I saliency
 * Eq. 1 of the paper: S_i = sum_h A^(h)_{0,i}, the attention that the [CLS] token (index 0) of the vision
 * encoder pays to visual token i, summed over the heads; Stage I keeps the tokens with the LARGEST S
 * (vitcop_select with largest = 1, then vitcop_compact_kv on the feature rows).
 * A^(h)_{0,j} = softmax over all M keys j (the [CLS] key included) of scale * q^(h) . k_j^(h).
 *   q_cls     bf16 [B, H, d]      query of the [CLS] token per head (d multiple of 8)
 *   K         bf16 [B, H, M, d]   keys of the layer; key 0 belongs to [CLS]
 *   scale     usually 1 / sqrt(d)
 *   saliency  fp32 [B, M - 1] out: S of the visual tokens 1 .. M-1 (may be NULL when M <= 1: nothing to write)
 *   cls_self  fp32 [B] out, optional: attention of [CLS] to itself, summed over heads
 *   workspace vitcop_workspace_bytes(VITCOP_OP_SALIENCY, B, H, M, ...) bytes
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
int vitcop_cls_saliency(const void* q_cls, const void* K, int B, int H, int M, int d, float scale,
                        float* saliency, float* cls_self, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- K-norm at the source of K
 * Eq. 4 needs the K vectors "from the LLM's attention module".  This call produces them: K^(h)_t = W_k^(h) x_t for
 * every head as one bf16 GEMM on the tensor cores, optional rotary position embedding, K written in bf16 in the cache
 * layout the other calls read, and the K-norm of the visual span from the same pass, so that the pruning step needs
 * no second read of K (its largest byte term).  The norm is taken on the bf16 values that are stored (what
 * vitcop_knorm_score would compute from K_out), squares and sums in fp32; a rotation does not change it beyond
 * rounding (Eq. 4 is rotation invariant).
 *   hidden        bf16 [B, N, Dh]     layer input (Dh multiple of 64)
 *   W_k           bf16 [H * d, Dh]    key projection, one row per output feature (d multiple of 32)
 *   rope_cos/sin  fp32 [n_pos, d / 2] or both NULL: pairs (e, e + d / 2) of a head are turned by the angle of the
 *                 token's position, (a, b) -> (a cos - b sin, b cos + a sin); needs d in {64, 128, 256}
 *   position_ids  int32 [B, N] or NULL (position = token index); clamped to [0, n_pos)
 *   K_out         bf16 [B, H, N, d] out
 *   score         fp32 [B, Nv] out, optional: Eq. 4 of tokens vis_start .. vis_start + Nv - 1
 *   workspace     vitcop_workspace_bytes(VITCOP_OP_KPROJ, B, H, N, d, ..) bytes
 * Errors: INVALID_ARG, UNSUPPORTED (divisibility, alignment), WORKSPACE, CUDA. */
int vitcop_kproj_knorm(const void* hidden, const void* W_k, int B, int N, int Dh, int H, int d,
                       const float* rope_cos, const float* rope_sin, const int32_t* position_ids, int n_pos,
                       void* K_out, int vis_start, int Nv, float* score,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------- schedule and cost model (host arithmetic)
 * Algorithm 1 prunes to floor(m * pi) tokens per stage (pi relative to the ORIGINAL m visual tokens); Appendix E
 * models the cost.  Layers are numbered from 1; Stage II acts at layer l_s, Stage III at layer l_d.
 *   vitcop_stage_count            floor(m * pi), evaluated in double
 *   vitcop_flops_layer            Eq. 7: 4 N^2 d + 16 N d^2
 *   vitcop_visual_tokens_at_layer Eq. 8: pi1*m for l < l_s, pi2*m for l_s <= l < l_d, pi3*m from l_d on
 *   vitcop_flops_total            Eq. 9: sum over the n_layers layers of Eq. 7 at Eq. 8's length plus n_text
 *   vitcop_cr_int                 Eq. 10: one minus the layer average of Eq. 8 over m */
int    vitcop_stage_count(int m, double pi);
double vitcop_flops_layer(double N, double d);
double vitcop_visual_tokens_at_layer(int l, double m, double pi1, double pi2, double pi3, int l_s, int l_d);
double vitcop_flops_total(double m, double n_text, double d, double pi1, double pi2, double pi3,
                          int l_s, int l_d, int n_layers);
double vitcop_cr_int(double pi1, double pi2, double pi3, int l_s, int l_d, int n_layers);

/* ---------------------------------------------------------------- fused pruning step without a workspace
 * The paper has no counterpart: this is vitcop_prune_step for callers that have no way to obtain device
 * memory for a workspace at the point of the call -- code that runs where cudaMalloc is off limits (inside a
 * serving loop that must not touch the allocator, a plugin that is handed tensors but no allocator, a
 * latency-critical path where an allocation could stall on another stream's work).  Same arguments and
 * results as vitcop_prune_step, minus `workspace`: the scratch (status word, scores, keep list, counts) is a
 * buffer of VITCOP_STATIC_SCRATCH_BYTES built into the library image, which every GPU that loads the library
 * holds until the process exits.  The call allocates and frees nothing.
 *   - Limit: vitcop_workspace_bytes(VITCOP_OP_PRUNE_STEP, B, .., Nv_cap, ..) must not exceed
 *     VITCOP_STATIC_SCRATCH_BYTES (roughly B * Nv_cap <= 520,000); larger problems return
 *     VITCOP_ERR_UNSUPPORTED and nothing is launched.
 *   - The first call on each device looks up the buffer's device address (with that device current).  Make that
 *     first call outside any stream capture.
 *   - All calls on a device share the one buffer and it keeps what the last call left; each call resets the
 *     status word it needs zeroed and overwrites the rest before reading it.  Two calls whose work overlaps on
 *     the GPU (different streams, no ordering between them) race on the buffer: order them.
 *   - The device status word cannot be polled here; a quota budget below the cluster count shows as
 *     n_keep_out[b] == 0 and out_len[b] == text length. */
#define VITCOP_STATIC_SCRATCH_BYTES (4u << 20)

int vitcop_prune_step_static(const void* hidden, const void* K, const void* V,
                             int B, int H, int N, int d, int Dh, const int32_t* seq_len,
                             int vis_start, const int32_t* vis_len, int vis_len_uniform, int Nv_cap,
                             const int32_t* label, int budget,
                             void* hidden_out, void* K_out, void* V_out, int Ncap,
                             int32_t* kept_pos, int32_t* out_len,
                             float* score_out, int32_t* keep_idx_out, int32_t* n_keep_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VITCOP_H_ */
