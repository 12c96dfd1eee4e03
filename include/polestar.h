/*
 * polestar.h -- C ABI of the Polestar denoising hot path for masked-diffusion LLMs
 * on NVIDIA B200 (sm_100a).
 *
 * One library call sequence decodes a batch of sequences:
 *
 *     polestar_init   -> block-0 entry forward        (Algorithm 1, block entry)
 *     loop:  polestar_commit -> polestar_step -> polestar_commit -> ...
 *
 * `polestar_step` runs ONE model forward (a block-entry forward or a within-block
 * step with drift-aware cache refresh); `polestar_commit` applies the confidence /
 * drift-event commit rule to the logits that forward produced and advances the
 * controller.  `polestar_init` already runs the first forward, so the first call
 * after it is `polestar_commit`.
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses of the current device,
 *     "host" pointers are ordinary CPU addresses.  No torch / C++ types cross the ABI.
 *   - The library allocates NO device memory (except where a function says so):
 *     weights and one workspace are caller-owned device buffers that must outlive
 *     the context.  The context itself is a small host object.
 *   - All work is enqueued on the CUDA stream given at init (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream).  `polestar_commit`,
 *     `polestar_tokens` and `polestar_read` synchronise that stream.
 *   - Every function returns 0 (POLESTAR_OK) or a negative error code and never
 *     throws or aborts.  Asynchronous CUDA errors surface at the next synchronising
 *     call as POLESTAR_E_CUDA.
 *   - Hidden states, logits, drift values and attention log-probabilities are
 *     float32.  Weights, K/V cache and GEMM operands have the model's dtype.
 *
 * Memory layout of the weights (device, model dtype, every matrix [out, in] row-major)
 *   embed, lm_head  [vocab, d_model]
 *   wqkv[l]         [(n_heads + 2 n_kv_heads) * head_dim, d_model]: query heads, then key
 *                   heads, then value heads.  Inside every query and key head the rows are
 *                   PAIR-INTERLEAVED: packed row 2i is logical row i and packed row 2i+1 is
 *                   logical row i + head_dim/2 (the two elements rotary embedding rotates
 *                   together).  Scores q.k do not depend on a common permutation of the head
 *                   dimension, so the cache simply keeps keys in this order.
 *   wo[l]           [d_model, n_heads * head_dim]
 *   w_gate_up[l]    [2 * d_ffn, d_model]: row 2f is gate row f, row 2f+1 is up row f
 *   w_down[l]       [d_model, d_ffn]
 *   norm1[l], norm2[l], final_norm   [d_model] float32 gains
 *
 *   TILE-MAJOR storage: a bf16 GEMM weight (wqkv, wo, w_gate_up, w_down, lm_head) whose
 *   out-features are a multiple of 256 and in-features a multiple of 64 is stored as contiguous
 *   [256][64] blocks, block (o / 256, i / 64) at block index (o / 256) * (in / 64) + i / 64 and
 *   element (o % 256, i % 64) inside it; the row order above applies to the index o.  Every
 *   other matrix (fp32 models, odd shapes, the embedding table) is plain row-major.  Streaming
 *   kernels then read each weight block as one sequential 32 KB burst.
 */
#ifndef POLESTAR_H
#define POLESTAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- error codes --------------------------------------------------------------- */
#define POLESTAR_OK            0
#define POLESTAR_E_INVAL      (-1)  /* bad argument / unsupported shape            */
#define POLESTAR_E_STATE      (-2)  /* call order violated                         */
#define POLESTAR_E_NOSPACE    (-3)  /* workspace too small                         */
#define POLESTAR_E_CUDA       (-4)  /* a CUDA call or kernel failed                */
#define POLESTAR_E_NONFINITE  (-5)  /* NaN / Inf met where a decision was needed   */
#define POLESTAR_E_TIMEOUT    (-6)  /* a bounded device-side wait ran out; the context
                                       is unusable afterwards (later calls: E_STATE)  */
#define POLESTAR_E_DONE       (-7)  /* every block is already decoded              */

/* ---- enumerations --------------------------------------------------------------- */
#define POLESTAR_F32  0
#define POLESTAR_BF16 1

/* stale-row selection (Sec. 4.1 "Measuring Drift and Layer-wise KV Updates") */
#define POLESTAR_SELECT_TOPK_FRAC 0   /* k = floor(select_frac * W + 1/2) largest drifts   */
#define POLESTAR_SELECT_TOPK_COUNT 1  /* k = select_k                                       */
#define POLESTAR_SELECT_THRESHOLD 2   /* drift > select_thresh                              */
#define POLESTAR_SELECT_ALL 3         /* every window row (full refresh)                    */
#define POLESTAR_SELECT_NONE 4        /* never refresh rows (drift still measured)          */
#define POLESTAR_SELECT_CLUSTER_TOPK 5 /* centroid proxies (the paper's default policy): drift is measured on
                                         n_clusters proxy rows per layer and the member rows of the cluster_k
                                         clusters with the largest drift are refreshed                       */

#define POLESTAR_FLAG_DRIFT_COMMIT  (1u << 0) /* drift-event clause of the commit rule (Sec. 4.2)  */
#define POLESTAR_FLAG_SUFFIX_COMMIT (1u << 1) /* suffix-block commit from the final packet          */
#define POLESTAR_FLAG_GE_COMPARE    (1u << 2) /* ">=" as in the text of Sec. 4.2; off: ">" (Alg. 1) */
#define POLESTAR_FLAG_NOCACHE       (1u << 3) /* every step is a full-sequence forward (baseline)   */
#define POLESTAR_FLAG_KEEP_HIDDEN   (1u << 4) /* keep per-layer active hidden states for read-back  */
#define POLESTAR_FLAG_SIMT_GEMM     (1u << 5) /* bf16 models: plain CUDA-core GEMMs (debug aid)     */
#define POLESTAR_FLAG_PROMPT_DEVICE (1u << 6) /* polestar_init: prompt ids are a DEVICE array       */
#define POLESTAR_FLAG_PROFILE       (1u << 7) /* bracket kernel families with CUDA events           */
#define POLESTAR_FLAG_NVFP4_HCACHE  (1u << 8) /* window hidden cache as NVFP4 residuals against the row's cluster
                                                 centroid (Sec. 4.1 "Cluster and Quantize Hidden States"; Appendix
                                                 "Quantization Format"): E2M1 codes, one E4M3 scale per 16 channels;
                                                 needs POLESTAR_SELECT_CLUSTER_TOPK and d_model % 128 == 0.  The
                                                 reference is the cluster's centroid at block entry (fixed for the
                                                 block); a row is encoded when it enters the cache (block entry, or
                                                 a packet row), and every later reader sees the decoded value.  */

/* kernel families reported by polestar_profile */
#define POLESTAR_PROF_GEMM_QKV     0
#define POLESTAR_PROF_GEMM_O       1
#define POLESTAR_PROF_GEMM_GATE_UP 2
#define POLESTAR_PROF_GEMM_DOWN    3
#define POLESTAR_PROF_GEMM_LM_HEAD 4
#define POLESTAR_PROF_ATTENTION    5
#define POLESTAR_PROF_STAGE        6  /* row table, embedding, RMSNorm staging */
#define POLESTAR_PROF_SELECT       7
#define POLESTAR_PROF_CONFIDENCE   8
#define POLESTAR_PROF_COMMIT       9
#define POLESTAR_PROF_MISC        10
#define POLESTAR_PROF_FAMILIES    11

#define POLESTAR_STEP_ENTRY_FULL   0
#define POLESTAR_STEP_ENTRY_WINDOW 1
#define POLESTAR_STEP_WITHIN       2

#define POLESTAR_MAX_BATCH 64

/* ---- plain-data descriptions ------------------------------------------------------ */
typedef struct polestar_ctx polestar_ctx;

/* Synthetic mask predictor: pre-norm Transformer, RMSNorm, rotary q/k at absolute
 * positions, grouped-query bidirectional attention, SwiGLU FFN, untied LM head. */
typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t dtype;                 /* POLESTAR_F32 | POLESTAR_BF16 */
    float   rms_eps, rope_theta;
    int32_t mask_id, eos_id;
} polestar_model;

/* All pointers are device pointers, BORROWED for the context's lifetime.
 * The six arrays of per-layer pointers are HOST arrays of n_layers device pointers. */
typedef struct {
    const void *embed, *lm_head;
    const float *final_norm;
    const void *const *wqkv, *const *wo, *const *w_gate_up, *const *w_down;
    const float *const *norm1, *const *norm2;
} polestar_weights;

/* Decoding parameters; defaults in comments are the paper's (Sec. 5.1, Appendix D Table
 * "Default hyperparameters"). */
typedef struct {
    int32_t batch, prompt_len, gen_len, block /*32*/, max_steps;
    int32_t win_prefix_blocks /*2*/, win_suffix_blocks /*1*/, full_entry_period /*2*/;
    int32_t select_mode /*TOPK_FRAC*/;
    float   select_frac /*0.25*/;
    int32_t select_k;
    float   select_thresh, drift_floor /*0*/;
    int32_t tau_upd /*3; <0: refresh every step; INT32_MAX: never*/, hist /*5*/;
    float   tau_s /*0.9*/, alpha /*10*/, tau_suffix /*0.9*/, logit_scale /*1*/;
    uint32_t flags /*DRIFT_COMMIT|SUFFIX_COMMIT|GE_COMPARE*/;
    /* Centroid proxies (Sec. 4.1 "Cluster and Quantize Hidden States", "Measuring Drift and Layer-wise KV
     * Updates"; Sec. 5.1: K = 8, k = 4), used by POLESTAR_SELECT_CLUSTER_TOPK only.  What the paper leaves open is
     * fixed as follows: spherical K-means of the window's layer-input hidden rows at every block entry, per layer,
     * centre j starting at the unit vector of window row floor((j + 1/2) W / K), kmeans_iters Lloyd iterations
     * (largest cosine, lowest cluster on ties; an empty cluster keeps its centre; no more rows than clusters:
     * every row its own cluster); a cluster's proxy is the mean of its members' hidden rows, queried at the
     * rounded mean of their positions, and follows its members when they are refreshed. */
    int32_t n_clusters /*8; 1..16*/, cluster_k /*4*/, kmeans_iters /*4; 1..16*/;
} polestar_params;

typedef struct {
    int32_t kind;            /* POLESTAR_STEP_*                                     */
    int32_t block_index;
    int32_t n_refreshing;    /* sequences whose cache is being refreshed this step  */
    int32_t rows;            /* rows forwarded per sequence (upper bound)           */
    int64_t forwards;        /* forwards so far, this one included                  */
} polestar_step_info;

typedef struct {
    int32_t n_committed, n_by_conf, n_by_drift, n_by_quota, n_suffix, n_eos; /* batch sums */
    int32_t rows_refreshed;  /* cache rows rewritten by the last step, all layers   */
    int32_t block_index;     /* block the commit belonged to                        */
    int32_t block_done;      /* 1: the next step is a block entry                   */
    int32_t all_done;        /* 1: every block decoded                              */
    int64_t forwards;        /* forwards so far                                     */
    int64_t generated, generated_non_eos;  /* running totals (TPF numerator, App. D.1) */
    int64_t launches;        /* kernels launched by this context so far             */
} polestar_commit_info;

/* ---- the decoding path ------------------------------------------------------------ */

/* Bytes of device workspace `polestar_init` needs for this model and these parameters
 * (0 if they are invalid), valid for any 256-byte aligned base address.  Pure host arithmetic. */
size_t polestar_workspace_bytes(const polestar_model *m, const polestar_params *p);

/* Create a context and run the block-0 entry forward (Algorithm 1: initial state,
 * block entry with a full-sequence forward, Sec. 4.1 "Initialization").
 *   prompt_ids_host  host, [batch][prompt_len] token ids in [0, vocab), none equal mask_id
 *                    (with POLESTAR_FLAG_PROMPT_DEVICE: a device array of the same shape, not
 *                    validated; out-of-range ids are clamped)
 *   workspace_dev    device, >= polestar_workspace_bytes(), 256-byte aligned, caller-owned;
 *                    the library zero-fills what it needs
 *   cuda_stream      cudaStream_t as void*
 * The POLESTAR_* environment switches are read here, once, into the context (and become the switches of the
 * stand-alone kernel calls below); nothing reads the environment on the launch path.
 * Errors: E_INVAL (NULLs, unsupported shape, bad ids), E_NOSPACE, E_CUDA. *out is NULL on error. */
int polestar_init(polestar_ctx **out, const polestar_model *m, const polestar_weights *w,
                  const polestar_params *p, const int32_t *prompt_ids_host,
                  void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/* One forward (Algorithm 1): a block-entry forward if the previous commit finished a block,
 * otherwise a within-block step: [patch caches from the packet -> active block over the
 * patched cache (Eq. 3) -> drift of the window rows (Eq. 4) -> select -> sparse forward of the
 * selected rows -> packet for the next layer] per layer, then logits and confidences.
 * Asynchronous.  info_host may be NULL.  Errors: E_STATE (commit pending), E_DONE, E_CUDA. */
int polestar_step(polestar_ctx *c, polestar_step_info *info_host);

/* Commit rule of Sec. 4.2 on the last forward's logits (confidence >= tau_s, or drift delta
 * >= alpha (tau_s - c)^2 on within-block steps, quota top-up, suffix rows by confidence),
 * Eq. 2 token update, controller bookkeeping.  Synchronises.  info_host may be NULL.
 * Errors: E_STATE (no forward pending, or the context failed earlier), E_NONFINITE, E_CUDA, and E_TIMEOUT
 * when a kernel of the forward gave up a bounded wait: its outputs may be partial and its counters are out of
 * step, so the context is dead from then on (every later step / commit returns E_STATE; destroy it). */
int polestar_commit(polestar_ctx *c, polestar_commit_info *info_host);

/* Copy the current token ids to host memory: out_host [batch][prompt_len + gen_len]. */
int polestar_tokens(polestar_ctx *c, int32_t *out_host);

/* Read-back of internal state for parity checks.  `what`: */
#define POLESTAR_READ_LOGITS      1  /* float [batch][block][vocab], last forward                */
#define POLESTAR_READ_CONF        2  /* float [batch][block]                                     */
#define POLESTAR_READ_YHAT        3  /* int32 [batch][block]                                     */
#define POLESTAR_READ_DELTA       4  /* float [batch][block] last-layer drift of active rows     */
#define POLESTAR_READ_DRIFT       5  /* float [batch][W_max] drift of window rows at `layer`     */
#define POLESTAR_READ_SEL_COUNT   6  /* int32 [batch] rows selected at `layer`                   */
#define POLESTAR_READ_SEL_IDX     7  /* int32 [batch][W_max] ascending window indices, `layer`   */
#define POLESTAR_READ_HIDDEN      8  /* float [batch][block][d] input of `layer` (0..n_layers;
                                        n_layers = final hidden); needs FLAG_KEEP_HIDDEN         */
#define POLESTAR_READ_KCACHE      9  /* model dtype [batch][N][n_kv*head_dim] (keys interleaved) */
#define POLESTAR_READ_VCACHE     10  /* model dtype [batch][N][n_kv*head_dim]                    */
#define POLESTAR_READ_HCACHE     11  /* float [batch][W_max][d] window hidden cache at `layer`   */
#define POLESTAR_READ_COMMIT     12  /* int32 [batch][block] bit0 commit, bit1 by confidence,
                                        bit2 by drift, bit3 by quota (last commit)               */
#define POLESTAR_READ_PPREV      13  /* float [batch][W_max][n_heads][N] stored log attention
                                        (log-probabilities, put together from the stored pair)   */
#define POLESTAR_READ_SUFFIX     14  /* int32 [batch][W_max] bit0 eligible, bit1 committed, bit2 the
                                        rule's own decision (confidence >= tau_suffix)           */
/* Quantities of the last commit (Sec. 4.2 "Current Block Commit"; Algorithm 1 after the layer loop): */
#define POLESTAR_READ_DRIFT_DELTA 15 /* float [batch][block] Delta = delta - mean(Theta)          */
#define POLESTAR_READ_TAU_D      16  /* float [batch][block] alpha (tau_s - c)^2                  */
#define POLESTAR_READ_THETA      17  /* float [batch][max(1,hist)][block] drift history ring: the
                                        vector pushed as number n (0-based) sits in slot n % hist */
#define POLESTAR_READ_THETA_COUNT 18 /* int32 [batch] vectors pushed since the block was entered  */
#define POLESTAR_READ_OWN_COMMIT 19  /* int32 [batch][block] the rule's own decision (bits as in
                                        READ_COMMIT), also when a forced decision replaced it    */
#define POLESTAR_READ_LABELS     20  /* int32 [batch][W_max] cluster of every window row at `layer`
                                        (centroid proxies; -1 beyond the window)                 */
/* With POLESTAR_SELECT_CLUSTER_TOPK, READ_DRIFT holds the drift of the n_clusters proxies in its first
 * n_clusters entries and READ_PPREV has the shape [batch][n_clusters][n_heads][N]. */
/* Libraries built with -DPOLESTAR_TRACE only (time stamps, see csrc/common.cuh): */
#define POLESTAR_READ_TRACE_KERNELS 98 /* int64 [8192]: next slot, then (kernel id, ns) pairs      */
#define POLESTAR_READ_TRACE_GEMM 99  /* int64 [CTAs][12] stamps of the traced GEMM kind            */
/* Synchronises, copies min(bytes, size of the item) bytes to dst_host.
 * Errors: E_INVAL (unknown item, bad layer, item not kept). */
int polestar_read(polestar_ctx *c, int32_t what, int32_t layer, void *dst_host, size_t bytes);

/* Forced decisions, for checking each step's arithmetic on its own when a near-tie would let
 * two correct implementations diverge.  `what`: */
#define POLESTAR_FORCE_SELECT 1  /* rows refreshed at `layer` in the next step: idx_host holds, per
                                    sequence, n ascending window indices ([batch][n])            */
#define POLESTAR_FORCE_COMMIT 2  /* positions committed by the next commit: idx_host holds, per
                                    sequence, n absolute positions ([batch][n]; -1 = unused)     */
#define POLESTAR_FORCE_CLEAR  3  /* drop all forced decisions                                     */
#define POLESTAR_FORCE_TOKENS 4  /* after FORCE_COMMIT with the same n: token ids written at those
                                    positions ([batch][n]) instead of the library's own argmax (two
                                    near-equal logits may rank differently in another arithmetic)  */
#define POLESTAR_FORCE_LABELS 5  /* centroid proxies: cluster labels of the window rows at `layer` for the next
                                    block-entry forward, instead of the library's own K-means ([batch][n],
                                    n = window rows; a near-tie between two centres may fall either way)  */
#define POLESTAR_FORCE_HCODES 6  /* NVFP4 hidden cache (context created with POLESTAR_FLAG_KEEP_HIDDEN too): codes
                                    of window rows at `layer`.  idx_host is a byte blob: mask uint8 [batch][n],
                                    codes uint8 [batch][n][d/2], scales uint8 [batch][n][d/16] (n = window rows).
                                    Rows with a non-zero mask take these codes now (the cache is rewritten), and
                                    again in place of the codec's own decision if the NEXT step encodes them
                                    (a value next to a code boundary may fall either way in another arithmetic) */
int polestar_force(polestar_ctx *c, int32_t what, int32_t layer, const int32_t *idx_host, int32_t n);

/* Per-family device time of the forwards so far (context created with POLESTAR_FLAG_PROFILE;
 * harvested at every polestar_commit).  out_host: double [POLESTAR_PROF_FAMILIES][4] =
 * {launch groups, milliseconds, algorithmic bytes, flops}.  reset != 0 clears the totals.
 * The paper has no counterpart (its Appendix D breakdown figure is the closest). */
int polestar_profile(polestar_ctx *c, double *out_host, int32_t reset);

void polestar_destroy(polestar_ctx *c);
const char *polestar_strerror(int code);

/* Re-read the POLESTAR_* environment switches for the stand-alone kernel calls below (contexts keep the
 * values they read at polestar_init).  The paper has no counterpart. */
int polestar_reload_env(void);

/* ---- single kernels of the path (unit parity, micro-benchmarks) --------------------- */
/* All pointers are device pointers owned by the caller; the calls are asynchronous on `cuda_stream`.
 * Return POLESTAR_OK or a negative code (POLESTAR_E_INVAL for null pointers, negative sizes,
 * unsupported shapes or misaligned buffers; POLESTAR_E_CUDA for a failed launch).  A call with zero
 * rows (R, rows, batch or W = 0) is a valid no-op: it returns POLESTAR_OK, touches nothing (select with
 * W = 0 writes zero counts) and accepts null row pointers. */


/* Drift of attention rows (Eq. 4; Algorithm 1 "ProxyAttn" + "KL"), optionally with the attention
 * output: for each of R query rows and each head, logp = log softmax_j(q.k_j / sqrt(head_dim))
 * over all N keys; kl[r][h] = sum_j p_j (logp_j - logp_prev_j); the stored row is then replaced
 * by the new one; out[r] = sum_j p_j v_j.
 * A stored row is a pair: row_prev_dev[r][h][:] and lse_prev_dev[r][h] with
 *     log-probability_j = row_prev[r][h][j] - lse_prev[r][h]
 * (callers that hold plain log-probabilities pass them with lse = 0).  On return the pair describes the
 * new distribution in the same way; which split the library chooses (scaled scores and their log-sum-exp,
 * or log-probabilities and 0) depends on the kernel that ran, so always subtract.
 *   q_dev [R][n_heads*head_dim], k_dev / v_dev [N][n_kv*head_dim] (model dtype; one sequence)
 *   row_prev_dev float [R][n_heads][N], lse_prev_dev float [R][n_heads], both in/out (both NULL: no KL,
 *   nothing stored)
 *   kl_dev float [R][n_heads] (NULL allowed iff row_prev_dev NULL), out_dev [R][n_heads*head_dim]
 *   model dtype (NULL: skipped). */
int polestar_k_attention(const void *q_dev, const void *k_dev, const void *v_dev,
                         float *row_prev_dev, float *lse_prev_dev, float *kl_dev, void *out_dev,
                         int32_t R, int32_t N, int32_t n_heads, int32_t n_kv_heads,
                         int32_t head_dim, int32_t dtype, void *cuda_stream);

/* Squared hidden-state change per row, sum_c (a[r][c] - b[r][c])^2 (Appendix B, Cor. 1's
 * Delta H): a_dev, b_dev [rows][d] model dtype -> out_dev float [rows]. */
int polestar_k_hidden_delta(const void *a_dev, const void *b_dev, float *out_dev,
                            int32_t rows, int32_t d, int32_t dtype, void *cuda_stream);

/* Stale-row selection and compaction (Sec. 4.1 top-k; Algorithm 1 "TopK").  Per sequence s of
 * `batch`: among the W rows with drift_dev[s][i] > floor choose by `mode` (POLESTAR_SELECT_*;
 * ties: lower index first) and write their indices ascending to idx_dev[s][0..count), count_dev[s].
 * W <= 4096. */
int polestar_k_select(const float *drift_dev, int32_t batch, int32_t W, int32_t mode, int32_t k,
                      float thresh, float floor_, int32_t *idx_dev, int32_t *count_dev,
                      void *cuda_stream);

/* Gathered K/V refresh (Sec. 4.1; Algorithm 1 "Patch"): for each sequence s and each
 * i < count_dev[s], row = idx_dev[s][i]: a = RMSNorm(h_dev[s][row]) * norm; (q,k,v) = a Wqkv^T;
 * rotary on q,k at position `row`; k,v written to kc_dev[s][row], vc_dev[s][row]; q to
 * q_out_dev[s][i] (NULL: dropped).  Rows not listed are not touched.
 *   h_dev [batch][P][d], kc_dev/vc_dev [batch][P][n_kv*head_dim], model dtype
 *   wqkv_dev as in polestar_weights; max_rows = upper bound of count (<= P)
 *   scratch_dev: >= polestar_k_refresh_scratch_bytes(...) bytes, 1024-byte aligned. */
size_t polestar_k_refresh_scratch_bytes(int32_t batch, int32_t max_rows, int32_t d,
                                        int32_t n_heads, int32_t n_kv_heads, int32_t head_dim);
int polestar_k_refresh(const void *h_dev, const int32_t *idx_dev, const int32_t *count_dev,
                       const void *wqkv_dev, const float *norm_dev, void *kc_dev, void *vc_dev,
                       void *q_out_dev, int32_t batch, int32_t P, int32_t max_rows, int32_t d,
                       int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float rms_eps,
                       float rope_theta, int32_t dtype, void *scratch_dev, size_t scratch_bytes,
                       void *cuda_stream);
/* Outcome of the last polestar_k_refresh on this scratch (same batch, max_rows, d, head_dim): synchronises the
 * stream; POLESTAR_OK, or POLESTAR_E_TIMEOUT if a bounded device-side wait of its projection gave up (the cache
 * rows of that call are then incomplete). */
int polestar_k_refresh_status(const void *scratch_dev, size_t scratch_bytes, int32_t batch, int32_t max_rows,
                              int32_t d, int32_t head_dim, void *cuda_stream);

/* The bounded device-side wait on its own (every wait of the library on a counter, flag or mbarrier has a limit; the
 * paper has no counterpart).  One thread waits until *counter_dev (uint32, wrap-safe comparison) reaches `expect` or
 * `limit_cycles` SM clock cycles (1 .. 2e9) have passed; synchronises the stream.  Returns POLESTAR_OK, or
 * POLESTAR_E_TIMEOUT when the wait gave up (*status_dev = 1): the CUDA context stays usable, nothing was trapped. */
int polestar_k_wait_probe(const uint32_t *counter_dev, uint32_t expect, int64_t limit_cycles, int32_t *status_dev,
                          void *cuda_stream);

/* The NVFP4 residual codec on its own (Appendix "Quantization Format"): for every row, codes and scales of
 * x - ref and the stored value ref + decode(...).  float32 arithmetic: scale = E4M3(amax / 6) (nearest even,
 * saturating), codes to the nearest E2M1 value (ties to the even code, saturating at 6).
 *   x_dev, ref_dev, deq_dev float [rows][d] (16-byte aligned), d % 128 == 0
 *   codes_dev uint8 [rows][d/2] (channel 2i in the low nibble: bit 3 sign, bits 0-2 grid index)
 *   scales_dev uint8 [rows][d/16] (E4M3 bit patterns). */
int polestar_k_nvfp4_residual(const float *x_dev, const float *ref_dev, int32_t rows, int32_t d,
                              uint8_t *codes_dev, uint8_t *scales_dev, float *deq_dev, void *cuda_stream);

/* Confidence of logits rows (Eq. 1; Sec. 2 sampler set): per row, y_hat = argmax over v != mask_id
 * (lowest id on ties), conf = softmax(logits)[y_hat].  logits_dev float [rows][vocab], 16-byte aligned
 * when vocab % 4 == 0 (E_INVAL otherwise); scratch_dev: >= rows * 512 bytes of device memory. */
int polestar_k_confidence(const float *logits_dev, int32_t rows, int32_t vocab, int32_t mask_id,
                          int32_t *yhat_dev, float *conf_dev, void *scratch_dev, size_t scratch_bytes,
                          void *cuda_stream);

/* Same result as polestar_k_confidence for callers that cannot provide or allocate device scratch
 * (a server whose memory pool owns every byte of the GPU, a loop that must not hit cudaMalloc's
 * device-wide synchronisation, a plug-in interface that passes inputs and outputs only).  The
 * partial results live in a 512 KB array that is part of the library image on every GPU using it.
 * The paper has no counterpart: this is a packaging variant of the confidence kernel.
 *   - rows <= POLESTAR_NOALLOC_MAX_ROWS, otherwise POLESTAR_E_NOSPACE (use polestar_k_confidence).
 *   - Calls no allocation routine.  The first call on each device looks up the array's device
 *     address (cudaGetSymbolAddress, with the caller's current device); make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array: calls that may overlap on the GPU (different
 *     streams without ordering) race on it and must be serialised by the caller.  Nothing in the
 *     array has to be cleared between calls; it simply keeps the last call's partial results. */
#define POLESTAR_NOALLOC_MAX_ROWS 1024
int polestar_k_confidence_noalloc(const float *logits_dev, int32_t rows, int32_t vocab, int32_t mask_id,
                                  int32_t *yhat_dev, float *conf_dev, void *cuda_stream);

/* Number of SMs of the device the library last sized grids for (0 before any call that launches kernels). */
int polestar_sm_count(void);

#ifdef __cplusplus
}
#endif
#endif /* POLESTAR_H */
