/*
 * actqkv.h -- C ABI of the B200 (sm_100a) ActQKV per-window retrieval library.
 *
 * The library implements, as hand-written CUDA kernels, the per-window hot path
 * of "Activation-aware Probe-Query: Effective Key-Value Retrieval for
 * Long-Context LLMs Inference" (arXiv 2502.13542):
 *
 *   activation_bias -> probe_query -> score_blocks -> select_cutoff
 *                   -> retrieval_attention -> append_window
 *
 * Equation numbers.  The paper does not number its equations; the comments of this library number
 * them in order of appearance:
 *   Eq. 1  prefill attention over the full cache          (Sec. 3.1)
 *   Eq. 2  prefill attention over the selected cache      (Sec. 3.1)
 *   Eq. 3  decode attention                               (Sec. 3.1)
 *   Eq. 4  cache update                                   (Sec. 3.1)
 *   Eq. 5  top-k retrieval objective                      (Sec. 3.2)
 *   Eq. 6  anchor-token criterion                         (Sec. 4.1)
 *   Eq. 7  Activation Bias phi                            (Sec. 4.1)
 *   Eq. 8  running mean and variance of the queries       (Sec. 4.1)
 *   Eq. 9  activation-aware probe-query                   (Sec. 4.1)
 *   Eq. 10 cosine score of a probe and a key              (Sec. 4.2)
 *   Eq. 11 information density (entropy of the scores)    (Sec. 4.2)
 *   Eq. 12 per-layer budget of the dynamic KV cut-off     (Sec. 4.2)
 *   Algorithm 1  the cut-off over all layers              (Sec. 4.2)
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Every data pointer is a DEVICE pointer unless it is marked "host".  The
 *    caller owns every buffer; the library allocates nothing and keeps no state
 *    between calls (running statistics, budget state, pages and the
 *    representative-key table are caller-owned buffers updated in place).
 *  - Every call only ENQUEUES work on `stream` (a cudaStream_t passed as void*;
 *    NULL = the legacy default stream) and never synchronises.
 *  - Stream order is kept for every result, but kernels of consecutive calls on
 *    one stream may be RESIDENT together (programmatic dependent launch): the
 *    kernels of steps 1-4 let the next kernel of the stream start at once, and a
 *    kernel of this library that starts early reads, before it has waited for
 *    its predecessor, only buffers that steps 1-5 never write: the step's Q / K /
 *    V, pos0, page_table, the cache pages and table rows of tokens before pos0.
 *    It waits for its predecessor before it reads anything else and before it
 *    writes.  actqkv_append_window, which writes those buffers, runs strictly
 *    after its predecessor and before its successor in the stream, and so does
 *    a caller's own kernel between two calls unless it opts into the mechanism.
 *  - Return value: ACTQKV_OK (0) or a negative actqkv_status for problems the
 *    host can see (null / misaligned pointer, unsupported shape).  Nothing is
 *    enqueued when a negative code is returned.
 *  - Problems only the device can see (page index out of range, n_cand larger
 *    than the table, non-finite probe) never trap: the kernel clamps or skips
 *    the access and ORs an ACTQKV_DEV_* bit into the int32 word `status` points
 *    to (device memory, may be NULL).  The caller zeroes and reads that word.
 *  - Element type of Q / K / V / pages / representative table / O is
 *    cfg->dtype (fp32 or bf16).  Statistics, phi, probes, scores, theta, inverse
 *    norms and lse are fp32.  All data pointers must be 16-byte aligned.
 *  - Batching: a call processes n_seq x n_layers "units" (one unit = one
 *    (sequence, layer) pair); unit u = seq * n_layers + layer_local.  Tensors
 *    documented with a leading [U] are dense over units in that order.  A NULL
 *    batch means one sequence, one layer, layer0 = 0.
 *
 * Token / block geometry (the paper leaves it open; this is the library's rule)
 * ---------------------------------------------------------------------------
 *  Blocks tile the past after the n_init initial tokens: block b holds tokens
 *  [n_init + b*B, n_init + (b+1)*B).  For a step whose first token sits at
 *  absolute position p0 the candidates are the
 *      n = max(0, floor((p0 - n_local_prev - n_init) / B))
 *  complete blocks; the step attends to
 *      [0, n_init) | selected blocks | [n_init + n*B, p0) | step tokens (causal),
 *  and to plain causal [0, p] while p0 <= n_init.
 */
#ifndef ACTQKV_H_
#define ACTQKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ACTQKV_VERSION 100

typedef enum actqkv_status {
  ACTQKV_OK = 0,
  ACTQKV_ERR_NULL = -1,         /* a required pointer is NULL                 */
  ACTQKV_ERR_ALIGN = -2,        /* a data pointer is not 16-byte aligned      */
  ACTQKV_ERR_SHAPE = -3,        /* unsupported head_dim / window / block ...  */
  ACTQKV_ERR_DTYPE = -4,        /* dtype not supported by this entry point    */
  ACTQKV_ERR_LAUNCH = -5,       /* the CUDA runtime refused the launch        */
  ACTQKV_ERR_UNSUPPORTED = -6,  /* valid request this build cannot serve      */
  ACTQKV_ERR_SCRATCH_LIMIT = -7 /* needs more than the built-in scratch array */
} actqkv_status;

/* bits ORed into *status by kernels */
#define ACTQKV_DEV_BAD_PAGE      1   /* page index outside [0, n_phys_pages)      */
#define ACTQKV_DEV_NCAND_CLAMPED 2   /* n_cand > n_cap, clamped                   */
#define ACTQKV_DEV_BAD_PROBE     4   /* probe norm zero or not finite: scores = 0 */
#define ACTQKV_DEV_BAD_SELECTION 8   /* sel_count / sel_idx out of range, skipped */
#define ACTQKV_DEV_TIMEOUT       16  /* a bounded device-side wait expired        */
#define ACTQKV_DEV_TABLE_FULL    32  /* completed block index >= n_cap, not stored*/

enum { ACTQKV_F32 = 0, ACTQKV_BF16 = 1 };
enum { ACTQKV_STATS_CUMULATIVE = 0, ACTQKV_STATS_WINDOW_ONLY = 1 };
enum { ACTQKV_REPR_CHUNK_MEAN = 0, ACTQKV_REPR_STRIDED_TOKEN = 1 };
enum { ACTQKV_AGG_MEAN = 0, ACTQKV_AGG_MAX = 1 };
enum { ACTQKV_THETABAR_STREAMING = 0, ACTQKV_THETABAR_ALG1 = 1 };
/* Token weights of the probe-query: Eq. 9 (default), or uniform = the mean-pooling probe the paper
 * compares against (Sec. 1; the "w/o APQ" row of its ablation, Sec. 5.3). */
enum { ACTQKV_PROBE_ACTIVATION = 0, ACTQKV_PROBE_MEAN_POOL = 1 };
/* Which kernel serves actqkv_retrieval_attention: chosen by shape (default); the general
 * fp32-accumulate kernel; the single-CTA tensor-core kernel; the 4-CTA-cluster kernel that serves
 * four query heads per KV-head tile (G a multiple of 4; measured slower than the default CTA-pair
 * kernel, kept for comparison).  The non-default values exist for testing one kernel against
 * another; results agree within the rounding of the products. */
enum { ACTQKV_ATTN_AUTO = 0, ACTQKV_ATTN_GENERAL = 1, ACTQKV_ATTN_SINGLE_CTA = 2, ACTQKV_ATTN_CLUSTER4 = 3 };

/* Host POD describing the model / cache geometry.  Passed by const pointer (host). */
typedef struct actqkv_config {
  int32_t n_layers;      /* L: layers of the model (budget B_kv = L * k_blocks)          */
  int32_t n_q_heads;     /* Hq                                                            */
  int32_t n_kv_heads;    /* Hkv; G = Hq / Hkv <= 8                                        */
  int32_t head_dim;      /* D in {64, 128}                                                */
  int32_t window;        /* W: max tokens per step (the paper's m)                        */
  int32_t block;         /* B: tokens per block, multiple of page_tokens and of n_repr    */
  int32_t n_repr;        /* r: representative keys per block                              */
  int32_t page_tokens;   /* tokens per cache page (16)                                    */
  int32_t n_init;        /* initial tokens always attended, multiple of page_tokens       */
  int32_t n_local_prev;  /* recent past tokens kept local in addition to the step itself  */
  int32_t k_blocks;      /* k: average per-layer block budget                             */
  int32_t cap_blocks;    /* per-layer cap on selected blocks (row length of sel_idx)      */
  int32_t dtype;         /* ACTQKV_F32 | ACTQKV_BF16                                      */
  int32_t stats_mode;    /* ACTQKV_STATS_*: Eq. 8 cumulative over windows (default)       */
  int32_t repr_mode;     /* ACTQKV_REPR_*                                                 */
  int32_t agg_mode;      /* ACTQKV_AGG_*: block score = mean | max of its r cosines       */
  int32_t thetabar_mode; /* ACTQKV_THETABAR_*                                             */
  int32_t n_cap;         /* rows (blocks) per head in repr_k / scores                     */
  int32_t max_pages;     /* row length of page_table (logical pages per sequence)         */
  int32_t n_phys_pages;  /* pages in the pool of one layer                                */
  float beta;            /* softmax(beta * s) in Eq. 11; 1 = the paper                    */
  float sm_scale;        /* attention scale; 0 => 1/sqrt(D)                               */
  float var_eps;         /* floor on sigma^2 in Eq. 7; 0 => 1e-12                         */
  int32_t out_dtype;     /* element type of the attention output: ACTQKV_F32 | ACTQKV_BF16 */
  int32_t probe_mode;    /* ACTQKV_PROBE_*: token weights of the probe-query                 */
  int32_t attention_kernel; /* ACTQKV_ATTN_*: 0 = pick by shape                              */
  /* Test hooks of the failure-detection path (leave both 0).  With test_wait_limit > 0 the decode
   * attention kernel gives its device-side waits that many polls instead of the normal 2^24 and
   * never issues the K copy of tile test_drop_k_tile of each CTA, so that the wait for that tile runs
   * out: the kernel must set ACTQKV_DEV_TIMEOUT, return, and leave the context usable. */
  int32_t test_wait_limit;
  int32_t test_drop_k_tile;
} actqkv_config;

typedef struct actqkv_batch {
  int32_t n_seq;     /* sequences in this call                                 */
  int32_t n_layers;  /* layers batched in this call (consecutive)              */
  int32_t layer0;    /* model layer index of the first batched layer (0-based) */
} actqkv_batch;

/* ---- helpers ------------------------------------------------------------------------ */
int actqkv_version(void);
const char* actqkv_strerror(int status);
/* Bytes of the per-sequence budget state: double[1 + 2 * n_layers] =
 * { B_kv remaining, theta_sum[L], theta_count[L] }.  Zero it before the first step. */
int64_t actqkv_budget_state_bytes(const actqkv_config* cfg);
/* Candidate blocks and local-segment start for a step starting at p0 (host arithmetic). */
int32_t actqkv_n_candidates(const actqkv_config* cfg, int64_t p0);

/* ---- step 1: Activation Bias (Eq. 7, statistics Eq. 8) --------------------------------
 * For every unit and query head: merges the step's queries into the running
 * per-channel statistics (count, mean, M2 = sum of squared deviations; Eq. 8 is
 * mean and M2 / (count - 1) over ALL queries seen so far, this step included),
 * then phi[j,h,c] = (q[j,h,c] - mean[h,c])^2 / max(var[h,c], var_eps) and the token
 * indicator phi_l1[h,j] = sum_c phi[j,h,c].
 *   q          [U][n_tokens][Hq][D]  dtype, in
 *   stats_count[U][Hq]               int64, in/out (tokens merged so far)
 *   stats_mean [U][Hq][D]            fp32, in/out
 *   stats_m2   [U][Hq][D]            fp32, in/out
 *   phi_l1     [U][Hq][n_tokens]     fp32, out
 *   phi_full   [U][n_tokens][Hq][D]  fp32, out, may be NULL
 * With stats_mode WINDOW_ONLY the running buffers are ignored and left untouched.
 * Needs n_tokens * D * sizeof(dtype) <= 160 KiB. */
int actqkv_activation_bias(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                           int32_t n_tokens, int64_t* stats_count, float* stats_mean,
                           float* stats_m2, float* phi_l1, float* phi_full, int32_t* status,
                           void* stream);

/* ---- step 2: activation-aware probe-query (Eq. 9) --------------------------------------
 * probe_qh[h] = sum_j (phi_l1[h,j] / sum_j phi_l1[h,j]) * q[j,h,:]  (uniform weights when the
 * sum is 0, and always with probe_mode MEAN_POOL, which ignores phi_l1);
 * probe_kv[g] = mean of probe_qh over the G query heads of KV head g.
 * A step of one token (decode) gives probe_qh = q: the paper's decode-stage probe (Sec. 4.2).
 *   probe_qh [U][Hq][D] fp32 out;  probe_kv [U][Hkv][D] fp32 out. */
int actqkv_probe_query(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                       int32_t n_tokens, const float* phi_l1, float* probe_qh, float* probe_kv,
                       int32_t* status, void* stream);

/* Steps 1 + 2 in one kernel (Q is read from HBM once).  phi_l1 / phi_full may be NULL. */
int actqkv_bias_probe(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                      int32_t n_tokens, int64_t* stats_count, float* stats_mean, float* stats_m2,
                      float* phi_l1, float* phi_full, float* probe_qh, float* probe_kv,
                      int32_t* status, void* stream);

/* ---- step 3: cosine scores (Eq. 10) and information density (Eq. 11) -------------------
 * s[g,b] = agg_i <probe_kv[g], R[g,b,i]> * inv_norm[g,b,i] / ||probe_kv[g]|| for b < n_cand,
 * theta[g] = entropy (nat) of softmax(beta * s[g, :n_cand]).
 *   probe_kv      [U][Hkv][D]            fp32 in
 *   repr_k        [U][Hkv][n_cap][r][D]  dtype in
 *   repr_inv_norm [U][Hkv][n_cap][r]     fp32 in (1 / ||R||, 0 for a zero key)
 *   n_cand        [n_seq]                int32 in (device; same for every batched layer)
 *   scores        [U][Hkv][n_cap]        fp32 out (entries >= n_cand untouched)
 *   theta         [U][Hkv]               fp32 out (0 when n_cand == 0) */
int actqkv_score_blocks(const actqkv_config* cfg, const actqkv_batch* batch, const float* probe_kv,
                        const void* repr_k, const float* repr_inv_norm, const int32_t* n_cand,
                        float* scores, float* theta, int32_t* status, void* stream);

/* ---- step 4: dynamic KV cut-off (Eq. 12) and top-c selection (Algorithm 1) -------------
 * Layer density = mean over KV heads of theta.  Shallow to deep, per sequence:
 *   B^l = theta^l / (theta^l + sum_{j>l} thetabar^j) * B_kv,  c^l = clamp(floor(B^l + 1/2),
 *   min(1, n), min(cap, n)),  B_kv <- B_kv - c^l,  B_kv reset to L * k when layer 0 is processed.
 * thetabar^j: STREAMING = mean of layer j's density over earlier calls (theta^l itself while
 * layer j has no history); ALG1 = theta^j of this call (requires the batch to hold all L layers).
 * The chain runs in fp64 on the fp32 theta values.  Then per KV head the c^l highest scores
 * (ties: lower block index first; NaN last) are written in ascending block order.
 *   budget_state [n_seq] x actqkv_budget_state_bytes   in/out
 *   sel_idx   [U][Hkv][cap_blocks] int32 out, entries >= sel_count are -1
 *   sel_count [U]                  int32 out (c^l, shared by the KV heads)
 *   budget_real [U] fp32 out, may be NULL: the un-rounded B^l (diagnostic) */
int actqkv_select_cutoff(const actqkv_config* cfg, const actqkv_batch* batch, const float* scores,
                         const float* theta, const int32_t* n_cand, void* budget_state,
                         int32_t* sel_idx, int32_t* sel_count, float* budget_real, int32_t* status,
                         void* stream);

/* Steps 3 + 4 with the density computed inside the cut-off kernel (one launch fewer). */
int actqkv_score_select(const actqkv_config* cfg, const actqkv_batch* batch, const float* probe_kv,
                        const void* repr_k, const float* repr_inv_norm, const int32_t* n_cand,
                        void* budget_state, float* scores, float* theta, int32_t* sel_idx,
                        int32_t* sel_count, float* budget_real, int32_t* status, void* stream);

/* ---- step 5: attention over [initial | selected | local | step] (Eq. 2, Eq. 3) ---------
 * out[j,h] = softmax_over_keys(q[j,h] . k * sm_scale) v, keys as in the geometry rule above with
 * the selected blocks of KV head h / G, causal inside the step.
 *   q            [U][n_tokens][Hq][D]   dtype in
 *   k_win, v_win [U][n_tokens][Hkv][D]  dtype in (the step's own keys / values)
 *   k_pages, v_pages [n_layers_batched][n_phys_pages][Hkv][page_tokens][D] dtype in
 *   page_table   [n_seq][max_pages]     int32 in (logical page -> physical page)
 *   pos0         [n_seq]                int64 in (device): p0 of each sequence
 *   sel_idx, sel_count                  as written by select_cutoff
 *   out          [U][n_tokens][Hq][D]   cfg->out_dtype out
 *   lse          [U][Hq][n_tokens]      fp32 out, may be NULL (natural-log sum of exp)
 * bf16, D = 128, 16-token pages: steps whose n_tokens is a multiple of 128 run on the tcgen05
 * prefill kernels (CTA pairs when G is even; that kernel also takes pages of 32, 64 or 128 tokens), steps of n_tokens <= 128 / G tokens on the tcgen05
 * decode kernel (one CTA per KV head; see actqkv_decode_attention for the split form); every
 * other shape runs on the general fp32-accumulate kernel.
 * Preconditions of the tcgen05 kernels (the general kernel has none of them):
 *  - p0 need not sit on a page boundary, but the rows of the last, partly filled cache page that
 *    lie past p0 must hold finite values: they are masked out of the softmax yet still enter the
 *    P V product with weight 0, and 0 x NaN is NaN.  A zero-initialised pool satisfies this, and
 *    actqkv_append_window zero-fills the rest of the last page it touches.
 *  - The cluster and CTA-pair kernels multiply P and V in fp16: |v| <= 65504 (larger finite values saturate). */
int actqkv_retrieval_attention(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                               const void* k_win, const void* v_win, int32_t n_tokens,
                               const void* k_pages, const void* v_pages, const int32_t* page_table,
                               const int64_t* pos0, const int32_t* sel_idx, const int32_t* sel_count,
                               void* out, float* lse, int32_t* status, void* stream);

/* ---- step 5 for short steps (decode, Eq. 3) with the key stream split over several CTAs --------
 * The same attention as actqkv_retrieval_attention for steps of n_tokens <= 128 / G tokens
 * (G = Hq / Hkv; bf16, D = 128, 16-token pages), which packs the G query heads of a KV head into
 * one tensor-core tile so that K and V are read once per group.  With few (sequence, layer) units a
 * single CTA per KV head cannot fill the GPU: n_splits > 1 cuts every key stream into n_splits
 * shares; each share writes a partial result to `workspace` and a second kernel merges them
 * (n_splits = 0 picks the count that fills the SMs once; actqkv_decode_splits returns it).
 *   workspace  device scratch of at least actqkv_decode_workspace_bytes(...) bytes, 16-byte
 *              aligned, caller-owned, contents undefined on entry and exit; may be NULL when
 *              the split count is 1.  Calls that overlap on the GPU need distinct workspaces.
 * The rows of the last, partly filled cache page that lie past p0 must hold finite values
 * (e.g. a zero-initialised pool): they are masked out of the softmax but still enter the
 * P V product with weight 0.
 * Returns ACTQKV_ERR_UNSUPPORTED for shapes this kernel does not serve, ACTQKV_ERR_SHAPE when
 * workspace_bytes is too small. */
int32_t actqkv_decode_splits(const actqkv_config* cfg, const actqkv_batch* batch);
int64_t actqkv_decode_workspace_bytes(const actqkv_config* cfg, const actqkv_batch* batch, int32_t n_tokens,
                                      int32_t n_splits);
int actqkv_decode_attention(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                            const void* k_win, const void* v_win, int32_t n_tokens, const void* k_pages,
                            const void* v_pages, const int32_t* page_table, const int64_t* pos0,
                            const int32_t* sel_idx, const int32_t* sel_count, void* out, float* lse,
                            int32_t n_splits, void* workspace, int64_t workspace_bytes, int32_t* status,
                            void* stream);

/* ---- the split decode attention for callers that cannot allocate device memory ---------------
 * (An addition of this library; the paper has no counterpart.)
 * actqkv_decode_attention needs a caller-allocated workspace as soon as the key stream is split.
 * Some callers cannot provide one: an inference server that hands all of the GPU's memory to its
 * KV-cache pool at start-up and forbids allocations afterwards, or a per-token decode loop in
 * which a cudaMalloc (which synchronises the whole device) is not acceptable.  For them this
 * variant computes exactly the same result with the scratch taken from a fixed array of
 * ACTQKV_STATIC_SCRATCH_BYTES (8 MiB) that is part of the library's device image.  It calls no
 * allocation routine of any kind.
 *  - The array exists once per GPU that loads the library and stays reserved until the process
 *    ends, used or not.
 *  - A call whose scratch need (actqkv_decode_workspace_bytes for the same arguments) exceeds
 *    the array returns ACTQKV_ERR_SCRATCH_LIMIT and enqueues nothing: use fewer splits, or the
 *    workspace form.
 *  - The first call on each device looks up that device's copy of the array (the device must be
 *    current, as for every call).  Make that first call before any stream capture begins.
 *  - All calls on a device share the one array and it keeps whatever the last call wrote.  The
 *    kernels never read stale contents, so nothing has to be cleared, but two calls that may
 *    run at the same time on one GPU (different streams) race on it: serialise them, or give
 *    all but one of them the workspace form.
 * Arguments and results as actqkv_decode_attention, without workspace and workspace_bytes. */
#define ACTQKV_STATIC_SCRATCH_BYTES (8u << 20)
int actqkv_decode_attention_static(const actqkv_config* cfg, const actqkv_batch* batch, const void* q,
                                   const void* k_win, const void* v_win, int32_t n_tokens, const void* k_pages,
                                   const void* v_pages, const int32_t* page_table, const int64_t* pos0,
                                   const int32_t* sel_idx, const int32_t* sel_count, void* out, float* lse,
                                   int32_t n_splits, int32_t* status, void* stream);

/* ---- step 6: cache append (Eq. 4) and representatives of the completed blocks ----------
 * Copies the step's keys / values into the pages of tokens [p0, p0 + n_tokens) and, for every
 * block completed by them, writes its r representative keys (CHUNK_MEAN: mean of the keys of
 * each of the r consecutive B/r-token chunks, accumulated in fp64 and rounded to dtype;
 * STRIDED_TOKEN: the middle key of each chunk) and their inverse norms.
 *   k_pages, v_pages in/out;  repr_k, repr_inv_norm in/out (rows of completed blocks). */
int actqkv_append_window(const actqkv_config* cfg, const actqkv_batch* batch, const void* k_win,
                         const void* v_win, int32_t n_tokens, const int64_t* pos0, void* k_pages,
                         void* v_pages, const int32_t* page_table, void* repr_k,
                         float* repr_inv_norm, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ACTQKV_H_ */
