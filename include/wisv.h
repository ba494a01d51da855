/*
 * wisv.h - C ABI of the WISV edge-side verifier for one NVIDIA B200 (sm_100a).
 *
 * One call verifies a batch of speculative-decoding windows the way the edge
 * server does in one round of Algorithm 1 of "WISV: Wireless-Informed Semantic
 * Verification for Distributed Speculative Decoding in Device-Edge LLM
 * Inference":
 *
 *   1. logits of the target model at the K+1 window positions (the LM-head part
 *      of Verify; Section IV-B: the logits serve mismatch localisation and
 *      correction) - never written out, only reduced;
 *   2. per position: argmax, log-sum-exp and the target probability of the draft
 *      token (Section II-A, greedy verification and Eq. 1);
 *   3. Localize: the candidate set S of mismatching positions (Section V-C);
 *   4. the CSI-aware decision head p = sigmoid(w2 . act(W1 [h^D; h^T; c] + b1) + b2)
 *      (Eqs. 23-25) on full-hidden (FH) or selective-hidden (SH) uploads
 *      (Section III-B);
 *   5. the earliest position of S whose rejection probability reaches tau
 *      (Eq. 27), the accepted length and the correction / bonus token (Algorithm 1,
 *      full-accept and commit-and-correct branches; Section III-A step 4).
 *
 * Indexing.  Request b has a draft window of K_b tokens (K_b <= 64).  Tokens are
 * addressed by t = k_off[b] + i (i = 0..K_b-1, T = sum K_b) and window rows by
 * r = k_off[b] + b + i (i = 0..K_b, R = T + B).  Row i < K_b holds the target's
 * final hidden state whose logits predict draft token i; row K_b yields the
 * bonus token of a full accept.  accept_len counts accepted draft tokens
 * (the paper's j-hat minus one, or K_b), correction_token = argmax of row
 * accept_len in both branches.
 *
 * Numerics.  Hidden states are rounded to bf16 (nearest even) before every
 * matrix product - fp32 and fp16 inputs are rounded by the library, bf16 inputs
 * are taken as they are; weights are bf16; accumulation and everything after
 * the products is fp32.  CSI features and the CSI columns of W1 enter in fp32.
 *
 * Conventions.  Every function returns 0 (WISV_OK) or a negative error code; no
 * function throws, aborts or prints.  Pointers marked "dev" are CUDA device
 * pointers owned by the caller; the library never frees them.  The weights are
 * borrowed for the lifetime of the context (the LM head is not copied).  The
 * context owns its workspace, a repacked copy of W1 and its TMA descriptors.
 * wisv_verify only enqueues work on the given stream: results are valid once
 * the caller has synchronised that stream.  A context serves one call at a time
 * (calls on one context must be stream-ordered).  There is no CPU fallback: on a
 * device that is not compute capability 10.x wisv_create fails with WISV_EARCH.
 */
#ifndef WISV_H_
#define WISV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define WISV_VERSION 100

/* error codes */
#define WISV_OK         0
#define WISV_EINVAL    -1   /* NULL pointer, bad enum, bad mode bits */
#define WISV_ESHAPE    -2   /* dimension out of the supported range */
#define WISV_EALIGN    -3   /* pointer or pitch not aligned as documented */
#define WISV_ECAPACITY -4   /* batch exceeds the capacities given at create */
#define WISV_ECUDA     -5   /* a CUDA runtime / driver call failed */
#define WISV_EARCH     -6   /* current device is not sm_100 */
#define WISV_ENOMEM    -7   /* allocation failed */
#define WISV_EDEVICE   -8   /* a kernel reported a pipeline time-out (see wisv_device_error) */

/* activation of the decision head */
#define WISV_ACT_RELU 0     /* Eq. 25 as printed */
#define WISV_ACT_GELU 1     /* exact erf form */

/* mode bits of wisv_batch.mode */
#define WISV_MODE_FH           0u  /* draft_hidden is dense [T, H_d] */
#define WISV_MODE_SH           1u  /* draft_hidden is packed [M_sel, H_d] with sel_off / sel_pos */
#define WISV_ACCEPT_GREEDY     0u  /* S = { i : draft token != argmax } */
#define WISV_ACCEPT_STOCHASTIC 2u  /* S = { i : !(u_i < min(1, p_T(y_i) / q_i)) }  (Eq. 1) */

/* per-request status bits written by the device */
#define WISV_ST_MISSING_HIDDEN 1   /* a position of S had no uploaded hidden state: rejected greedily */
#define WISV_ST_BAD_TOKEN      2   /* a draft token id was outside [0, V): clamped */
#define WISV_ST_NONFINITE      4   /* a non-finite log-sum-exp or head logit was seen */
#define WISV_ST_BAD_SELECT     8   /* a sel_pos entry was outside [0, K_b): ignored */
#define WISV_ST_BAD_WINDOW    16   /* k_off gave this request a window outside 0..WISV_MAX_K tokens: only its first
                                      WISV_MAX_K positions (or none) were verified.  k_off lives on the device, so
                                      wisv_verify cannot check it; wisv_verify_host does and returns WISV_ESHAPE */

/* element type of a hidden-state array (wisv_batch.target_hidden_dtype / draft_hidden_dtype) */
#define WISV_DT_F32  0      /* fp32: rounded to bf16 (nearest even) by the library */
#define WISV_DT_BF16 1      /* bf16: used as it is */
#define WISV_DT_F16  2      /* fp16 (the 16-bit upload format of Section IV-A, b_h = 16): rounded to bf16 (nearest even) */

#define WISV_MAX_K   64
#define WISV_MAX_DC  16

typedef struct wisv_ctx wisv_ctx;

typedef struct {
    int32_t H;              /* target hidden size; H % 8 == 0 */
    int32_t V;              /* vocabulary size */
    int32_t H_d;            /* drafter hidden size; H_d % 8 == 0 */
    int32_t d_c;            /* CSI features, 0..WISV_MAX_DC */
    int32_t d_J;            /* decision-head hidden width */
    int32_t act;            /* WISV_ACT_* */
    int32_t head_row_shift; /* 0: h^T_i is window row i (the row scored against draft token i); 1: row i+1 */
    float   tau;            /* default threshold: reject iff p >= tau; 0 = greedy, > 1 = accept all */
    int32_t max_requests;   /* capacity: B */
    int32_t max_rows;       /* capacity: R = T + B */
    int32_t max_sel;        /* capacity: M_sel (SH); 0 = max_rows */
    int32_t vocab_base;     /* vocabulary sharding: lm_head holds tokens [vocab_base, vocab_base + V) ... */
    int32_t vocab_total;    /* ... of a vocabulary of vocab_total tokens; 0 = not sharded (vocab_base must be 0) */
} wisv_config;

typedef struct {
    const void*  lm_head;   /* dev bf16 [V, H] row-major, 16-byte aligned */
    const void*  W1;        /* dev bf16 [d_J, H_d + H + d_c] row-major, columns [h^D | h^T | c] (Eq. 23) */
    const float* b1;        /* dev fp32 [d_J] */
    const float* w2;        /* dev fp32 [d_J] */
    float        b2;
} wisv_weights;

typedef struct {
    int32_t B;                     /* requests */
    int32_t K;                     /* uniform window length, or 0 with k_off != NULL */
    const int32_t* k_off;          /* dev int32 [B+1] prefix sums of K_b (ragged), or NULL */
    int32_t T_total;               /* sum of K_b (host-known; = B*K when uniform) */
    const void*    target_hidden;  /* dev [R, H], element type target_hidden_dtype (fp32 by default), 16-byte aligned */
    const int32_t* draft_tokens;   /* dev int32 [T] */
    const void*    draft_hidden;   /* dev [T, H_d] (FH) or [M_sel, H_d] (SH), element type draft_hidden_dtype */
    const int32_t* sel_off;        /* SH: dev int32 [B+1], CSR offsets into sel_pos */
    const int32_t* sel_pos;        /* SH: dev int32 [M_sel], window-relative positions */
    int32_t M_sel;                 /* SH: number of uploaded hidden states */
    const float*   csi;            /* dev fp32 [B, d_c] */
    const float*   draft_q;        /* stochastic: dev fp32 [T], drafter probability of its token */
    const float*   uniforms;       /* stochastic: dev fp32 [T], u in [0, 1) */
    uint32_t mode;                 /* WISV_MODE_* | WISV_ACCEPT_* */
    float    tau;                  /* NaN: use the context default */
    int32_t  target_hidden_dtype;  /* WISV_DT_*: element type of target_hidden (0 = fp32) */
    int32_t  draft_hidden_dtype;   /* WISV_DT_*: element type of draft_hidden; the drafter uploads its hidden states with
                                      b_h = 16 bits per element (Section IV-A, Eq. 3), i.e. WISV_DT_F16 or WISV_DT_BF16 */
} wisv_batch;

typedef struct {
    int32_t*  accept_len;        /* dev [B], required */
    int32_t*  correction_token;  /* dev [B], required */
    int32_t*  argmax;            /* dev [R], optional */
    float*    lse;               /* dev [R], optional */
    float*    p_draft;           /* dev [T], optional: target probability of each draft token */
    float*    head_prob;         /* dev [T] (FH) or [M_sel] (SH), optional */
    uint64_t* mismatch_mask;     /* dev [B], optional: bit i set iff position i is in S */
    int32_t*  n_mismatch;        /* dev [B], optional: |S| (m_r of Section IV-A) */
    int32_t*  status;            /* dev [B], optional: WISV_ST_* bits */
} wisv_result;

/*
 * Create a verifier context on the current CUDA device (Algorithm 1's Require
 * line: decision head g_theta, threshold tau; the LM head belongs to the target
 * model T).  Validates dimensions and alignment, allocates the workspace for the
 * stated capacities, splits W1 into a bf16 [d_J, H_d+H] block and an fp32
 * [d_J, d_c] CSI block (device-to-device, on the default stream, synchronised
 * before returning) and encodes the TMA descriptors.  *out is NULL on failure.
 */
int wisv_create(const wisv_config* cfg, const wisv_weights* weights, wisv_ctx** out);

/*
 * Enqueue one verification round (Algorithm 1, from Verify's logits to the
 * feedback pair) for a batch on `cuda_stream` (a cudaStream_t; NULL = default
 * stream).  All pointers in `batch` and `result` are device pointers.  Host-side
 * argument errors are returned before anything is launched; conditions only the
 * device can see are reported through result->status.  Does not synchronise.
 */
int wisv_verify(wisv_ctx* ctx, const wisv_batch* batch, const wisv_result* result, void* cuda_stream);

/*
 * The selective-hidden protocol in the two steps the paper runs it in (Algorithm 1:
 * Verify and Localize, then RequestHidden / Upload of the hidden states of S, then the
 * decision; Section III-B option 2 and the payloads B_req, B_u2 of Eqs. 8-9).
 *
 * wisv_localize runs steps 1-3 of the round: it needs B, K / k_off, T_total,
 * target_hidden, draft_tokens (and draft_q, uniforms for the stochastic test) and
 * writes any of mismatch_mask, n_mismatch (m_r, what the edge requests from the
 * device), argmax, lse, p_draft; if accept_len / correction_token are given they
 * receive the plain greedy result (what the round yields if no hidden state ever
 * arrives).  The context keeps the per-row argmax and the candidate sets.
 *
 * wisv_decide runs steps 4-5 for the batch of the preceding wisv_localize on the same
 * context (same B, K / k_off pointer and T_total, else WISV_ESHAPE; WISV_EINVAL if no
 * localize is pending): it needs target_hidden again (h^T is a head input),
 * draft_hidden with sel_off / sel_pos (WISV_MODE_SH) or dense (WISV_MODE_FH), csi and
 * tau, and writes accept_len, correction_token and optionally head_prob,
 * mismatch_mask, n_mismatch, status.  Localize followed by decide gives exactly the
 * result of one wisv_verify on the same inputs.  Both calls only enqueue work.
 */
int wisv_localize(wisv_ctx* ctx, const wisv_batch* batch, const wisv_result* result, void* cuda_stream);
int wisv_decide(wisv_ctx* ctx, const wisv_batch* batch, const wisv_result* result, void* cuda_stream);

/*
 * The LM head sharded by vocabulary over several GPUs (each window is verified independently,
 * Section II-A, and the logits of a row reduce associatively over the vocabulary): every GPU creates
 * a context on its slice of the LM head (wisv_config.vocab_base / vocab_total) and on the whole
 * decision head.
 *
 * wisv_shard_rows reduces this shard's logits of the R window rows to one 16-byte partial per row
 * (out: dev [R]); it needs the same batch fields as wisv_localize.  The caller gathers the partials of
 * all G shards into one dev array [G][R] (an all-gather of R * 16 bytes per GPU; any order of shards)
 * and passes it to wisv_verify_gathered on the same context, which needs the batch fields of
 * wisv_verify and completes the round: same outputs as wisv_verify on the unsharded LM head, argmax
 * bit-identical outside exact ties between shards, log-sum-exp up to fp32 summation order.
 */
typedef struct {
    float   max;        /* largest logit of the row in this shard */
    int32_t argidx;     /* its global token id (lowest on ties) */
    float   sumexp;     /* sum of exp(logit - max) over the shard */
    float   tok_logit;  /* logit of the row's draft token if this shard owns it, else -inf */
} wisv_row_partial;

int wisv_shard_rows(wisv_ctx* ctx, const wisv_batch* batch, wisv_row_partial* out, void* cuda_stream);
int wisv_verify_gathered(wisv_ctx* ctx, const wisv_batch* batch, const wisv_row_partial* gathered, int32_t n_shards,
                         const wisv_result* result, void* cuda_stream);

/*
 * Same round with HOST buffers: every pointer in `batch` and `result` is host
 * memory, pinned or pageable, with no alignment requirement.  A hidden-state
 * array of at most 1 MiB in pinned, 16-byte aligned memory is read in place by
 * the first kernel; otherwise it is copied to a staging buffer owned by the
 * context (allocated on first use).  All other inputs are packed into one
 * pinned block, which the kernels read in place when it is at most 8 KB and
 * which travels in one copy otherwise.  The last kernel writes the requested
 * results into a device-mapped pinned block and then a completion word; the
 * call waits for that word (looking at the stream now and then, so a failed
 * launch or kernel ends the wait with WISV_ECUDA), copies the results to the
 * caller's arrays and returns: the results are valid on return, the stream may
 * still be retiring the last kernel.  Not for use during stream capture.
 * One call at a time per context: the staging memory is reused by the next
 * call.  Returns WISV_EDEVICE if a kernel reported a time-out.
 */
int wisv_verify_host(wisv_ctx* ctx, const wisv_batch* batch, const wisv_result* result, void* cuda_stream);

/* Free the context and everything it owns.  The caller must have synchronised. */
int wisv_destroy(wisv_ctx* ctx);

/*
 * Read (and clear) the device error word: non-zero if a bounded wait inside a
 * kernel gave up.  Synchronises the given stream first.
 */
int wisv_device_error(wisv_ctx* ctx, void* cuda_stream, int32_t* flags);

/*
 * Per-stage device timing.  After wisv_profile_enable(ctx, n) the library
 * records CUDA events around each kernel of the next calls (ring of n calls);
 * wisv_profile_read synchronises and returns, for stage s (0 = pack/cast,
 * 1 = LM head, 2 = decision head, 3 = merge + scan), the elapsed milliseconds
 * of up to `cap` recorded calls, oldest first.  n = 0 disables profiling.
 */
int wisv_profile_enable(wisv_ctx* ctx, int32_t n_calls);
int wisv_profile_read(wisv_ctx* ctx, int32_t stage, float* ms, int32_t cap, int32_t* n_out);

/*
 * Override the launch plan (0 in a field = choose automatically): vocabulary rows
 * per LM-head tile and decision-head columns per tile (multiples of 16, <= 256)
 * and the depth of the shared-memory stage ring (>= 2; capped by what fits).
 * NULL restores the automatic plan.  The partial buffers are sized for any legal
 * setting; results do not depend on the plan beyond fp32 summation order.
 */
typedef struct {
    int32_t lm_tile_n, lm_stages, head_tile_n, head_stages;
    int32_t lm_single_cta;   /* 1: never use the CTA-pair LM-head kernel (batches with more than 128 window rows) */
    int32_t head_ctas;       /* where the two GEMMs share one launch (always up to 256 window rows; with more rows
                                when it costs the LM head no extra round of tiles): CTAs given to the decision head
                                there (0 = chosen automatically), -1 = always two launches */
    int32_t lm_mma_m;        /* 128: never use 64-row MMAs (the default for GEMMs with at most 64 valid rows) */
    int32_t lm_kb_per_stage; /* CTA-pair LM-head kernel: K blocks (of 64) per shared-memory stage: 1, 2 or 4 */
    int32_t lm_teams;        /* CTA-pair LM-head kernel with 2 or more row blocks: 1 = one team of pairs per row block,
                                each dealing out the whole vocabulary with carried row state (whenever all window rows
                                fit in L2), -1 = never (round-robin work items), 0 = chosen automatically */
} wisv_tuning;
int wisv_set_tuning(wisv_ctx* ctx, const wisv_tuning* tuning);

/*
 * The launch planner on its own (host arithmetic only, no CUDA call, no context): the plan wisv_verify would use
 * for a batch with R window rows and P head positions on a device with sm_count SMs and max_smem_bytes of
 * opt-in shared memory per block, for the dimensions in cfg (H, V, H_d, d_c, d_J).  For tests and capacity
 * planning.  *_carry = 1: every CTA (or CTA pair) owns one contiguous range of the weight rows, units_base units
 * each (the first units_rem one more; a unit is 16 rows, 32 for pairs), cut into tiles_per_cta tiles of at most
 * tile_n rows.  With lm_pair = 1, lm_carry = 1 and lm_row_blocks > 1 the pairs form one team per row block and the
 * ranges are those of one team (lm_ctas / 2 / lm_row_blocks pairs each).  lm_rounds / lm_rounds_alone: rounds of tiles
 * the slowest CTA (pair) works through with and without decision-head CTAs in the launch (the tiles of a pair's own
 * range for teams; 0 when one row tile or block uses carried ranges).
 */
typedef struct {
    int32_t kernels;                 /* kernels per round: 3 or 4 */
    int32_t head_in_lm_launch;       /* decision-head CTAs ride in the LM-head launch */
    int32_t lm_pair, lm_carry, lm_tile_n, lm_ctas, lm_m_tiles, lm_n_tiles, lm_stages, lm_smem_bytes;
    int32_t lm_units_base, lm_units_rem, lm_tiles_per_cta, lm_rounds, lm_rounds_alone;
    int32_t head_carry, head_tile_n, head_ctas, head_m_tiles, head_n_tiles, head_k_splits, head_kb_per_split;
    int32_t head_stages, head_smem_bytes, head_units_base, head_units_rem, head_tiles_per_cta;
    int32_t lm_n_cols, lm_row_blocks;  /* CTA pairs: the window rows are cut into lm_row_blocks blocks of lm_n_cols rows (the N
                                          of the MMAs, a multiple of 16) */
    int32_t lm_parts;                /* LM-head partials per window row */
} wisv_plan_info;
int wisv_plan_host(const wisv_config* cfg, int32_t sm_count, int32_t max_smem_bytes, int32_t R, int32_t P,
                   wisv_plan_info* out);

/* Number of kernels this context has launched so far. */
int64_t wisv_launch_count(const wisv_ctx* ctx);

/*
 * Launch geometry the next wisv_verify would use for a batch with R window rows
 * and P head positions: vocabulary rows per LM-head tile, LM-head tiles, CTAs.
 * Any output pointer may be NULL.
 */
int wisv_plan(const wisv_ctx* ctx, int32_t R, int32_t P, int32_t* lm_tile_n, int32_t* lm_tiles,
              int32_t* lm_ctas, int32_t* head_tile_n, int32_t* head_tiles, int32_t* head_ctas);

/*
 * Kernels one wisv_verify round launches for such a batch: 4 (pack, LM head,
 * decision head, merge + scan), or 3 when decision-head CTAs ride in the LM-head
 * launch (every batch of at most 256 window rows; larger ones when the LM head
 * needs no additional round of tiles for it), or when P = 0.
 * Negative on bad arguments.
 */
int wisv_plan_kernels(const wisv_ctx* ctx, int32_t R, int32_t P);

/*
 * Link model of Section IV-A (host arithmetic only).  For one round with K_r draft
 * tokens of which m_r were requested, computes the payloads in bits - B_hid (Eq. 3),
 * B_fb (Eq. 4), B_u^FH (Eq. 5), B_u1^SH (Eq. 7), B_req (Eq. 8), B_u2^SH (Eq. 9) with
 * b_id = ceil(log2 V) - and the communication latencies T_comm^FH (Eq. 6) and
 * T_comm^SH (Eq. 10) in seconds.  m_r is the n_mismatch the verifier reports.
 * Rates are in bit/s, PER in [0, 1), the round-trip time in seconds.
 */
typedef struct {
    double rate_up_bps, rate_down_bps;   /* R_u(c), R_d(c) */
    double per_up, per_down;             /* PER_u(c), PER_d(c) */
    double rtt_s;                        /* tau_RTT */
    double hdr_up_bits, hdr_down_bits;   /* B_hdr,u, B_hdr,d */
    int32_t d_h, b_h;                    /* drafter hidden size and bits per element */
    int32_t b_pos;                       /* bits per position index */
} wisv_link;

typedef struct {
    int32_t b_id;
    double B_hid, B_fb, B_u_FH, B_u1_SH, B_req, B_u2_SH;
    double T_comm_FH, T_comm_SH;
} wisv_link_cost;

int wisv_link_cost_round(const wisv_link* link, int32_t V, int32_t K_r, int32_t m_r, wisv_link_cost* out);

/* Protocol rule reported with the testbed (Section VII): WISV_MODE_FH if rtt_s > 10 ms, else WISV_MODE_SH. */
int wisv_choose_protocol(double rtt_s);

/*
 * Bring-up / test hook: the raw fp32 logits L = bf16(target_hidden) . lm_head^T
 * of R rows (Algorithm 1, Verify), written to logits_out (dev fp32 [R, V]) by the
 * same TMA + tcgen05 main loop with a store epilogue.  target_hidden: dev fp32
 * [R, H].  Not used by wisv_verify, which never materialises logits.
 */
int wisv_debug_logits(wisv_ctx* ctx, const float* target_hidden, int32_t R, float* logits_out, void* cuda_stream);

/*
 * LM-head reduction without any allocation (the paper has no counterpart: this
 * entry point exists for deployment, not for the method).
 *
 * For callers that are not allowed to allocate device memory - a plug-in inside
 * a serving process whose framework has reserved the whole GPU for its own pool,
 * or a latency-critical loop that must stay out of the driver's allocator - and
 * therefore cannot use wisv_create.  Computes, for R <= WISV_STATIC_MAX_ROWS rows,
 *     argmax[r] = lowest v maximising  bf16(target_hidden[r]) . lm_head[v]
 *     lse[r]    = log sum_v exp(that logit)
 * with the same TMA + tcgen05 kernel as wisv_verify, keeping its scratch (the
 * bf16 copy of the rows and the per-tile partials) in a fixed array of about
 * 4 MiB that is part of the library image: every GPU that loads the library
 * holds it until the process exits.
 *
 * lm_head: dev bf16 [V, H] row-major, 16-byte aligned; target_hidden: dev fp32
 * [R, H], 16-byte aligned; argmax: dev int32 [R]; lse: dev fp32 [R].  Limits:
 * R <= WISV_STATIC_MAX_ROWS, 64 <= H <= WISV_STATIC_MAX_H with H % 8 == 0,
 * V <= WISV_STATIC_MAX_V; anything larger returns WISV_ECAPACITY and launches
 * nothing.  The call only enqueues work on `cuda_stream`; it calls no cudaMalloc,
 * cudaFree or other allocating routine.  The first call on each device looks up
 * the array's device address and raises the kernel's shared-memory limit; make
 * that first call outside any stream capture.  All calls on a device share the
 * array, which keeps the previous call's contents (each call rewrites what it
 * reads): calls that may overlap on the GPU race on it, so order them on one
 * stream or with events.  If a bounded wait inside the kernel gives up, every
 * argmax is -1 and every lse is NaN.
 */
#define WISV_STATIC_MAX_ROWS 128
#define WISV_STATIC_MAX_H    8192
#define WISV_STATIC_MAX_V    262144
int wisv_lm_head_reduce_static(const void* lm_head, int32_t V, int32_t H, const float* target_hidden, int32_t R,
                               int32_t* argmax, float* lse, void* cuda_stream);

/*
 * Test hook for the failure path (no counterpart in the paper): launches one small kernel that waits,
 * with the bounded wait all pipeline waits in this library use, on a barrier nothing arrives on.  After
 * limit_cycles SM clocks (<= 2e9) the wait gives up and sets bit 1 of the device error word, which
 * wisv_device_error then reports and clears; the context stays usable.
 */
int wisv_debug_wait_probe(wisv_ctx* ctx, uint64_t limit_cycles, void* cuda_stream);

/*
 * Test hooks standing in for a memory checker (no counterpart in the paper): fill every scratch buffer the
 * context owns - the bf16 copies of the hidden states, the LM-head and decision-head partials, the split-K
 * scratch, the row and position maps, the state kept between wisv_localize and wisv_decide (a pending localize
 * is dropped) - with NaN / out-of-range patterns, stream-ordered on `cuda_stream`.  The arrival counters and the
 * error word keep their values: zero between calls is their documented invariant, not stale data.
 * A following round must give the same results as without the call: every byte a round reads it has written
 * itself.  wisv_debug_poison_static does the same to the scratch array of wisv_lm_head_reduce_static.
 */
int wisv_debug_poison(wisv_ctx* ctx, void* cuda_stream);
int wisv_debug_poison_static(void* cuda_stream);

const char* wisv_strerror(int code);
int wisv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* WISV_H_ */
