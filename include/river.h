/*
 * river.h -- C ABI of the B200 (sm_100a) early-exit decode library.
 *
 * The library runs the hot path of River-LLM: the token-level early-exit autoregressive
 * decode step of a decoder-only transformer with a KV-Shared Exit River
 * (paper Section 4.1 "KV-Shared Exit Layer", Section 4.2 "Inference with Seamless Exit", Eq. 1).
 *
 * Conventions
 *   - Pointers marked [dev] are device pointers on the CUDA device that was current at
 *     river_init; pointers marked [host] are ordinary host memory.  All caller-owned: the
 *     library never frees them, and weights / KV pool / workspace must outlive the context.
 *   - Matrices are row-major [out, in] bf16.  A river (exit-layer) matrix is 4-bit weight-only:
 *     codes u8 [out, in/2] (low nibble = even input index), scale bf16 [out, in/group],
 *     zero bf16 [out, in/group]; the weight is (code - zero) * scale (Section 4.1, W4A16).
 *   - Layers are numbered 1..L; exit_layer = number of backbone blocks a token ran, in
 *     [entry_layer, L] (L = never left the backbone).
 *   - Every call returns RIVER_OK (0) or a negative RIVER_E_* code; river_last_error() gives
 *     a text.  No exceptions, no aborts, no device traps.
 *   - Work is enqueued on the stream given to river_init; device outputs are valid once the
 *     caller has synchronised that stream (the *_host variants synchronise themselves).
 *   - A context is not thread-safe.
 */
#ifndef RIVER_H_
#define RIVER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    RIVER_OK = 0,
    RIVER_E_BADARG = -1,  /* null pointer, out-of-range value */
    RIVER_E_SHAPE = -2,   /* unsupported model shape */
    RIVER_E_NOMEM = -3,   /* workspace or KV pool too small */
    RIVER_E_NOPAGE = -4,  /* no free KV page / sequence full */
    RIVER_E_BADSLOT = -5, /* slot out of range, duplicated in a batch, or empty */
    RIVER_E_DEVICE = -6,  /* a CUDA call failed, or a kernel flagged an error */
    RIVER_E_TIMEOUT = -7  /* a bounded device-side wait ran out */
};

enum { RIVER_EXIT_PER_TOKEN = 0, RIVER_EXIT_BATCH_MIN = 1 };

/* flags */
enum {
    RIVER_F_GRAPH = 1,    /* replay each decode step as a CUDA graph (captured on first use) */
    RIVER_F_NO_TC = 2,    /* diagnostic: every projection on the CUDA-core kernels, never the tcgen05 GEMMs */
    RIVER_F_NO_W4TC = 16, /* diagnostic: exit-layer rows of batches on the CUDA-core kernel instead of the dequantising
                             tcgen05 GEMM */
    RIVER_F_TMA_ATTN = 32, /* diagnostic: steps of 1-4 rows through the TMA-fed attention kernel too (default: the
                              small-step kernel) */
    RIVER_F_SERIAL_TC = 64 /* diagnostic: the two tcgen05 GEMMs of a projection (backbone rows, exit-layer rows) one
                              after the other (default: in flight together) */
};

typedef struct river_config {
    int32_t L, d, Hq, Hkv, dh, F, V; /* layers, hidden, query heads, KV heads, head dim, FFN dim, vocabulary */
    float rms_eps, rope_theta;
    int32_t entry_layer;       /* L_s of Section 4.2: the first block after which a token may exit (0..L-1) */
    int32_t group;             /* quantisation group along the input dimension (64) */
    int32_t page_size;         /* tokens per KV page (16) */
    int32_t max_seqs;          /* sequence slots */
    int32_t max_pages_per_seq; /* page-table width: max context = max_pages_per_seq * page_size */
    int32_t n_pages;           /* pages in the KV pool (shared by all layers: one page id addresses L layers) */
    int32_t max_batch;         /* max rows per decode step (<= 1024) */
    int32_t exit_mode;         /* RIVER_EXIT_PER_TOKEN: Eq. 1 per row; RIVER_EXIT_BATCH_MIN: Eq. 1 literally */
    uint32_t page_shuffle_seed;/* != 0: hand pages out in a seeded shuffled order */
    uint32_t flags;
    int32_t prefill_chunk;     /* prompt positions river_prefill runs per pass through the blocks (0 = max_batch, at most
                                  256): every pass streams the weights once, so larger chunks make prefill cheaper; the
                                  workspace grows with max(max_batch, prefill_chunk) */
    int32_t kv_strategy;       /* what happens in the blocks a token skips (Section 3; RIVER_KV_*): the method's KV-Shared
                                  Exit River, or one of the strategies it is compared with, on the same kernels */
} river_config;

/* river_config.kv_strategy.  In all of them the rows that have left still get their logits from the original LM head.
 *   RIVER_KV_RIVER             (Section 4.1) the 4-bit copy of every skipped block runs and writes the token's K/V into
 *                              the backbone's cache slot.
 *   RIVER_KV_STATE_PROPAGATION (Section 3) the hidden state at the exit is the input of every later block's K / V
 *                              projection (that block's norm and bf16 weights); no attention, no feed-forward there,
 *                              the hidden state reaches the LM head unchanged.  Needs no exit-layer weights.
 *   RIVER_KV_MONO_DECREASING   (Section 3) nothing runs in a skipped block, and a token leaves no later than the previous
 *                              token of its sequence did (whatever its score, and before a later forced exit), so no
 *                              cache entry it attends to is ever missing; the cap of a sequence starts at L, follows
 *                              every token (prefill: the prefill depth) and is reset by river_release.
 *   RIVER_KV_MASK              (Section 3) nothing runs in a skipped block either, and exits are free: attention in block
 *                              l sees only the cached positions whose token ran block l (and the row's own position).
 *                              Needs groups of at most four query heads per KV head. */
#define RIVER_KV_RIVER 0
#define RIVER_KV_STATE_PROPAGATION 1
#define RIVER_KV_MONO_DECREASING 2
#define RIVER_KV_MASK 3

typedef struct river_w4 {
    const void *codes, *scale, *zero; /* [dev] */
} river_w4;

typedef struct river_layer_weights {
    const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *wg, *wu, *wd; /* [dev] bf16 backbone block */
    river_w4 rq, rk, rv, ro, rg, ru, rd; /* [dev] its exit-layer copy; all NULL if the layer has none */
} river_layer_weights;

typedef struct river_weights {
    const void *embed, *lm_head, *final_norm; /* [dev] bf16 [V,d], [V,d], [d] */
    const river_layer_weights *layers;        /* [host] array of L entries (copied by river_init) */
} river_weights;

typedef struct river_stats_t {
    int64_t steps;               /* decode steps run */
    int64_t launches_total;      /* kernels launched by this context */
    int32_t launches_last_step;  /* kernels in the last decode step */
    int32_t batch_last;          /* rows of the last decode step */
    int32_t device_error;        /* sticky device error word (0 = none) */
    int32_t pages_in_use;
    double alg_bytes_last_step;  /* algorithmic HBM bytes of the last step (executed-layer weights + KV read/written
                                    + LM head + embedding rows + logits), from its actual exit pattern */
    double layers_executed_last; /* mean exit_layer / L over the rows of the last step */
    int64_t offload_fetches;     /* backbone blocks copied from host memory since river_init (river_offload) */
} river_stats_t;

typedef struct river_ctx river_ctx;

/* Bytes the caller must provide as workspace / KV pool for this configuration (0 on a bad config).
 * KV pool layout: bf16 [L][n_pages][2 (K,V)][Hkv][page_size][dh]; K is stored after RoPE.
 * One page id addresses the same slot in every layer, for backbone and exit layers alike
 * ("identical KV cache addressing", Section 4.1). */
size_t river_workspace_bytes(const river_config *cfg);
size_t river_kv_pool_bytes(const river_config *cfg);

/* Create a context.  kv_pool, workspace: [dev], 256-byte aligned.  cuda_stream: a cudaStream_t (NULL = default
 * stream).  Copies the config and the layer-pointer table; does not copy weights. */
int river_init(const river_config *cfg, const river_weights *w, void *kv_pool, size_t kv_pool_bytes,
               void *workspace, size_t workspace_bytes, void *cuda_stream, river_ctx **out);

/* Prefill with sequence-level exit (Section 4.2, "Prefill Phase"): every token of a prompt runs backbone blocks
 * 1..e and exit layers above e (e = L: the whole backbone), causal attention, and fills the KV cache of every
 * (token, layer).
 *   prefill_exit_layer  e in [entry_layer, L] for every prompt of the call, or -1: chosen per prompt by Eq. 1 with
 *       the prompt as the batch - the first block l in [max(entry_layer, 1), L-1] after which every position of the
 *       prompt has s > tau, else L (costs a second pass over the prompts whose depth comes out below L);
 *   tau     threshold of the -1 rule (unused otherwise);
 *   slots   [host] n_seqs empty sequence slots;   tok [dev] int32 token ids, all prompts concatenated;
 *   offsets [host] n_seqs+1 prefix offsets into tok;
 *   logits_last [dev] fp32 [n_seqs, V] or NULL;  next_tok [dev] int32 [n_seqs] or NULL (greedy, ties -> lowest id);
 *   depth_out [host] int32 [n_seqs] or NULL: the depth each prompt left the backbone at. */
int river_prefill(river_ctx *ctx, int n_seqs, const int32_t *slots, const int32_t *tok, const int32_t *offsets,
                  int prefill_exit_layer, float tau, float *logits_last, int32_t *next_tok, int32_t *depth_out);

/* One token-level early-exit decode step (Section 4.2, "Generation Phase"; Eq. 1).
 * Row b appends token tok[b] to sequence slots[b] (distinct slots).  After backbone block l with
 * entry_layer <= l < L the row's state-transition similarity s = cos(h^(l-1), h^(l)) is compared with tau[b]
 * (strict >, fp32); on exit the row finishes blocks l+1..L in the exit layers, which write their K/V into the
 * backbone's cache slots, and all rows end at the original LM head.
 *   slots [host] int32 [batch];  tok [dev] int32 [batch];  tau [dev] fp32 [batch];
 *   forced_exit [dev] int32 [batch] or NULL -- test hook: a value >= 0 replaces the score test by "leave after
 *       block forced_exit[b]" (L = never; 0 = exit layers from block 1 on, legal only with entry_layer 0);
 *   logits [dev] fp32 [batch, V] or NULL;  next_tok [dev] int32 [batch];  exit_layer [dev] int32 [batch];
 *   scores [dev] fp32 [batch, L] or NULL -- s of every backbone block the row ran, NaN elsewhere. */
int river_decode_step(river_ctx *ctx, int batch, const int32_t *slots, const int32_t *tok, const float *tau,
                      const int32_t *forced_exit, float *logits, int32_t *next_tok, int32_t *exit_layer,
                      float *scores);

/* The same step with HOST buffers: copies tok / tau / forced_exit to the device, runs the step, copies
 * next_tok / exit_layer (and logits, scores if not NULL) back, and synchronises the stream.
 *
 * Device-side errors (a token id or page id out of range, a forced exit layer out of range, a bounded wait that
 * ran out) are recorded in a sticky error word and the offending access is skipped or redirected; the kernels always
 * return.  This call, river_stats and river_selftest_wait_timeout read the word back and return RIVER_E_TIMEOUT for
 * a wait that ran out, RIVER_E_DEVICE otherwise; river_decode_step and river_prefill (which do not synchronise) report
 * it at the next such call.  Once the host has seen the word the context refuses further steps with the same code
 * until river_clear_device_error. */
int river_decode_step_host(river_ctx *ctx, int batch, const int32_t *slots, const int32_t *tok, const float *tau,
                           const int32_t *forced_exit, float *logits, int32_t *next_tok, int32_t *exit_layer,
                           float *scores);

/* Copy n cached positions of one sequence and layer (1-based) out / in: bf16 [n, Hkv, dh], [dev].
 * river_write_kv is a test hook; it may extend the sequence (allocating pages) up to pos0 + n. */
int river_read_kv(river_ctx *ctx, int slot, int layer, int pos0, int n, void *k_out, void *v_out);
int river_write_kv(river_ctx *ctx, int slot, int layer, int pos0, int n, const void *k_in, const void *v_in);

/* Free-running greedy generation (Section 4.2, "Generation Phase"): n_steps decode steps in which every row's next
 * token is fed back on the device - step t reads the tokens step t-1 wrote - with no host synchronisation in between
 * (the host only enqueues; with RIVER_F_GRAPH every step is one graph launch).  Thresholds are the same for all steps.
 *   tok0 [dev] int32 [batch] first input tokens;  tau [dev] fp32 [batch];
 *   out_tok [dev] int32 [n_steps, batch] generated tokens;  out_exit [dev] int32 [n_steps, batch] or NULL.
 * Fails like river_decode_step (e.g. RIVER_E_NOPAGE when a sequence fills up); steps enqueued before stay valid. */
int river_generate(river_ctx *ctx, int batch, const int32_t *slots, const int32_t *tok0, const float *tau, int n_steps,
                   int32_t *out_tok, int32_t *out_exit);

/* Backbone offloading (Section 4.2, "Backbone Offloading"): the bf16 matrices of backbone blocks
 * first_offloaded_layer..L live in PINNED HOST memory and are copied into device memory only for a step whose rows are
 * still in the backbone when they reach such a block (the exit layers, which carry most tokens, stay resident).
 *   host_layers [host] array of L entries; in entries >= first_offloaded_layer wq, wk, wv, wo, wg, wu, wd are pinned
 *       host pointers to the bf16 matrices (norm gains and exit-layer weights stay as given to river_init);
 *   device side: at river_init the offloaded blocks must have been given device matrices that alternate between TWO
 *       staging slots (blocks l and l + 2 the same seven pointers): a block is staged while the previous one runs.
 * With offloading on, a step synchronises with the host once per offloaded block (the host must see whether any row is
 * still in the backbone before it copies 2 P bytes), graph replay is off and the exit score runs as a kernel of its
 * own.  first_offloaded_layer = 0 turns it off.  river_stats.offload_fetches counts the block copies.  Not with
 * RIVER_KV_STATE_PROPAGATION (which needs the backbone K / V matrices of every skipped block). */
int river_offload(river_ctx *ctx, int first_offloaded_layer, const river_layer_weights *host_layers);

/* Which blocks are sparsely used (Section 4.2: the blocks to offload follow from where the tokens leave).
 * river_exit_histogram: counts [host] L + 1 entries, counts[e] = decoded tokens so far (decode steps and river_generate,
 *   not prompts) that ran e backbone blocks; reset != 0 clears the counters afterwards.  Synchronises the stream.
 * river_suggest_offload: the first block l >= 2 that at most max_deep_fraction of the decoded tokens have reached (exit
 *   layer >= l) - the value to hand to river_offload - or 0 when no block qualifies or nothing has been decoded yet;
 *   negative on error. */
int river_exit_histogram(river_ctx *ctx, int64_t *counts, int reset);
int river_suggest_offload(river_ctx *ctx, double max_deep_fraction);

/* Two stages of the path on their own, for kernel-level tests and the exit-aware attention microbenchmark.  Both take
 * a compacted list of rows: row i belongs to sequence slots[i] ([host], distinct, non-empty) and sits at that
 * sequence's LAST cached position p_i; both enqueue on the context's stream like a decode step.
 *
 * river_attention - step a3, paged GQA decode attention: out[i] = softmax(q[i] K^T / sqrt(dh)) V over the cached
 *   positions 0..p_i of block `layer` (1-based);  q, out [dev] fp32 [n_rows, Hq*dh].
 * river_project_kv - step a2: x = RMSNorm(h[i]) with the block's attention-norm gain, q, k, v = W x on the block's
 *   bf16 weights (use_exit_layer = 0) or on its 4-bit exit-layer copy (1: the K/V generation of a bypassed block,
 *   Section 4.1), rotary embedding at position p_i, and k, v stored (bf16) over the cache entry of position p_i - the
 *   slot both weight sets share;  h [dev] fp32 [n_rows, d];  q_out [dev] fp32 [n_rows, Hq*dh] or NULL. */
int river_attention(river_ctx *ctx, int layer, int n_rows, const int32_t *slots, const float *q, float *out);
int river_project_kv(river_ctx *ctx, int layer, int use_exit_layer, int n_rows, const int32_t *slots, const float *h,
                     float *q_out);

/* Row lists of the last decode step, [host] out: act_idx / riv_idx int32 [(L+1), batch] (entry l-1: rows in the
 * backbone / in the exit layers entering block l, ascending, -1 padded; entry L: at the LM head) and their counts
 * int32 [L+1].  Synchronises the stream. */
int river_last_lists(river_ctx *ctx, int32_t *act_idx, int32_t *n_act, int32_t *riv_idx, int32_t *n_riv);

/* Per-kernel timing.  river_profile(ctx, 1) zeroes the counters and makes every later step record a CUDA event
 * before and after each kernel launch on the context's stream and synchronise at the end of the step (the step gets
 * slower: use it for a separate measuring pass, never inside a timed region); river_profile(ctx, 0) turns it off.
 * river_profile_read fills out[0..*n_out) ([host], cap entries) with one record per kernel of the step sequence:
 * its launches, summed device time, and summed algorithmic HBM bytes (weights of the weight sets that actually ran,
 * KV bytes read / written, LM head, logits). */
typedef struct river_kernel_time {
    char name[24];
    int64_t launches;
    double ms_total;
    double alg_bytes_total;
} river_kernel_time;
int river_profile(river_ctx *ctx, int enable);
int river_profile_read(river_ctx *ctx, river_kernel_time *out, int cap, int *n_out);

/* Greedy token selection over logits the caller already holds, without allocating anything.
 * (The paper has no counterpart: this is a utility for callers of the library.)
 * For callers that cannot allocate at the point of the call and have no context workspace to lend: a sampling hook
 * inside a serving loop whose device memory was all handed out at start-up, or a latency-critical loop where an
 * allocation would serialise the device.  The scratch (per-CTA partial maxima, per-row arrival counters, 66 KB)
 * is a fixed array in the library's device image; every GPU that loads the library holds it until process exit.
 *   logits [dev] fp32 [n_rows, V];  next_tok [dev] int32 [n_rows]: index of the row maximum, ties -> lowest id
 *   (the rule river_decode_step uses; NaNs never win, and a row that holds nothing but NaNs yields token 0, as in
 *   river_decode_step);  cuda_stream: a cudaStream_t (NULL = default stream); the call is
 *   asynchronous on it.
 * n_rows > RIVER_NOALLOC_MAX_ROWS returns RIVER_E_NOMEM (split the batch); null pointers, n_rows <= 0, V <= 0 or
 * V > INT_MAX - 128 return RIVER_E_BADARG.  Every call clears the per-row arrival counters with a memset on the
 * stream before its launch.
 * The first call on a device looks up the scratch array's device address (with that device current); make that
 * first call before any stream capture.  Calls no cudaMalloc / cudaFree or allocating library routine.  All calls
 * on a device share the one array: two calls that overlap on the GPU (different streams) race; issue them on one
 * stream or order them yourself. */
#define RIVER_NOALLOC_MAX_ROWS 64
int river_argmax_noalloc(const float *logits, int n_rows, int V, int32_t *next_tok, void *cuda_stream);

/* Reset the sticky device error word (synchronises the stream). */
int river_clear_device_error(river_ctx *ctx);

/* Self-test of the bounded device-side waits: runs the library's mbarrier wait on a barrier nobody completes, with a
 * poll limit of poll_limit (1 .. 2^20).  The kernel gives up after that many polls, records the time-out and returns;
 * the call synchronises and returns RIVER_E_TIMEOUT (the expected outcome), leaving the error word set. */
int river_selftest_wait_timeout(river_ctx *ctx, int poll_limit);

/* The exit layers' weights from the backbone's (Section 4.1: an exit layer is a copy of its backbone block whose
 * Attention and FFN matrices go through a training-free 4-bit weight-only quantisation with a refined zero-point).
 *   w [dev] bf16 row-major [out, in], 16-byte aligned;  group in {32, 64, 128} dividing `in`;
 *   refine_iters: rounds of the half-quadratic zero-point refinement (0 = plain min/max round-to-nearest grid; 20 is
 *       the published default);
 *   codes [dev] u8 [out, in/2] (low nibble = even input), scale / zero [dev] bf16 [out, in/group]: the layout
 *       river_init takes.  No context needed; asynchronous on cuda_stream.  Returns RIVER_E_SHAPE for an unsupported
 *       group, RIVER_E_BADARG for null / misaligned pointers or non-positive sizes. */
int river_quantize_w4(const void *w, int out, int in, int group, int refine_iters, void *codes, void *scale, void *zero,
                      void *cuda_stream);

int river_seq_len(const river_ctx *ctx, int slot);       /* tokens cached in the slot, or RIVER_E_BADSLOT */
int river_release(river_ctx *ctx, int slot);             /* free the slot's pages */
int river_stats(river_ctx *ctx, river_stats_t *host_out); /* synchronises the stream; fills host_out even when it
                                                             returns a device-error code */
void river_destroy(river_ctx *ctx);
const char *river_last_error(const river_ctx *ctx);      /* ctx may be NULL: error of the last failed river_init */

#ifdef __cplusplus
}
#endif
#endif /* RIVER_H_ */
