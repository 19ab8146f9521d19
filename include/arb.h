/*
 * arb.h -- C ABI of the Arbitrage hot path on one B200 (sm_100a).
 *
 * Three operations make up the data-parallel part of step-level speculative generation with an
 * advantage-aware router (Algorithm 1 of the paper):
 *
 *   arb_attn      grouped-query attention of a batch of query chunks against per-sequence paged KV
 *                 caches.  q_len = 1 is one autoregressive decode token of a draft or target step
 *                 (Section 3.1: z_i ~ q(z_i | x, z_<i)); q_len = step length is the router's single
 *                 forward over a completed draft step (Section 4.2, "one forward pass per step").
 *   arb_route     the router decision (Section 4.2; Figure 1; Algorithm 1, "Routing decision"):
 *                 y_hat = sigmoid(hidden_last . w + b); escalate to the target iff y_hat > tau,
 *                 accept the draft step iff y_hat <= tau.
 *   arb_rollback  the escalation branch of Algorithm 1: the target regenerates the step from the
 *                 same prefix x, so a cache that absorbed the rejected draft step drops it by
 *                 resetting its length; no KV bytes move.
 *
 * Around them: arb_kv_append (the cache write of a step's new tokens), arb_decode_step (one decode token:
 * cache write, attention and length update in one launch), arb_policy (the escalation rules
 * the paper compares on PRM scores: RSD, oracle threshold / arg max, budgeted oracle, with the wasted
 * target calls) and arb_route_classes (the C-way heads of the router ablation).
 *
 * Conventions shared by every call
 *   - Pointers are DEVICE pointers unless the argument says "host".  The caller owns every tensor;
 *     the library owns only the arb_ctx (split-KV partials, arrival counters, a status word and
 *     staging buffers), allocated by arb_create / grown by the *_host calls, never by arb_attn,
 *     arb_route or arb_rollback.
 *   - Calls enqueue work on `stream` and return; they do not synchronise (arb_poll_status and the
 *     *_host calls do).  One arb_ctx must not be used from two streams at the same time: calls
 *     share its workspace.
 *   - Host-checkable problems (null pointer, bad dimension, pointer not 16-byte aligned,
 *     unsupported head_dim / group size, workspace too small) return a non-zero arb_status and
 *     launch nothing.  Problems only the device can see (page id out of range, seq_len < q_len,
 *     seq_len beyond the block table, rollback below zero) set a bit in a device status word, the
 *     offending sequence is skipped (its output rows are zero-filled) or clamped, and the kernel
 *     carries on: nothing traps.  Read the bits with arb_poll_status.
 *   - Layouts are dense row-major with the last index fastest.
 */
#ifndef ARB_H_
#define ARB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ARB_OK = 0,
    ARB_ERR_INVALID_ARG = 1,   /* null pointer, non-positive dimension, misaligned pointer */
    ARB_ERR_UNSUPPORTED = 2,   /* head_dim, group size, page size or dtype outside the built set */
    ARB_ERR_WORKSPACE = 3,     /* the ctx workspace is smaller than arb_attn_workspace_bytes() */
    ARB_ERR_CUDA = 4,          /* a CUDA runtime call failed (allocation, launch, copy) */
    ARB_ERR_DEVICE_STATUS = 5, /* arb_poll_status: the device status word is non-zero */
    ARB_ERR_STATIC_LIMIT = 6   /* arb_attn_decode_static: the call needs more than the built-in scratch */
} arb_status;

typedef enum { ARB_F32 = 0, ARB_BF16 = 1 } arb_dtype;

/* bits of the device status word (arb_poll_status) */
enum {
    ARB_DEV_BAD_SEQ_LEN = 1u,        /* q_len > 0 and (seq_len < q_len or seq_len > max_pages*page) */
    ARB_DEV_BAD_PAGE = 2u,           /* block_table entry outside [0, num_pages) */
    ARB_DEV_ROLLBACK_UNDERFLOW = 4u, /* step_len < 0 or step_len > seq_len */
    ARB_DEV_WAIT_TIMEOUT = 8u,       /* a bounded wait on an asynchronous copy or MMA gave up */
    ARB_DEV_CHECK_FAILED = 16u       /* bounds-check build only: an index the device derived was out of range; the access was skipped */
};

/* escalation policies of arb_policy */
typedef enum {
    ARB_POLICY_RSD = 0,              /* escalate iff s_d <= tau (the step is accepted iff s_d > tau) */
    ARB_POLICY_ORACLE_THRESHOLD = 1, /* escalate iff s_t - s_d > tau */
    ARB_POLICY_ORACLE_ARGMAX = 2,    /* escalate iff s_t > s_d */
    ARB_POLICY_ORACLE_BUDGET = 3     /* escalate the min(budget, #{s_t - s_d > 0}) largest positive advantages */
} arb_policy_kind;

/* what a policy did, accumulated on the device by arb_policy */
typedef struct {
    uint32_t escalated; /* steps sent to the target */
    uint32_t wasted;    /* of those, steps with s_t <= s_d: the target call bought nothing */
    double realised;    /* sum over steps of the score of the step that was kept: a ? s_t : s_d */
    double gain;        /* sum over escalated steps of s_t - s_d */
} arb_policy_stats;

/* C-way router heads of arb_route_classes */
typedef enum { ARB_HEAD_SOFTMAX = 0, ARB_HEAD_ORDINAL = 1 } arb_head_kind;
#define ARB_MAX_CLASSES 16

typedef struct CUstream_st *arb_stream_t; /* same type as cudaStream_t */
typedef struct arb_ctx arb_ctx;

/*
 * Shape of one arb_attn call.  Notation: B = batch, Hq = num_q_heads, Hkv = num_kv_heads,
 * g = Hq / Hkv (query heads h*g .. h*g+g-1 share KV head h), D = head_dim, P = page_size.
 */
typedef struct {
    int32_t dtype;             /* arb_dtype of q, k_pages, v_pages and out; accumulation is fp32 */
    int32_t batch;             /* 1 .. 1024 */
    int32_t num_q_heads;       /* multiple of num_kv_heads, g <= 8 */
    int32_t num_kv_heads;
    int32_t head_dim;          /* 64 or 128 */
    int32_t page_size;         /* 16 */
    int32_t num_pages;         /* pages in the pool that k_pages / v_pages point to */
    int32_t max_pages_per_seq; /* row length of block_table */
    int32_t total_q;           /* sum of q_lens (rows of q and out); the host knows it */
    int32_t max_q_len;         /* max of q_lens; 1 selects the decode kernel alone */
    float softmax_scale;       /* <= 0 selects 1/sqrt(head_dim) */
    uint32_t flags;            /* ARB_ATTN_* bits, 0 for none */
} arb_attn_params;

/*
 * arb_attn_params.flags.
 * ARB_ATTN_OVERLAP_PREVIOUS: the caller states that no input of this call (q, k_pages, v_pages,
 * block_table, seq_lens, q_lens) is written by the kernel that precedes it on the stream.  The
 * decode kernel is then launched as a programmatic dependent of that kernel: it may start streaming
 * KV while its predecessor is still finishing, and waits for the predecessor's completion only
 * before its first write to `out` (and to the workspace, unless the workspace set it uses is known
 * to be free).  A flagged call is taken to be one of a back-to-back series: a small one spreads
 * over half as many CTAs as an unflagged call, so that more calls of the series are in flight at
 * once; that changes where its sequences are split, so results agree with the unflagged call
 * within rounding (same tolerances), not bit for bit.  The same flagged call always gives the same
 * bits.  Typical use: independent decode calls queued behind one another whose q and KV cache are
 * ready.  Do not set it when the preceding kernel produces q, appends K/V or changes seq_lens.
 * ARB_ATTN_NO_TENSOR_CORES: run decode and step chunks on the CUDA-core kernels even where the
 * tensor-core kernels apply (bf16, head_dim 128).  Same results within the stated tolerances; for
 * comparison runs and for keeping both paths under test.
 */
enum { ARB_ATTN_OVERLAP_PREVIOUS = 1u, ARB_ATTN_NO_TENSOR_CORES = 2u };

/*
 * Create a context on `device`.  workspace_bytes = 0 picks a default that covers every shape the
 * library supports with batch * num_kv_heads <= 8192.  Allocates device memory; call it outside
 * any stream capture.  Errors: ARB_ERR_INVALID_ARG, ARB_ERR_CUDA.
 */
arb_status arb_create(arb_ctx **ctx, int device, size_t workspace_bytes);
arb_status arb_destroy(arb_ctx *ctx);

/* Workspace an arb_attn call with these parameters needs (0 if the parameters are invalid). */
size_t arb_attn_workspace_bytes(const arb_attn_params *params);

/*
 * Paged grouped-query attention (the forward passes of Algorithm 1's "Sample draft step",
 * "Sample target step" and "Routing decision"; Section 3.1 for the token-by-token step).
 *
 *   q, out       [total_q, Hq, D]; rows packed by sequence: sequence b owns q_lens[b] consecutive
 *                rows, in batch order.  out has q's dtype.
 *   k_pages,
 *   v_pages      [num_pages, Hkv, P, D]: one (page, kv head) tile is P*D contiguous elements.
 *   block_table  int32 [B, max_pages_per_seq]; entry [b][j] is the pool page holding tokens
 *                j*P .. j*P+P-1 of sequence b.  Entries at or beyond ceil(seq_len / P) are never
 *                read.
 *   seq_lens     int32 [B]: tokens in the cache INCLUDING the q_lens[b] new ones, whose K/V the
 *                caller has already written.
 *   q_lens       int32 [B]: 0 (idle slot, no rows), 1 (decode) or the step length.
 *
 * Query token i (0-based) of sequence b sits at position pos = seq_lens[b] - q_lens[b] + i and
 * attends keys 0 .. pos inclusive:  out = sum_j softmax_j(scale * q . k_j) v_j.  Slots beyond
 * pos are never used, not even multiplied by zero, so stale or non-finite values there (a rolled
 * back step) cannot reach the output.
 *
 * Asynchronous on `stream`.  Errors: ARB_ERR_INVALID_ARG, ARB_ERR_UNSUPPORTED, ARB_ERR_WORKSPACE,
 * ARB_ERR_CUDA; device-side: ARB_DEV_BAD_SEQ_LEN (rows zero-filled), ARB_DEV_BAD_PAGE (the bad
 * page is skipped or replaced by page 0; that sequence's rows are unspecified but finite-safe).
 */
arb_status arb_attn(arb_ctx *ctx, const arb_attn_params *params, const void *q,
                    const void *k_pages, const void *v_pages, const int32_t *block_table,
                    const int32_t *seq_lens, const int32_t *q_lens, void *out,
                    arb_stream_t stream);

/*
 * arb_attn for callers whose per-step tensors live in HOST memory (pinned memory makes the copies
 * asynchronous).  q_host, block_table_host, seq_lens_host, q_lens_host and out_host are host
 * pointers with the shapes above; k_pages and v_pages stay DEVICE pointers (the cache is resident
 * state, not a per-step input).  Copies the inputs to staging buffers owned by ctx (grown here if
 * too small -- the one call besides arb_create that may allocate), runs arb_attn, copies out back
 * (a page-locked out_host is written by the kernels directly instead) and synchronises `stream`
 * before returning.
 */
arb_status arb_attn_host(arb_ctx *ctx, const arb_attn_params *params, const void *q_host,
                         const void *k_pages, const void *v_pages,
                         const int32_t *block_table_host, const int32_t *seq_lens_host,
                         const int32_t *q_lens_host, void *out_host, arb_stream_t stream);

/*
 * arb_attn_host in two halves, for callers that issue several host-side calls before they need a
 * result (the layers of one decode token, the caches of one round of Algorithm 1).
 *
 * arb_attn_host_begin takes the arguments of arb_attn_host.  Before it returns it has copied the
 * four input arrays into staging owned by ctx (the caller may overwrite them at once) and has
 * enqueued: the inputs' copy to the device on a copy stream of ctx, the arb_attn kernels on
 * `stream` (in call order, so cache updates enqueued on `stream` between two calls are seen by the
 * later one), and the copy of the result into out_host on a second copy stream of ctx.  out_host
 * (page-locked memory keeps that copy asynchronous) must not be read before arb_attn_host_wait has
 * returned ARB_OK; synchronising `stream` alone does not cover the copy back.  Up to 32 calls are in
 * flight per ctx; a further call first waits for the oldest.  Staging grows here when a call needs
 * more (allocation, as in arb_attn_host).  Not for a stream that is being captured into a graph.
 * A call flagged ARB_ATTN_OVERLAP_PREVIOUS whose out_host is page-locked uses no copies at all: its
 * kernels read the staged inputs and write out_host in place over the bus (the faster way for a
 * series of small calls).  `stream` must stay alive until arb_attn_host_wait has returned.
 *
 * arb_attn_host_wait blocks until every call begun on ctx has delivered its result.
 * Errors: as arb_attn_host; after an error nothing of the failed call is left in flight.
 */
arb_status arb_attn_host_begin(arb_ctx *ctx, const arb_attn_params *params, const void *q_host,
                               const void *k_pages, const void *v_pages,
                               const int32_t *block_table_host, const int32_t *seq_lens_host,
                               const int32_t *q_lens_host, void *out_host, arb_stream_t stream);
arb_status arb_attn_host_wait(arb_ctx *ctx);

/*
 * Decode attention (q_len = 1 for every sequence) for callers that must not allocate.
 *
 * The paper has no counterpart to this call; it exists for the way the library gets embedded.
 * Some hosts cannot afford a cudaMalloc at any point after start-up: a serving process that has
 * already given every free byte of device memory to its KV-cache pool, or a plug-in that runs in
 * the middle of another framework's operator, where an allocation would stall the whole device
 * and may fail outright.  arb_create allocates, so such callers cannot hold an arb_ctx.  This
 * entry point needs none: the split-KV partials, the arrival counters and the status word live in
 * a fixed 4 MiB array that is part of the library image (every GPU that loads the library carries
 * it until the process exits).  It calls no cudaMalloc, cudaFree or any other allocating routine.
 *
 * Arguments are those of arb_attn with params->max_q_len == 1 and params->total_q equal to the
 * number of sequences with q_lens[b] == 1 (other q_lens must be 0).  device_status is an optional
 * caller-owned device word: device-side problems (ARB_DEV_* bits) are OR-ed into it; pass NULL to
 * ignore them.  Results equal arb_attn's.
 *
 * Limits and sharing.  The call is refused with ARB_ERR_STATIC_LIMIT, and nothing is launched,
 * when batch * num_kv_heads > 1024 or when the call's scratch,
 *     (batch * num_kv_heads + 2 * SM count) * (g * head_dim + 2 * roundup4(g)) * 4 + 4352 bytes,
 * exceeds the 4 MiB array (the draft- and target-shaped decode workloads need under 1 MiB).  All
 * calls in the process that target the same GPU share the one array and it keeps whatever the last call left:
 * the counters and the internal status word are cleared on `stream` at the start of every call,
 * but two calls that overlap on the GPU (different streams, or a programmatic dependent of each
 * other) race on it and corrupt each other's results; ARB_ATTN_OVERLAP_PREVIOUS is therefore
 * rejected with ARB_ERR_INVALID_ARG.  The current device must be the one the pointers live on.
 * The first call on a device looks up the array's device address and sets the kernel's
 * shared-memory attribute; make that first call before any stream capture begins.  That set-up is
 * serialised inside the library, so first calls from several host threads are safe.  With
 * device_status == NULL the ARB_DEV_* bits of a call (a wait that timed out included) go to a word inside
 * the array that no API reads and that the next call clears: pass a word if you need to see them.
 */
arb_status arb_attn_decode_static(const arb_attn_params *params, const void *q, const void *k_pages,
                                  const void *v_pages, const int32_t *block_table,
                                  const int32_t *seq_lens, const int32_t *q_lens, void *out,
                                  uint32_t *device_status /* nullable */, arb_stream_t stream);

/*
 * Router head and threshold decision (Section 4.2, Figure 1, Algorithm 1 "Routing decision": the score
 * estimates the probability that escalating improves the step; the draft step is rejected iff
 * y_hat > tau and accepted iff y_hat <= tau; Section 4.2 "Training": the head reads the hidden state of the
 * step's final token).  A two-class softmax head (accept = 0,
 * escalate = 1) is the same function with w = w1 - w0 and b = b1 - b0.
 *
 *   hidden     [n_steps, hidden_dim]; row i is the final-layer hidden state of the last token of
 *              step i.  hidden_dim must be a multiple of 8.
 *   w          [hidden_dim], same dtype as hidden.
 *   b, tau     host scalars.
 *   scores     fp32 [n_steps]: sigmoid(hidden_i . w + b), accumulated in fp32.
 *   decisions  uint8 [n_steps]: 1 = escalate (score > tau), 0 = accept (score <= tau; a tie
 *              accepts).
 */
arb_status arb_route(arb_ctx *ctx, int32_t dtype, int32_t n_steps, int32_t hidden_dim,
                     const void *hidden, const void *w, float b, float tau, float *scores,
                     uint8_t *decisions, arb_stream_t stream);

/*
 * Step rollback (Algorithm 1, escalation branch: the step is regenerated from the same prefix).
 *   seq_lens[i] -= step_lens[i]  for every i with decisions == NULL or decisions[i] != 0.
 * Block-table entries and page contents are left as they are; later attention ignores the stale
 * slots and later appends overwrite them.  step_lens[i] < 0 leaves seq_lens[i] unchanged and
 * step_lens[i] > seq_lens[i] clamps it to 0; both raise ARB_DEV_ROLLBACK_UNDERFLOW.
 */
arb_status arb_rollback(arb_ctx *ctx, int32_t batch, int32_t *seq_lens, const int32_t *step_lens,
                        const uint8_t *decisions /* nullable */, arb_stream_t stream);

/*
 * Escalation decisions from PRM scores, for the policies the paper compares (Section 3.1: the RSD
 * baseline accepts a draft step iff s_d > tau; Section 4.1: the oracle keeps the higher-scoring of the
 * draft and target step, or escalates iff the advantage Delta = s_t - s_d exceeds tau; Appendix B,
 * Theorem: under a budget of B escalations the best policy takes the largest positive advantages), and
 * what each costs (Section 3.2: a target call is wasted when s_t <= s_d; Section 4.1: the realised
 * score is S(a) = s_d + a Delta).
 *
 *   s_d, s_t   fp32 [n_steps]: PRM score of the draft step and of the target's counterpart.  s_t may be
 *              NULL for ARB_POLICY_RSD when stats is NULL.  Scores are finite.
 *   tau        threshold (RSD, oracle threshold); budget: escalations allowed (budgeted oracle,
 *              n_steps <= 65536).
 *   decisions  uint8 [n_steps]: 1 = escalate to the target, 0 = keep the draft step.  Ties: RSD escalates
 *              at s_d == tau; the oracle rules keep the draft at Delta == tau / s_t == s_d; among equal
 *              advantages the budgeted rule takes the lower index first.
 *   stats      nullable; zeroed on `stream`, then filled by the kernel (sums in fp64).
 * Delta and every comparison are taken in fp32 (IEEE subtraction, no flush to zero).
 * Errors: ARB_ERR_INVALID_ARG (null pointer, unknown kind, s_t missing), ARB_ERR_UNSUPPORTED (budgeted
 * rule beyond 65536 steps).
 */
arb_status arb_policy(arb_ctx *ctx, int32_t kind, int32_t n_steps, const float *s_d, const float *s_t, float tau,
                      int32_t budget, uint8_t *decisions, arb_policy_stats *stats /* nullable */,
                      arb_stream_t stream);

/*
 * C-way router heads (Section 6.1, "Label Granularity" and "Classification vs. Regression": heads over
 * 2, 4 or 10 ordered classes of the advantage, and a 4-level ordinal head).  The paper does not say how
 * a C-way head becomes one routing score; here it is the expected class level scaled to [0, 1],
 * score = sum_c p_c * c / (C - 1), and the step escalates iff score > tau (a tie accepts).  For C = 2
 * that is arb_route with w = w1 - w0, b = b1 - b0.
 *
 *   mode       ARB_HEAD_SOFTMAX: logits l_c = hidden . w[c] + b[c], p = softmax(l); w is [C, hidden_dim].
 *              ARB_HEAD_ORDINAL: one logit z = hidden . w[0] + b[0] and cut points b[1] <= ... <= b[C-1]:
 *              P(y >= k) = sigmoid(z - b[k]), p_k = P(y >= k) - P(y >= k + 1); w is [hidden_dim].
 *   hidden     [n_steps, hidden_dim], hidden_dim a multiple of 8; w has hidden's dtype.
 *   b_host     HOST pointer to n_classes floats (2 <= n_classes <= ARB_MAX_CLASSES).
 *   probs      nullable, fp32 [n_steps, n_classes]; scores fp32 [n_steps]; decisions uint8 [n_steps].
 */
arb_status arb_route_classes(arb_ctx *ctx, int32_t dtype, int32_t mode, int32_t n_steps, int32_t hidden_dim,
                             int32_t n_classes, const void *hidden, const void *w, const float *b_host, float tau,
                             float *probs /* nullable */, float *scores, uint8_t *decisions, arb_stream_t stream);

/*
 * KV append: writes the keys and values of each sequence's new tokens into the paged cache behind the
 * tokens it already holds (the cache write that every "Sample draft step" / "Sample target step" of
 * Algorithm 1 implies before the next arb_attn call may attend to them; after a rollback the same slots
 * are overwritten by the regenerated step).
 *
 *   params     dtype, batch, num_kv_heads, head_dim, page_size, num_pages and max_pages_per_seq are
 *              used; the other fields are ignored.
 *   k_new,
 *   v_new      [total_new, Hkv, D], packed by sequence in batch order: sequence b owns new_lens[b] rows.
 *   seq_lens   int32 [B]: tokens held BEFORE the call.  Token j of sequence b goes to position
 *              seq_lens[b] + j, i.e. page block_table[b][pos / P], slot pos % P.  With update_lens != 0
 *              seq_lens[b] becomes seq_lens[b] + new_lens[b] (written by the CTA of the append kernel that
 *              finishes last, once every CTA has read the old lengths), which is the
 *              value arb_attn expects when it is called with q_lens = new_lens.
 *   new_lens   int32 [B], >= 0; total_new >= their sum (rows beyond the sum are ignored).
 * A sequence whose new tokens do not fit under its block-table row, or whose target pages lie outside
 * the pool, is left untouched (pools and length) and raises ARB_DEV_BAD_SEQ_LEN / ARB_DEV_BAD_PAGE; a
 * negative new_len raises ARB_DEV_BAD_SEQ_LEN.  Values are copied bit for bit.
 */
arb_status arb_kv_append(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                         const void *v_new, const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens,
                         int32_t update_lens, void *k_pages, void *v_pages, arb_stream_t stream);

/*
 * One decode token in one launch: arb_kv_append of the token's K/V rows, arb_attn with q_len = 1 over the
 * cache that now holds them, and the length update, fused (Algorithm 1, "Sample draft step" / "Sample target
 * step": a step is generated token by token, z_i ~ q(z_i | x, z_<i), Section 3.1; every token of every step
 * pays this call once per layer, and each call reads what the one before it wrote, so its latency -- not its
 * bytes -- is what the loop sees).
 *
 *   params     as for arb_attn with max_q_len == 1; total_q >= the number of sequences with q_lens[b] == 1
 *              (the rows of q, k_new, v_new and out; rows beyond that number are ignored), total_q <= batch.
 *              ARB_ATTN_OVERLAP_PREVIOUS is refused (ARB_ERR_INVALID_ARG): the call writes the cache it reads.
 *   q, out     [total_q, Hq, D], rows in batch order of the sequences that take part.
 *   k_new,
 *   v_new      [total_q, Hkv, D], same row order: the token's key and value rows.
 *   k_pages,
 *   v_pages    the pools, written (one row per sequence and kv head) and read.
 *   seq_lens   int32 [B]: tokens held BEFORE the call.  The token of sequence b goes to position seq_lens[b],
 *              attends keys 0 .. seq_lens[b] inclusive (itself included), and seq_lens[b] becomes seq_lens[b] + 1.
 *   q_lens     int32 [B]: 1 = the sequence takes part, 0 = idle slot (nothing read, written or advanced).
 * The result equals arb_kv_append(new_lens = q_lens, update_lens = 1) followed by arb_attn(max_q_len = 1),
 * within the tolerances of arb_attn.  A sequence whose token does not fit under its block-table row is left
 * untouched (pools, length), its out row is zero-filled and ARB_DEV_BAD_SEQ_LEN is raised; a sequence whose
 * new row would land on a page outside the pool keeps its length and pools, raises ARB_DEV_BAD_PAGE, and its
 * out row is unspecified but finite-safe (as for arb_attn).  q_lens other than 0 and 1 count as 0 with the
 * status bit.  bf16 / head_dim 128 / g <= 8 run as one kernel; other shapes as the two calls above.
 * Asynchronous on `stream`; launched as a programmatic dependent of the kernel before it (it touches no
 * memory before that kernel has completed, so this is safe behind any kernel).
 */
arb_status arb_decode_step(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                           const void *v_new, void *k_pages, void *v_pages, const int32_t *block_table,
                           int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream);

/*
 * Decode attention (every q_len 1 or 0) over an E4M3 KV cache: keys are k_scale * code, values v_scale * code,
 * one byte per element -- half the bytes per token of the bf16 cache, for the token-by-token steps of a
 * quantised draft model (Section 3.1: z_i ~ q(z_i | x, z_<i); Section 5.1 runs 4-bit and 3-bit drafts; the
 * cache format is this library's choice).  q and out are bf16; head_dim 128; g <= 8.
 *
 *   params     as for arb_attn, dtype ARB_BF16 (the type of q and out), max_q_len 1.  ARB_ATTN_OVERLAP_PREVIOUS
 *              has the meaning it has for arb_attn.
 *   k_codes,
 *   v_codes    uint8 [num_pages, Hkv, P, D], written by arb_kv_append_e4m3 with inv_scale = 1 / scale.
 *   k_scale,
 *   v_scale    > 0, host scalars.
 * The codes widen to f16 exactly; products run on the tensor cores in f16 with fp32 accumulation and the
 * softmax weights are rounded to f16.  Against an oracle that reads the same codes the result meets the
 * tolerance of the bf16 path; what quantisation itself costs is a property of the format, not of this call.
 */
arb_status arb_attn_decode_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const uint8_t *k_codes,
                                const uint8_t *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                                const int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream);

/*
 * arb_attn over an E4M3 KV cache, decode rows and step chunks alike (q_lens 0, 1 or a step length): what a
 * quantised draft's cache needs for all of Algorithm 1 -- its own token-by-token steps, and the causal chunk by
 * which it absorbs the target's step after an escalation (Section 5.1 for the quantised-draft regime; the cache
 * format is this library's choice).  Arguments as for arb_attn_decode_e4m3, params->max_q_len = the largest
 * q_len.  Decode rows run on that call's kernel; chunks on the tcgen05 kernel of arb_attn with the codes widened
 * to f16 on their way into its operand tiles (exact), q converted bf16 -> f16 (|q| must stay below the f16
 * range, 65504) and the softmax weights rounded to f16.  batch <= 512 when chunks are present.  Against an oracle
 * that reads the same codes the result meets the tolerance of the bf16 tensor-core paths.
 */
arb_status arb_attn_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const uint8_t *k_codes,
                         const uint8_t *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                         const int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream);

/*
 * Quantising KV append: as arb_kv_append, but the pools hold E4M3 codes, one byte per element (1 sign bit,
 * 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value 448) -- the
 * reduced-precision cache of a quantised draft model (Section 5.1 of the paper runs 4-bit and 3-bit drafts;
 * the cache format is this library's choice, the paper names none).
 *
 *   params        dtype is the type of k_new / v_new (fp32 or bf16); the other fields as for arb_kv_append.
 *   k_inv_scale,
 *   v_inv_scale   > 0.  code = e4m3(x * inv_scale): the product in fp32, the conversion to the nearest code,
 *                 ties to the even code, saturating at +-448.  The reader multiplies by 1 / inv_scale.
 *   k_codes,
 *   v_codes       uint8 [num_pages, Hkv, P, D].
 * Everything else (placement, length update, refusals and status bits) as arb_kv_append.
 */
arb_status arb_kv_append_e4m3(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                              const void *v_new, float k_inv_scale, float v_inv_scale, const int32_t *block_table,
                              int32_t *seq_lens, const int32_t *new_lens, int32_t update_lens, uint8_t *k_codes,
                              uint8_t *v_codes, arb_stream_t stream);

/*
 * One decode token of a quantised draft in one launch: arb_kv_append_e4m3 of the token's K/V rows (update_lens = 1),
 * arb_attn_decode_e4m3 over the cache that now holds them, and the length update, fused -- arb_decode_step for an
 * E4M3 cache (Section 3.1: z_i ~ q(z_i | x, z_<i), one call per token and layer; Section 5.1's quantised drafts).
 *
 *   params, q, out, k_new, v_new, block_table, seq_lens, q_lens
 *              as for arb_decode_step; dtype ARB_BF16 (q, out, k_new, v_new), head_dim 128, g <= 8.
 *   k_codes,
 *   v_codes    uint8 pools [num_pages, Hkv, P, D], written (code = e4m3(x * inv_scale): product in fp32, nearest
 *              code, ties to even, saturating at +-448) and read (key = k_scale * code, value = v_scale * code).
 *   k_scale, v_scale, k_inv_scale, v_inv_scale   > 0; the caller keeps inv_scale = 1 / scale (the library does not
 *              divide, so that the codes are those of arb_kv_append_e4m3 given the same inv_scale).
 * The codes written are bit-identical to arb_kv_append_e4m3's, the rows equal arb_attn_decode_e4m3's within its
 * tolerance.  Refused sequences, idle slots, status bits and stream behaviour as for arb_decode_step.
 * Errors: ARB_ERR_INVALID_ARG, ARB_ERR_UNSUPPORTED (dtype, head_dim, g > 8, ARB_ATTN_NO_TENSOR_CORES),
 * ARB_ERR_WORKSPACE, ARB_ERR_CUDA.
 */
arb_status arb_decode_step_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                                const void *v_new, uint8_t *k_codes, uint8_t *v_codes, float k_scale, float v_scale,
                                float k_inv_scale, float v_inv_scale, const int32_t *block_table, int32_t *seq_lens,
                                const int32_t *q_lens, void *out, arb_stream_t stream);

/*
 * One decode token over a 4-bit KV cache in one launch: arb_decode_step with the token's K/V rows quantised on the
 * way in (Section 3.1: z_i ~ q(z_i | x, z_<i); Section 5.1 runs 4-bit and 3-bit drafts; the cache format is this
 * library's own and is fixed here).
 *
 * Format.  Every (token, kv head) row of D = 128 values x has one fp32 scale s = max|x| / 7 (IEEE division in fp32;
 * 0 for a row of zeros) and 128 codes c = clamp(rint(x * (7 / max|x|)), -7, 7) (the reciprocal by IEEE division in
 * fp32, the product in fp32, nearest with ties to even; 0 for a row of zeros); the value read back is s * c.  A
 * nibble holds c + 8.  A group of 8 dimensions d0 .. d7 is one little-endian 32-bit word whose nibbles 0 .. 7 (from the
 * least significant) hold d0, d2, d4, d6, d1, d3, d5, d7.  NaN and infinities are outside the format.
 *
 *   params, q, out, k_new, v_new, block_table, seq_lens, q_lens
 *              as for arb_decode_step; dtype ARB_BF16 (q, out, k_new, v_new), head_dim 128, g <= 8.
 *   k_codes,
 *   v_codes    uint8 pools [num_pages, Hkv, P, D / 2], written (one row per sequence and kv head) and read.
 *   k_scales,
 *   v_scales   fp32 pools [num_pages, Hkv, P], written and read; 16-byte aligned.
 * Codes and scales written are bit-identical to the format's definition; the rows are attention over s * c within
 * the tolerance of arb_attn (the weights that reach the tensor core are rounded to bf16 after they took the value
 * scale).  Refused sequences, idle slots, status bits and stream behaviour as for arb_decode_step.
 * Errors: ARB_ERR_INVALID_ARG, ARB_ERR_UNSUPPORTED (dtype, head_dim, g > 8, ARB_ATTN_NO_TENSOR_CORES),
 * ARB_ERR_WORKSPACE, ARB_ERR_CUDA.
 */
arb_status arb_decode_step_i4(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                              const void *v_new, uint8_t *k_codes, uint8_t *v_codes, float *k_scales, float *v_scales,
                              const int32_t *block_table, int32_t *seq_lens, const int32_t *q_lens, void *out,
                              arb_stream_t stream);

/*
 * The 4-bit cache's quantising append: arb_kv_append with the rows encoded on the way in (the format of
 * arb_decode_step_i4: per-row scale max|x| / 7, codes rint(x * 7 / max|x|) in -7 .. 7, interleaved nibbles).  The cache
 * write of a step's tokens, or of a prefix (Algorithm 1 absorbs steps into the caches; Section 5.1's quantised drafts).
 *
 *   params, total_new, k_new, v_new, block_table, seq_lens, new_lens, update_lens
 *              as for arb_kv_append; dtype ARB_BF16 (the type of k_new / v_new), head_dim 128.
 *   k_codes, v_codes    uint8 pools [num_pages, Hkv, P, D / 2];  k_scales, v_scales    fp32 pools [num_pages, Hkv, P].
 * Placement, refusals and status bits are arb_kv_append's; codes and scales are bit-identical to the format's definition.
 * Errors: ARB_ERR_INVALID_ARG, ARB_ERR_UNSUPPORTED (dtype, head_dim, page size, batch), ARB_ERR_CUDA.
 */
arb_status arb_kv_append_i4(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                            const void *v_new, const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens,
                            int32_t update_lens, uint8_t *k_codes, uint8_t *v_codes, float *k_scales, float *v_scales,
                            arb_stream_t stream);

/*
 * Spearman's rank correlation of two samples (Section 4.2, "Evaluation", and Tables 1-3 of the paper:
 * the correlation between the router's predicted scores and the oracle advantage Delta).  Each value is
 * replaced by its rank within its sample, equal values sharing the mean of the ranks they span, and
 * rho is the Pearson correlation of the two rank variables.
 *
 *   x, y   fp32 [n], finite;  n <= 65536 (ranks are found by counting, n^2 comparisons).
 *   rho    DEVICE pointer to one double (8-byte aligned): the result, NaN when n < 2 or a sample is
 *          constant.  Sums are taken in fp64.
 * Uses three accumulators in the ctx: one call at a time per ctx.
 */
arb_status arb_spearman(arb_ctx *ctx, int32_t n, const float *x, const float *y, double *rho, arb_stream_t stream);

/*
 * Lengths of the next call of a phase of Algorithm 1, derived on the device so that the loop never reads
 * a length or a decision on the host: after the routing decision, accepted steps are absorbed by the
 * caches that did not generate them, and escalated steps are regenerated token by token by the target.
 *
 *   step_lens  int32 [B] (negative counts as 0);  decisions  uint8 [B], nullable.
 *   A sequence takes part iff decisions is NULL or (decisions[b] != 0) == (want != 0).
 *   t >= 0:  out[b] = 1 if it takes part and t < step_lens[b], else 0   (token t of a step decoded token by token)
 *   t <  0:  out[b] = step_lens[b] if it takes part, else 0             (a whole step absorbed as one chunk)
 *   out        int32 [B]; may be used as q_lens of arb_attn and as new_lens of arb_kv_append.
 */
arb_status arb_phase_lens(arb_ctx *ctx, int32_t batch, const int32_t *step_lens, const uint8_t *decisions /* nullable */,
                          int32_t want, int32_t t, int32_t *out, arb_stream_t stream);

/*
 * arb_phase_lens for all tokens of a step that is generated token by token, in one launch: the lengths of
 * token t depend only on step_lens and decisions, which are fixed while the step is generated.
 *   out  int32 [n_tokens, B]:  out[t][b] = 1 if b takes part and t < step_lens[b], else 0;  row t is what
 *        arb_phase_lens gives for that t.  batch * n_tokens <= 2^30.
 */
arb_status arb_phase_lens_tokens(arb_ctx *ctx, int32_t batch, const int32_t *step_lens,
                                 const uint8_t *decisions /* nullable */, int32_t want, int32_t n_tokens, int32_t *out,
                                 arb_stream_t stream);

/*
 * Synchronise `stream`, read the device status word into *bits (nullable) and clear it together
 * with the split-KV arrival counters.  Returns ARB_OK if the word was zero, else
 * ARB_ERR_DEVICE_STATUS.
 */
arb_status arb_poll_status(arb_ctx *ctx, arb_stream_t stream, uint32_t *bits);

/*
 * ---- Self-test ----------------------------------------------------------------------------------
 * Every wait inside the kernels (on a TMA copy, on a tensor-core commit) gives up after a bounded number of
 * cycles, raises ARB_DEV_WAIT_TIMEOUT, makes the other waits of its CTA return at once and lets the kernel
 * end normally.  A healthy run never takes that path, so this call exists to exercise it: it launches one
 * small kernel (64 threads) that waits, with the library's own wait routine, on a barrier nothing will ever
 * signal.  The first warp gives up after limit_cycles SM cycles (1 .. 2^31, i.e. up to about a second); the
 * second warp is given a far longer limit and must leave through the CTA's abort flag.  Nothing faults or
 * traps; the ctx stays usable and the next arb_poll_status reports and clears ARB_DEV_WAIT_TIMEOUT.
 *   report   DEVICE pointer to three int32: [0] = 1 once the kernel has run to its end, [1] = threads whose
 *            wait returned "gave up" (64 expected), [2] = cycles the first thread waited.
 * The paper has no counterpart; this is failure-detection plumbing of the library.
 */
arb_status arb_selftest_wait_timeout(arb_ctx *ctx, int64_t limit_cycles, int32_t *report, arb_stream_t stream);

/*
 * The bounds-check build (python -m paper_2512_05033_b200.build --checks, libarb_checks.so, -DARB_CHECKS) tests
 * the indices the kernels derive on the device before they are used (ring stage, block-table entry, workspace
 * slot, output row, pool offset): a failing test raises ARB_DEV_CHECK_FAILED and skips the access.  In that
 * build every buffer a ctx owns also lies between two guard zones of a fixed byte pattern.  This call counts,
 * on `stream`, the guard bytes that no longer hold the pattern and returns the count in *bad (host pointer)
 * after synchronising; the ordinary build owns no guard zones and returns 0.  *checked receives the number of
 * guard bytes looked at.  The paper has no counterpart; this stands in for a memory checker.
 */
arb_status arb_selftest_guard_zones(arb_ctx *ctx, arb_stream_t stream, int64_t *bad, int64_t *checked);

/* Number of kernels the library has launched through this ctx since arb_create. */
uint64_t arb_launch_count(const arb_ctx *ctx);

const char *arb_status_string(arb_status status);

#ifdef __cplusplus
}
#endif
#endif /* ARB_H_ */
