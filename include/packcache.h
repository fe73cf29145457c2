/*
 * packcache.h — C ABI of the PackCache hot path on one B200 (sm_100a).
 *
 * The library keeps a video generator's KV cache small and runs the current
 * frame's attention over it: text and conditioning-image tokens ("anchors") are
 * always kept, every earlier frame keeps a number of tokens that shrinks with
 * its temporal distance, and kept tokens carry their original (t, h, w)
 * coordinates so that 3D rotary attention stays spatially coherent (paper
 * Sec. 3.4; attention is Eq. 2 of Sec. 3.1).
 *
 * Conventions
 *  - Plain C, no CUDA types: a stream is passed as void* (a cudaStream_t; NULL
 *    is the default stream).
 *  - Pointers marked "device" are device memory owned by the caller and must be
 *    16-byte aligned; pointers marked "host" are ordinary host memory, read
 *    before the call returns.  The library never frees or keeps caller memory.
 *    It owns only the context (rotary tables, a status word, scratch sized at
 *    pc_create from the limits in pc_layer_desc).
 *  - Layout is token-major: K/V [token][kv_head][head_dim], Q/O
 *    [token][q_head][head_dim], pos [token][4] int32 = (t, h, w, tag) holding
 *    already scaled integer coordinates (MM-RoPE scales latent coordinates by
 *    (4, 8, 8), Sec. 3.1) and an opaque tag that compaction copies unchanged.
 *    Element type is pc_layer_desc.dtype for K, V, Q and O.
 *  - Errors the host can see (bad arguments, budgets, capacities) are returned
 *    at once and nothing is enqueued.  Device work is asynchronous on the given
 *    stream.  A kernel that meets a bad index, an out-of-table position or a
 *    wait that ran out records the first such event in the context's status
 *    word, skips the access and finishes; pc_poll_status returns it.
 *  - Calls on one context must be issued from one host thread at a time, and
 *    calls that share a context's scratch must be ordered on the GPU (same
 *    stream or explicit dependencies).
 */
#ifndef PACKCACHE_H
#define PACKCACHE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PC_OK = 0,
    PC_ERR_INVALID_ARG = 1, /* null / misaligned pointer, bad size, position outside the rotary tables */
    PC_ERR_BUDGET = 2,      /* a frame's budget exceeds its tokens, or kept-whole frames exceed the total */
    PC_ERR_CAPACITY = 3,    /* destination segment or context scratch too small */
    PC_ERR_UNSUPPORTED = 4, /* head_dim not 64/128, heads not divisible, dtype unknown */
    PC_ERR_CUDA = 5,        /* a CUDA runtime call failed */
    PC_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up */
} pc_status;

enum { PC_F32 = 0, PC_BF16 = 1 };

/* decay kernels g(dist), dist = 1 for the most recent history frame (Eq. 5-7) */
enum {
    PC_GEOMETRIC = 0,   /* g = param^dist, 0 < param < 1 (Eq. 5) */
    PC_CLOSED_HALF = 1, /* g = 2^-min(dist, W-1), the deployed closed form (Eq. 7) */
    PC_LINEAR = 2,      /* g = W + 1 - dist */
    PC_HALFLIFE = 3     /* g = 2^-((dist - 1 - keep_full) / param), param = half-life in frames */
};

#define PC_MAX_FRAMES 256 /* most history frames one pc_score call accepts */

typedef struct pc_ctx pc_ctx;

typedef struct {
    int32_t n_q_heads;  /* Hq */
    int32_t n_kv_heads; /* Hkv, divides Hq (grouped-query attention) */
    int32_t head_dim;   /* 64 or 128 */
    int32_t dtype;      /* PC_F32 or PC_BF16: storage type of Q, K, V, O */
    double rope_base;   /* rotary base, e.g. 10000 */
    int32_t max_pos[3]; /* exclusive upper bound of t, h, w: extents of the rotary tables */
    int32_t max_q;      /* most query tokens in one call */
    int32_t max_keys;   /* most keys attended in one call (anchors + history + current), and most
                           history tokens scored in one call */
} pc_layer_desc;

/* A run of tokens: anchors, history, or the frame being generated. */
typedef struct {
    void *k;          /* device [capacity][Hkv][d] */
    void *v;          /* device [capacity][Hkv][d] */
    int32_t *pos;     /* device [capacity][4] */
    int32_t n_tokens; /* tokens in use */
    int32_t capacity; /* tokens allocated */
} pc_segment;

/* The cache C_t of Sec. 3.4: anchors held apart from the decayed history. */
typedef struct {
    pc_segment anchors;         /* [text | conditioning image]; never moved, never scored */
    pc_segment history;         /* history frames, oldest -> newest, contiguous */
    int32_t n_frames;           /* history frames */
    const int32_t *frame_count; /* host [n_frames]: tokens of each frame; sums to history.n_tokens */
} pc_cache;

typedef struct {
    int32_t kind;      /* PC_GEOMETRIC ... PC_HALFLIFE */
    double param;      /* rho or half-life, see the enum */
    int64_t total;     /* history tokens to retain in all, anchors not counted (B_one of Eq. 8) */
    int32_t keep_full; /* most recent frames kept whole (counted inside total) */
    int32_t min_quota; /* b_min of Sec. 3.4 in tokens: every frame that takes part keeps at least this many; 0 = none */
} pc_budget_params;

/* Create / destroy a context on the current CUDA device.  Builds the rotary
 * cos/sin tables (Sec. 3.1: pair i of d/2 turns with axis i mod 3 at frequency
 * base^(-(i div 3)/n_axis)) and allocates scratch for max_q / max_keys.
 * Shapes: head_dim 64 or 128; n_q_heads a multiple of n_kv_heads; at most 4096 elements in a key row over all KV heads.
 * Scoring (pc_score, pc_frame_step, the cache window) further needs a key row (n_kv_heads * head_dim elements of the
 * dtype) of 512, 1024, 1536, 2048, 3072 or 4096 bytes and a query row that is a multiple of 512 bytes, and returns
 * PC_ERR_UNSUPPORTED otherwise, before anything is enqueued; pc_compact and pc_attend_frame take any accepted shape.
 * Errors: PC_ERR_UNSUPPORTED, PC_ERR_INVALID_ARG, PC_ERR_CUDA. */
pc_status pc_create(const pc_layer_desc *desc, pc_ctx **out);
pc_status pc_destroy(pc_ctx *ctx);

/* Per-frame token budgets (Sec. 3.4, Eq. 5-8; anchors are excluded from the
 * decay and always kept).  Host only, integers after one quantisation of the
 * weights to 2^-32: the keep_full newest frames keep everything; the rest of
 * `total` is shared in proportion to g(dist) by largest remainder (ties to the
 * nearer frame); a frame granted more than avail keeps avail and the surplus is
 * re-shared.  With min_quota > 0 every frame that takes part is first guaranteed min(min_quota, avail) tokens and the
 * decay kernel shares out the rest on top; if the guarantees of all frames exceed the budget, the oldest frames leave
 * the window first (first in, first out) and get nothing.  avail and budget are host arrays [n_frames], oldest -> newest.
 * The result sums to min(total, sum(avail)) (over the frames that take part).
 * Errors: PC_ERR_INVALID_ARG (null, negative, bad param),
 * PC_ERR_BUDGET (kept-whole frames exceed total). */
pc_status pc_plan_budget(const pc_budget_params *params, int32_t n_frames, const int32_t *avail,
                         int32_t *budget);

/* Score every history token and pick each frame's budget[f] best (Sec. 3.4,
 * "attention-relevant" retention).  score_j = mean over the n_q queries and all
 * query heads of the scaled rotary logit (R q).(R k_j)/sqrt(d), computed in
 * fp32 through a pooled query.  Per frame the budget[f] highest scores are
 * kept, equal scores by lower index (-0 == +0), and written to sel_idx as
 * ascending global history indices, frames oldest -> newest.
 *   q device [n_q][Hq][d]; q_pos device [n_q][4]; budget host [n_frames];
 *   valid device [n_src] bytes or NULL (0 = masked cache position, Eq. 1: never
 *   kept unless the budget exceeds the valid tokens);
 *   scores_override device [n_src] fp32 or NULL: skip scoring, select on these (4-byte alignment is enough here, so
 *   an offset into a longer score array, such as the attention masses past the anchors, can be passed);
 *   scores device out [n_src] fp32 (may be NULL with an override);
 *   sel_idx device out [sum(budget)].
 * Errors: PC_ERR_INVALID_ARG, PC_ERR_BUDGET (budget[f] > frame_count[f]),
 * PC_ERR_CAPACITY (n_src > max_keys, n_q > max_q, n_frames > PC_MAX_FRAMES). */
pc_status pc_score(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q,
                   const int32_t *budget, const uint8_t *valid, const float *scores_override,
                   float *scores, int32_t *sel_idx, void *stream);

/* Pack the selected rows into dst (Fig. 6b: evicted positions are removed, not
 * zero-filled) with the spatially preserving rebase (Eq. 9): dst history row r
 * is src history row sel_idx[r]; K, V, (h, w, tag) are bit copies, t has
 * delta_t subtracted.  dst.history.n_tokens / n_frames are set by the caller to
 * sum(budget) / src.n_frames; dst anchors are not touched (anchors never move).
 *   sel_idx device [sum(budget)]; budget host [src.n_frames].
 * Errors: PC_ERR_INVALID_ARG (dst aliases src, null), PC_ERR_BUDGET,
 * PC_ERR_CAPACITY (sum(budget) > dst.history.capacity). */
pc_status pc_compact(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget,
                     int32_t delta_t, pc_cache *dst, void *stream);

/* Attention of the current frame's queries over anchors ++ history ++ current
 * (Eq. 2; a whole-frame query block sees every cached key, so no mask is left):
 *   out[i][h] = softmax_j((R q_ih).(R k_j,g)/sqrt(d)) v_j,g,  g = h / (Hq/Hkv).
 * Rotary embedding is applied from the stored positions inside the call.
 *   current may be NULL; q device [n_q][Hq][d]; out device [n_q][Hq][d];
 *   lse device [n_q][Hq] fp32 natural-log sum of exponentials, or NULL.
 * bf16 with head_dim 128 runs on tcgen05 tensor cores (fp32 accumulate and softmax) when Hkv*d and Hq*d are
 * multiples of 256; everything else runs on CUDA cores.  Errors: PC_ERR_INVALID_ARG, PC_ERR_CAPACITY (keys > max_keys,
 * n_q > max_q), PC_ERR_CUDA. */
pc_status pc_attend_frame(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, const void *q,
                          const int32_t *q_pos, int32_t n_q, void *out, float *lse, void *stream);

/* The same attention in two parts, for a frame that is generated over several passes that all attend to one unchanged
 * cache (the diffusion steps of Sec. 3.1 / Fig. 4): pc_attend_prepare fixes the key set (anchors ++ history ++ current)
 * and applies the rotary embedding to its keys once; pc_attend_prepared then runs one pass for the given queries and
 * only rotates those.  Results are identical to pc_attend_frame on the same inputs.  The caller must not change the
 * segments' K, V or positions between the two calls; the prepared key set lives in the context's scratch and is
 * dropped by the next pc_attend_prepare or pc_attend_frame on this context.
 * Errors: as pc_attend_frame; pc_attend_prepared returns PC_ERR_INVALID_ARG when nothing is prepared. */
pc_status pc_attend_prepare(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, void *stream);
pc_status pc_attend_prepared(pc_ctx *ctx, const void *q, const int32_t *q_pos, int32_t n_q, void *out, float *lse,
                             void *stream);

/* One frame of the steady state in one call (Fig. 6b-c: score, keep each frame's quota, pack, then attend with Eq. 2):
 * the same results as pc_score (no mask, no override) -> pc_compact -> pc_attend_frame over src's anchors ++ the packed
 * history, with q serving both the scores and the attention.  What the one call saves on the bf16 tensor-core path: Q is
 * read and rotated once (the pass that pools it for the scores also leaves the rotated queries of Eq. 2), the pack
 * kernel also leaves the rotated keys of the rows it packs (at their rebased positions, Eq. 9), and the anchors'
 * rotated keys are kept in the context from the first step that sees an anchor segment (same k / pos pointers and
 * token count) — anchors never move (Sec. 3.4, condition anchoring) — so attention starts without a rotary pre-pass.
 * Outputs are bit-identical to the three separate calls.
 *   budget host [src.n_frames] (from pc_plan_budget); dst: its history buffers receive the packed rows, its
 *   history.n_tokens and n_frames are set to sum(budget) and src.n_frames (frame_count is left to the caller), its
 *   anchors field is ignored; scores device out [n_src]; sel_idx device out [sum(budget)]; out, lse as pc_attend_frame.
 * Call pc_forget_anchors after changing the anchors' K or positions in place; pc_attend_frame / pc_attend_prepare on
 * the same context drop the kept anchor keys as well (they are rebuilt by the next step).
 * Errors: as the three calls. */
pc_status pc_frame_step(pc_ctx *ctx, const pc_cache *src, const int32_t *budget, int32_t delta_t, pc_cache *dst,
                        const void *q, const int32_t *q_pos, int32_t n_q, float *scores, int32_t *sel_idx, void *out,
                        float *lse, void *stream);
pc_status pc_forget_anchors(pc_ctx *ctx);

/* Attention mass of every key (Sec. 3.4: retention is guided by the attention a cached token receives):
 *   mass_j = 1/(n_q*Hq) * sum over the query rows (i, h) of softmax_j((R q_ih).(R k_j,g(h))/sqrt(d)),
 * the mean, over the frame's queries and heads, of the probabilities of Eq. 2; the masses of all keys sum to one.
 * It is computed for the key set and the queries of the most recent pc_attend_frame / pc_attend_prepared call on this
 * context, whose rotated keys and queries are still in the context's scratch: call it after that call, ordered behind
 * it on the GPU, with the lse that call wrote, and before any other attention call on the context.
 *   lse device [n_q][Hq] fp32 (as written by the attention call); n_keys = all keys of that call;
 *   mass device out [n_keys] fp32 in key order anchors ++ history ++ current.
 * mass + (number of anchor tokens), i.e. the masses of history ++ current, can be passed as scores_override to
 * pc_score or — once the current frame has been appended, and past the tokens of any frame the window is about to
 * drop — to pc_window_update, which then ranks by attention mass instead of by the mean logit.
 * bf16 tensor-core path only.  Errors: PC_ERR_UNSUPPORTED (fp32 context, head_dim != 128, Hkv*d or Hq*d not a
 * multiple of 256, CUDA-core kernel chosen),
 * PC_ERR_INVALID_ARG (null or misaligned pointer, no such attention call precedes, n_keys differs from that call's),
 * PC_ERR_CUDA. */
pc_status pc_attend_mass(pc_ctx *ctx, const float *lse, float *mass, int32_t n_keys, void *stream);

/* One frame step with inputs and output in HOST memory (pinned memory keeps the copies asynchronous): copies Q,
 * positions, anchors and the history frames into the caller's device workspace, plans the budget, scores, selects,
 * packs and attends (anchors ++ packed history), copies the output back and waits for the stream.  Everything the
 * four calls above state applies; the workspace capacities bound the sizes (PC_ERR_CAPACITY). */
typedef struct {
    const void *q;              /* host [n_q][Hq][d] */
    const int32_t *q_pos;       /* host [n_q][4] */
    int32_t n_q;
    const void *anchor_k, *anchor_v; /* host [n_anchor][Hkv][d] */
    const int32_t *anchor_pos;  /* host [n_anchor][4] */
    int32_t n_anchor;
    const void *hist_k, *hist_v; /* host [sum(frame_count)][Hkv][d] */
    const int32_t *hist_pos;    /* host [sum(frame_count)][4] */
    int32_t n_frames;
    const int32_t *frame_count; /* host [n_frames] */
    void *out;                  /* host out [n_q][Hq][d] */
} pc_host_frame;

typedef struct {
    pc_cache src;     /* device staging for anchors and history (capacities used, counts ignored) */
    pc_cache dst;     /* device destination of the packed history (its anchors field is ignored) */
    void *q;          /* device [>= n_q][Hq][d] */
    int32_t *q_pos;   /* device [>= n_q][4] */
    float *scores;    /* device [>= history tokens] */
    int32_t *sel_idx; /* device [>= retained tokens] */
    void *out;        /* device [>= n_q][Hq][d] */
} pc_device_workspace;

pc_status pc_frame_step_host(pc_ctx *ctx, const pc_host_frame *in, pc_device_workspace *ws,
                             const pc_budget_params *params, int32_t delta_t, void *stream);

/* Scoring for callers that cannot allocate.  (The paper has no counterpart: this entry point exists for the sake of
 * host programs, not of the method.)  Some hosts cannot call cudaMalloc where they need scores — their device memory
 * was given to an arena of their own at start-up and driver allocations are forbidden afterwards, or they sit on a
 * latency-critical thread that cannot take the device-wide synchronisation an allocation or a free implies — and so
 * cannot create a pc_ctx either.  This call needs no context and calls neither cudaMalloc nor cudaFree nor any
 * allocating routine: the rotary table, the pooled query and its accumulator live in one fixed device array
 * of 332,288 bytes that is part of the library image (every GPU that loads the library holds it until exit).
 *
 * Computes the same scores as pc_score (mean scaled rotary logit of every history token over the n_q queries and
 * all query heads, fp32); selection is not included.  desc->max_q / max_keys are ignored.
 *   hist_k device [n_src][Hkv][d]; hist_pos device [n_src][4]; q device [n_q][Hq][d]; q_pos device [n_q][4];
 *   valid device [n_src] bytes or NULL; scores device out [n_src] fp32;
 *   status device [2] int32, zeroed by the caller: receives (PC_ERR_INVALID_ARG, where) if a position lies outside
 *   desc->max_pos (the position is clamped and the call completes); the caller copies it back when it wants it.
 * Limits (PC_ERR_CAPACITY with a message on stderr beyond them): n_kv_heads*head_dim <= 1024;
 * sum over the three axes of max_pos[a] * (rotary pairs on axis a) <= 32768; n_q_heads*head_dim <= 12288.
 * The first call on each device looks up the array's device address (that device must be current); make that
 * first call outside any stream capture.  All calls share the one array, which keeps the previous call's
 * contents (the call rewrites the table and clears the accumulator before it uses them): two calls that may overlap on the GPU — different
 * streams without an ordering between them — race; order them.  Work is asynchronous on the given stream.
 * Other errors: PC_ERR_INVALID_ARG (null or misaligned pointer, n_src or n_q <= 0), PC_ERR_UNSUPPORTED, PC_ERR_CUDA. */
pc_status pc_score_tokens_static(const pc_layer_desc *desc, const void *hist_k, const int32_t *hist_pos,
                                 int32_t n_src, const void *q, const int32_t *q_pos, int32_t n_q,
                                 const uint8_t *valid, float *scores, int32_t *status, void *stream);

/* ---- Cache window: the Fill / Pack / Slide regimes of Sec. 3.4 (Fig. 6) around the calls above.
 *
 * The window keeps at most `window` history frames (W of Eq. 3) in one of two caller-owned history buffers.
 *   Fill : appended frames are kept whole while they fit the token budget (budget.total) and the window.
 *   Pack : once they do not, every retained frame is cut to its quota (pc_plan_budget over the frames' current token
 *          counts), keeping the tokens that score best against the current frame's queries, and the survivors are packed
 *          into the other buffer, which becomes the active one.
 *   Slide: a frame beyond the window is dropped first (first in, first out), the rest is re-packed under the same rule, and
 *          with `rebase` set the temporal coordinate of every retained history token drops by t_step per dropped frame
 *          (Eq. 9: only t moves; h, w and the tag are carried).  Anchors are never touched.  The caller builds the next
 *          frames' positions in the shifted frame of reference: pc_window_state reports the accumulated shift.
 *          Frames that a plan leaves with nothing at the old end of the window (budget.min_quota starves the oldest frames first
 *          when the budget cannot serve every frame) leave it in the same way and count in the rebase.
 * Re-selection is incremental: the source of a pack is what the last pack kept plus the frames appended since.
 * All device memory is the caller's: the two history buffers (each must hold budget.total tokens plus the frames
 * appended between two packs), a score buffer and an index buffer of the same token capacity. */
typedef struct pc_window pc_window;

typedef struct {
    int32_t window;          /* W: most history frames kept */
    pc_budget_params budget; /* decay kernel and token budget of the history (anchors not counted) */
    int32_t rebase;          /* 1: apply the temporal rebase of Eq. 9 when frames are dropped */
    int32_t t_step;          /* temporal coordinate units per frame (4 under MM-RoPE's scaling) */
} pc_window_params;

enum { PC_WINDOW_FILL = 0, PC_WINDOW_PACK = 1, PC_WINDOW_SLIDE = 2 };

/* scores device [capacity] fp32 and sel_idx device [capacity] int32, capacity = the smaller history buffer's.
 * Errors: PC_ERR_INVALID_ARG (null, window < 1, t_step < 0, empty buffers, misaligned). */
pc_status pc_window_create(pc_ctx *ctx, const pc_window_params *params, const pc_segment *anchors,
                           const pc_segment *hist_a, const pc_segment *hist_b, float *scores, int32_t *sel_idx,
                           pc_window **out);
pc_status pc_window_destroy(pc_window *w);

/* Append a finished frame (device K, V, pos; positions already in the shifted frame of reference) as the newest
 * history frame: device-to-device copies on the stream.  Errors: PC_ERR_CAPACITY (active buffer full). */
pc_status pc_window_append(pc_window *w, const pc_segment *frame, void *stream);

/* Append only the unmasked positions of a finished frame (cache mask of Eq. 1; Fig. 6b: masked positions are removed,
 * not stored): valid is a device array of frame->n_tokens bytes, non-zero = keep; n_valid (host) is how many are
 * non-zero, which the caller knows from its masking schedule.  Kept rows keep their order and positions.  A mask
 * whose count differs from n_valid is recorded in the context's status word (PC_ERR_INVALID_ARG).
 * Errors: PC_ERR_INVALID_ARG, PC_ERR_CAPACITY. */
pc_status pc_window_append_masked(pc_window *w, const pc_segment *frame, const uint8_t *valid, int32_t n_valid, void *stream);

/* Bring the cache back inside window and budget for the frame whose queries are q (see the regimes above); regime
 * (host out, may be NULL) receives PC_WINDOW_FILL / PACK / SLIDE.  scores_override: device fp32 scores of the source
 * tokens (after the frames beyond the window; frames the plan then starves are skipped inside) to select on instead of
 * scoring, or NULL.  Errors as pc_score / pc_compact. */
pc_status pc_window_update(pc_window *w, const void *q, const int32_t *q_pos, int32_t n_q, const float *scores_override,
                           int32_t *regime, void *stream);

/* Update and attention in one call: what pc_window_update (without an override) followed by pc_attend_frame over the
 * window's cache give, bit for bit, through the fused frame step (pc_frame_step) whenever the update packs.
 *   q, q_pos device; out device [n_q][Hq][d]; lse device or NULL; regime host out or NULL. */
pc_status pc_window_step(pc_window *w, const void *q, const int32_t *q_pos, int32_t n_q, void *out, float *lse,
                         int32_t *regime, void *stream);

/* The same step with its per-frame inputs and its output in HOST memory, the cache staying resident on the device
 * (Fig. 6c: in the steady state a frame brings only its own keys, values and queries; Eq. 3: the cache itself is
 * bounded): copies the frame that was just finished (its K, V, positions; n_frame may be 0) to the end of the active
 * history buffer and the new frame's queries and positions into the workspace, runs pc_window_step, copies the
 * output back and waits for the stream.  Pinned host memory keeps the copies asynchronous.  All arguments are checked
 * before anything is enqueued.  Errors: as pc_window_append and pc_window_step. */
typedef struct {
    const void *frame_k, *frame_v; /* host [n_frame][Hkv][d]: the frame to append as the newest history frame */
    const int32_t *frame_pos;      /* host [n_frame][4], in the shifted frame of reference (pc_window_state) */
    int32_t n_frame;
    const void *q;                 /* host [n_q][Hq][d] */
    const int32_t *q_pos;          /* host [n_q][4] */
    int32_t n_q;
    void *out;                     /* host out [n_q][Hq][d] */
} pc_host_window_step;

typedef struct {
    void *q;        /* device [>= n_q][Hq][d] */
    int32_t *q_pos; /* device [>= n_q][4] */
    void *out;      /* device [>= n_q][Hq][d] */
} pc_window_step_workspace;

pc_status pc_window_step_host(pc_window *w, const pc_host_window_step *in, const pc_window_step_workspace *ws,
                              int32_t *regime, void *stream);

/* The current cache as a pc_cache for pc_attend_frame (frame_count points into the window: valid until the next
 * append / update / destroy). */
pc_status pc_window_cache(pc_window *w, pc_cache *out);

/* Host-side state: frames kept, their token counts oldest -> newest (counts may be NULL, else room for window + 1),
 * the accumulated temporal shift, and which buffer (0 = hist_a, 1 = hist_b) is active. */
pc_status pc_window_state(pc_window *w, int32_t *n_frames, int32_t *counts, int64_t *t_shift, int32_t *active);

/* Wait for the stream, then return and clear the first device-side event
 * recorded since the last poll (PC_OK if none). */
pc_status pc_poll_status(pc_ctx *ctx, void *stream);

/* Choose the bf16 attention kernel: 0 = tcgen05 tensor-core kernel (default), 1 = CUDA-core kernel (a slow second
 * opinion).  Returns PC_ERR_INVALID_ARG otherwise. */
pc_status pc_set_attend_impl(pc_ctx *ctx, int32_t impl);

/* Fix the number of key ranges the tensor-core attention kernel splits the keys into (1..4); 0 lets each call
 * choose the count that fills the GPU's SMs best.  Results agree up to fp32 rounding order. */
pc_status pc_set_kv_splits(pc_ctx *ctx, int32_t n);

/* How the key ranges of the tensor-core attention kernel are merged: 0 (default) = each range writes fp32 partials to
 * context scratch and a second kernel merges them; 1 = the ranges of one work item run as a thread-block cluster and
 * merge inside the kernel through distributed shared memory (no partials in global memory, one launch less).  On a
 * B200 only 45 clusters of three CTAs are resident at a time (135 of 148 SMs), so the cluster form pays only when the
 * number of work items fits that; results agree up to fp32 rounding order. */
pc_status pc_set_cluster_merge(pc_ctx *ctx, int32_t on);

/* Limit of every bounded device-side wait of the context's tensor-core attention kernel, in microseconds (0 = the
 * default of about one second).  A wait that runs out records PC_ERR_TIMEOUT in the status word, the CTA gives up its
 * remaining work, lets its copies land, frees its tensor memory and exits; the context stays usable. */
pc_status pc_set_wait_limit_us(pc_ctx *ctx, uint32_t limit_us);
/* Test hook for that path: the attention kernel's first barrier of every CTA is told to expect n_bytes more than are
 * ever sent, so its wait runs out after the limit above and pc_poll_status returns PC_ERR_TIMEOUT; the call's output
 * is then undefined.  0 switches the hook off.  Nothing traps and nothing waits without a limit. */
pc_status pc_test_expect_extra_bytes(pc_ctx *ctx, uint32_t n_bytes);

/* Per-kernel timing for benchmarks.  With timing on, each call records CUDA events on its stream at the boundaries
 * of its kernels (a few microseconds of overhead per call); pc_get_timing waits for the last recorded events and
 * writes the duration in milliseconds of each kernel of the most recent calls, -1 for a kernel that did not run.
 * ms is a host array [PC_N_STAGES]. */
enum { PC_STAGE_QPOOL = 0 /* the query pass */, PC_STAGE_SCORE = 1, PC_STAGE_SELECT = 2, PC_STAGE_PACK = 3, PC_STAGE_ROPE = 4,
       PC_STAGE_ATTEND = 5, PC_STAGE_COMBINE = 6, PC_STAGE_MASS = 7, PC_N_STAGES = 8 };
pc_status pc_set_timing(pc_ctx *ctx, int32_t on);
pc_status pc_get_timing(pc_ctx *ctx, float *ms);
/* The marks themselves, for finer measurements.  An event between two kernels drains the stream: the kernel behind it
 * starts from an idle GPU instead of overlapping its launch with the tail of the kernel before, so a span of one
 * kernel overstates it by a few microseconds.  pc_set_timing_skip leaves out the marks whose bits are set (bit i = mark
 * i); pc_get_span gives the time between any two recorded marks, -1 if either is missing.  With the mark between two
 * kernels left out, their common span minus the first kernel's own span is the second kernel's duration as it runs in
 * the untimed sequence.  Marks: a scoring call records SCORE0, QPOOL (after the query pass), SCORE (after the scoring
 * kernel), SELECT; a pack PACK0, PACK; an attention call ATT0, ROPE (only when a rotary pre-pass ran), ATTEND, COMBINE;
 * pc_attend_mass MASS0, MASS. */
enum { PC_MARK_SCORE0 = 0, PC_MARK_QPOOL = 1, PC_MARK_SCORE = 2, PC_MARK_SELECT = 3, PC_MARK_PACK0 = 4, PC_MARK_PACK = 5,
       PC_MARK_ATT0 = 6, PC_MARK_ROPE = 7, PC_MARK_ATTEND = 8, PC_MARK_COMBINE = 9, PC_MARK_MASS0 = 10, PC_MARK_MASS = 11,
       PC_N_MARKS = 12 };
pc_status pc_set_timing_skip(pc_ctx *ctx, uint32_t mark_mask);
pc_status pc_get_span(pc_ctx *ctx, int32_t mark_a, int32_t mark_b, float *ms);

/* Measurement support (the paper has no counterpart): streams n_rows rows of row_bytes (a multiple of 512) from device
 * memory with the access pattern of the scoring kernel — 16-byte streaming loads, two rows per warp in flight — and
 * writes one 32-bit word per row; no arithmetic beyond an xor.  Timed beside the scoring and pack kernels it says what
 * a kernel that only moves those bytes reaches on the GPU at hand, by an event pair per launch and back to back.
 *   src device [n_rows][row_bytes]; out device [n_rows] uint32.  Errors: PC_ERR_INVALID_ARG, PC_ERR_CUDA. */
pc_status pc_probe_stream_read(const void *src, int32_t n_rows, int32_t row_bytes, uint32_t *out, void *stream);

/* Measurement support (the paper has no counterpart): the tensor-core issue stream of the attention kernel alone.  n_cta
 * CTAs (one per SM; more than the GPU has SMs run in waves) each issue `rounds` rounds of the 128 x 128 x 16 bf16
 * multiply-adds the attention kernel issues per key tile for its two query tiles — form 0: the Q K^T ones only (both
 * operands in shared memory, 16 per round); form 1: the P V ones only (A in tensor memory, 16 per round); form 2: both in
 * the kernel's order (32 per round) — on pseudo-random operands, two rounds in flight, and record the SM cycles and the
 * global-timer nanoseconds the rounds took.  cycles / (rounds x multiply-adds per round) is what one multiply-add costs
 * when the tensor core never waits; cycles / nanos is the SM clock under that load.  Waits are bounded like the
 * attention kernel's (pc_set_wait_limit_us; a give-up shows in pc_poll_status).
 *   cycles, nanos device [n_cta] int64.  Errors: PC_ERR_INVALID_ARG, PC_ERR_UNSUPPORTED, PC_ERR_CUDA. */
pc_status pc_probe_mma_rate(pc_ctx *ctx, int32_t form, int32_t rounds, int32_t n_cta, int64_t *cycles, int64_t *nanos, void *stream);

const char *pc_status_string(pc_status s);

#ifdef __cplusplus
}
#endif
#endif /* PACKCACHE_H */
