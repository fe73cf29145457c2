/*
 * PackCache CPU oracle.  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, double-precision statement of what the compaction + attention
 * path computes, written from the paper (Sec. 3.1, Sec. 3.4) so that a reader
 * can check it against the text by eye.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library shares no code,
 * table or constant with it.
 *
 * Inputs are float arrays that already hold values exactly representable in
 * the workload's storage type (fp32 or bf16); everything after the load is
 * fp64.  Loops are written in the order of the definitions; OpenMP only splits
 * independent output elements between threads, so results do not depend on the
 * thread count.
 *
 * Layouts (token-major): K/V [token][kv_head][d]; Q/O [token][q_head][d];
 * pos [token][4] = (t, h, w, tag) with already-scaled integer coordinates.
 *
 * Pins: every function here is pinned by tests that do not call it to produce
 * the expected value (closed forms, the paper's printed allocation pattern,
 * brute force, numpy complex-number rotary arithmetic, library softmax).  The
 * one exception is the *choice* of the scoring rule in po_score: the paper says
 * retention is attention-guided but prints no formula, so that choice has
 * parity unpinned against the authors' system; it is pinned only as a
 * definition (mean pre-softmax logit).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { PO_GEOMETRIC = 0, PO_CLOSED_HALF = 1, PO_LINEAR = 2, PO_HALFLIFE = 3 };
enum { PO_OK = 0, PO_ERR_ARG = 1, PO_ERR_BUDGET = 2, PO_ERR_NAN = 3 };

int po_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void po_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------------
 * 3D rotary embedding (Sec. 3.1, the operator R in Eq. 2).
 * d/2 pairs; pair i = elements (2i, 2i+1); pair i turns with axis a = i mod 3
 * (t, h, w in turn), and is the m-th pair of that axis, m = i div 3.  With n_a
 * pairs on axis a the frequency is base^(-m / n_a) and the angle is
 * pos_a * frequency.  The same operator is applied to queries and keys.
 * ------------------------------------------------------------------------ */
static int pairs_on_axis(int n_pairs, int a) {
    int n = 0;
    for (int i = 0; i < n_pairs; ++i)
        if (i % 3 == a) ++n;
    return n;
}

void po_rope(const float *x, const int32_t *pos, int d, double base, double *out) {
    int n_pairs = d / 2;
    for (int i = 0; i < n_pairs; ++i) {
        int a = i % 3, m = i / 3;
        double theta = pow(base, -(double)m / (double)pairs_on_axis(n_pairs, a));
        double phi = (double)pos[a] * theta;
        double c = cos(phi), s = sin(phi);
        double x0 = (double)x[2 * i], x1 = (double)x[2 * i + 1];
        out[2 * i] = x0 * c - x1 * s;
        out[2 * i + 1] = x0 * s + x1 * c;
    }
}

/* rotate every head of every token of a [n][heads][d] array */
static double *rope_all(const float *x, const int32_t *pos, int64_t n, int heads, int d, double base) {
    double *r = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * heads * d);
    if (!r) return NULL;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j)
        for (int h = 0; h < heads; ++h)
            po_rope(x + ((size_t)j * heads + h) * d, pos + 4 * j, d, base, r + ((size_t)j * heads + h) * d);
    return r;
}

/* ------------------------------------------------------------------------
 * Budget plan (Sec. 3.4: decay kernel Eq. 5, normalised allocation Eq. 6,
 * closed form Eq. 7, per-frame token budget Eq. 8; anchors are outside it).
 *
 * Frames are passed oldest -> newest; temporal distance of frame f is
 * dist = n_frames - f (1 = most recent).  Weights: GEOMETRIC rho^dist;
 * CLOSED_HALF 2^-min(dist, W-1); LINEAR W+1-dist; HALFLIFE
 * 2^-((dist-1-keep_full)/h), i.e. rho = 2^(-1/h).  Each weight is turned once
 * into an integer floor(g * 2^32 + 1/2); after that only integers are used:
 *   1. the keep_full most recent frames keep all their tokens;
 *   2. the remaining total is shared by largest remainder: floor(B w / S),
 *      left-over units one each to the largest remainders (B w mod S), ties to
 *      the nearer frame;
 *   3. a frame given more than it holds is fixed at what it holds and leaves
 *      the share-out, which is repeated over the others with what is left.
 * The result sums to min(total, sum of avail).
 * ------------------------------------------------------------------------ */
typedef unsigned __int128 u128;

int po_plan_budget_min(int kind, double param, int64_t total, int keep_full, int min_quota, int n_frames,
                       const int32_t *avail_in, int32_t *budget) {
    if (n_frames < 0 || total < 0 || keep_full < 0 || min_quota < 0) return PO_ERR_ARG;
    if (kind == PO_GEOMETRIC && !(param > 0.0 && param < 1.0)) return PO_ERR_ARG;
    if (kind == PO_HALFLIFE && !(param > 0.0)) return PO_ERR_ARG;
    if (kind < 0 || kind > 3) return PO_ERR_ARG;
    int W = n_frames;
    if (W == 0) return PO_OK;
    uint64_t *w = (uint64_t *)calloc((size_t)W, sizeof(uint64_t));
    char *active = (char *)calloc((size_t)W, 1);
    int32_t *avail = (int32_t *)calloc((size_t)W, sizeof(int32_t));   /* room left in a frame above its guaranteed part */
    int32_t *floor_q = (int32_t *)calloc((size_t)W, sizeof(int32_t)); /* guaranteed part (minimum quota) */
    if (!w || !active || !avail || !floor_q) { free(w); free(active); free(avail); free(floor_q); return PO_ERR_ARG; }
    int64_t B = total;
    for (int f = 0; f < W; ++f) {
        int dist = W - f;
        if (avail_in[f] < 0) { free(w); free(active); free(avail); free(floor_q); return PO_ERR_ARG; }
        avail[f] = avail_in[f];
        budget[f] = 0;
        if (dist <= keep_full) {
            budget[f] = avail[f];
            B -= avail[f];
            continue;
        }
        double g;
        switch (kind) {
        case PO_GEOMETRIC: g = pow(param, (double)dist); break;
        case PO_CLOSED_HALF: g = ldexp(1.0, -(dist < W - 1 ? dist : W - 1)); break;
        case PO_LINEAR: g = (double)(W + 1 - dist); break;
        default: g = exp2(-(double)(dist - 1 - keep_full) / param); break;
        }
        w[f] = (uint64_t)floor(g * 4294967296.0 + 0.5);
        active[f] = 1;
    }
    if (B < 0) { free(w); free(active); free(avail); free(floor_q); return PO_ERR_BUDGET; }
    /* Minimum quota b_min (Sec. 3.4): a frame that takes part is guaranteed min_quota tokens (or all it holds, if
     * fewer).  When the guarantees of all frames would exceed the budget, the window shrinks first in, first out: only
     * the nearest floor(B / min_quota) frames take part, the farther ones get nothing.  The guarantees are set aside
     * and the decay kernel shares out what is left, on top of them. */
    if (min_quota > 0) {
        int64_t can_hold = B / min_quota, taking_part = 0;
        for (int f = W - 1; f >= 0; --f) {              /* nearest frame first */
            if (!active[f]) continue;
            if (taking_part >= can_hold) { active[f] = 0; continue; }
            ++taking_part;
            floor_q[f] = avail[f] < min_quota ? avail[f] : min_quota;
            avail[f] -= floor_q[f];
            B -= floor_q[f];
        }
    }
    for (;;) {
        u128 S = 0;
        int64_t room = 0;
        for (int f = 0; f < W; ++f)
            if (active[f]) { S += w[f]; room += avail[f]; }
        if (S == 0 || B == 0) break;
        if (B >= room) { /* everything that is left fits: all active frames are kept whole */
            for (int f = 0; f < W; ++f)
                if (active[f]) { budget[f] = avail[f]; active[f] = 0; }
            break;
        }
        int64_t given = 0;
        for (int f = 0; f < W; ++f)
            if (active[f]) { budget[f] = (int32_t)(((u128)B * w[f]) / S); given += budget[f]; }
        int64_t left = B - given;
        /* hand out the left-over units by largest remainder, ties to the nearer (later) frame */
        char *got = (char *)calloc((size_t)W, 1);
        while (left > 0) {
            int best = -1;
            u128 best_rem = 0;
            for (int f = W - 1; f >= 0; --f) {
                if (!active[f] || got[f]) continue;
                u128 rem = ((u128)B * w[f]) % S;
                if (best < 0 || rem > best_rem) { best = f; best_rem = rem; }
            }
            if (best < 0) break;
            budget[best] += 1;
            got[best] = 1;
            --left;
        }
        free(got);
        int capped = 0;
        for (int f = 0; f < W; ++f)
            if (active[f] && budget[f] > avail[f]) {
                budget[f] = avail[f];
                active[f] = 0;
                B -= avail[f];
                capped = 1;
            }
        if (!capped) break;
        for (int f = 0; f < W; ++f)
            if (active[f]) budget[f] = 0;
    }
    for (int f = 0; f < W; ++f) budget[f] += floor_q[f];
    free(w);
    free(active);
    free(avail);
    free(floor_q);
    return PO_OK;
}

int po_plan_budget(int kind, double param, int64_t total, int keep_full, int n_frames,
                   const int32_t *avail, int32_t *budget) {
    return po_plan_budget_min(kind, param, total, keep_full, 0, n_frames, avail, budget);
}

/* ------------------------------------------------------------------------
 * Token score (Sec. 3.4, "attention-relevant" retention).  The paper prints no
 * formula; the reading taken is the mean pre-softmax logit of history token j
 * over every current-frame query i and every query head h:
 *     s_j = 1/(Hq Nq) * sum_h sum_i (R(p_i) q_ih) . (R(p_j) k_j,g(h)) / sqrt(d)
 * with g(h) = h div (Hq/Hkv).  Written as that double loop.  A token whose
 * valid byte is 0 (a masked cache position, Eq. 1) scores -infinity.
 * idx == NULL scores tokens 0..n_idx-1; otherwise the listed tokens.
 * ------------------------------------------------------------------------ */
int po_score(const float *k, const int32_t *k_pos, int64_t n_src,
             const float *q, const int32_t *q_pos, int n_q,
             int n_q_heads, int n_kv_heads, int d, double base,
             const uint8_t *valid, const int64_t *idx, int64_t n_idx, double *scores) {
    if (n_q <= 0 || n_q_heads % n_kv_heads) return PO_ERR_ARG;
    int G = n_q_heads / n_kv_heads;
    double *rq = rope_all(q, q_pos, n_q, n_q_heads, d, base);
    if (!rq) return PO_ERR_ARG;
    double inv_sqrt_d = 1.0 / sqrt((double)d);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t e = 0; e < n_idx; ++e) {
        int64_t j = idx ? idx[e] : e;
        if (j < 0 || j >= n_src) { scores[e] = NAN; continue; }
        if (valid && !valid[j]) { scores[e] = -INFINITY; continue; }
        double rk[8 * 256];
        double *rkp = (n_kv_heads * d <= 8 * 256) ? rk : (double *)malloc(sizeof(double) * n_kv_heads * d);
        for (int g = 0; g < n_kv_heads; ++g)
            po_rope(k + ((size_t)j * n_kv_heads + g) * d, k_pos + 4 * j, d, base, rkp + (size_t)g * d);
        double acc = 0.0;
        for (int h = 0; h < n_q_heads; ++h) {
            const double *kk = rkp + (size_t)(h / G) * d;
            for (int i = 0; i < n_q; ++i) {
                const double *qq = rq + ((size_t)i * n_q_heads + h) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += qq[c] * kk[c];
                acc += dot * inv_sqrt_d;
            }
        }
        scores[e] = acc / ((double)n_q_heads * (double)n_q);
        if (rkp != rk) free(rkp);
    }
    free(rq);
    return PO_OK;
}

/* The same score through the pooled query (sum over a head group of the mean
 * rotated query); equal to po_score by linearity.  Kept so that full-size cases
 * can be scored on the host in seconds; tests check the two agree. */
int po_score_pooled(const float *k, const int32_t *k_pos, int64_t n_src,
                    const float *q, const int32_t *q_pos, int n_q,
                    int n_q_heads, int n_kv_heads, int d, double base,
                    const uint8_t *valid, double *scores) {
    if (n_q <= 0 || n_q_heads % n_kv_heads) return PO_ERR_ARG;
    int G = n_q_heads / n_kv_heads;
    double *rq = rope_all(q, q_pos, n_q, n_q_heads, d, base);
    double *pool = (double *)calloc((size_t)n_kv_heads * d, sizeof(double));
    if (!rq || !pool) { free(rq); free(pool); return PO_ERR_ARG; }
    for (int i = 0; i < n_q; ++i)
        for (int h = 0; h < n_q_heads; ++h)
            for (int c = 0; c < d; ++c)
                pool[(size_t)(h / G) * d + c] += rq[((size_t)i * n_q_heads + h) * d + c] / (double)n_q;
    double scale = 1.0 / ((double)n_q_heads * sqrt((double)d));
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_src; ++j) {
        if (valid && !valid[j]) { scores[j] = -INFINITY; continue; }
        double acc = 0.0;
        for (int g = 0; g < n_kv_heads; ++g) {
            double rk[1024];
            po_rope(k + ((size_t)j * n_kv_heads + g) * d, k_pos + 4 * j, d, base, rk);
            for (int c = 0; c < d; ++c) acc += pool[(size_t)g * d + c] * rk[c];
        }
        scores[j] = acc * scale;
    }
    free(rq);
    free(pool);
    return PO_OK;
}

/* ------------------------------------------------------------------------
 * Per-frame selection (Sec. 3.4: each history frame keeps its budgeted number
 * of most relevant tokens).  Order within a frame: higher score first, equal
 * scores by lower index (-0 equals +0).  The first budget[f] tokens of that
 * order are kept and written in ascending index order, frames oldest ->
 * newest.  Indices are global offsets into the history.  NaN is an error.
 * ------------------------------------------------------------------------ */
typedef struct { float s; int32_t i; } po_item;

static int cmp_score_desc_index_asc(const void *a, const void *b) {
    const po_item *x = (const po_item *)a, *y = (const po_item *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);
}

static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int po_select(const float *scores, int n_frames, const int32_t *frame_count, const int32_t *budget,
              int32_t *sel_idx) {
    int64_t base = 0, out = 0;
    for (int f = 0; f < n_frames; ++f) {
        int n = frame_count[f], t = budget[f];
        if (t < 0 || t > n) return PO_ERR_BUDGET;
        po_item *it = (po_item *)malloc(sizeof(po_item) * (size_t)(n > 0 ? n : 1));
        for (int j = 0; j < n; ++j) {
            float s = scores[base + j];
            if (s != s) { free(it); return PO_ERR_NAN; }
            it[j].s = s;
            it[j].i = (int32_t)(base + j);
        }
        qsort(it, (size_t)n, sizeof(po_item), cmp_score_desc_index_asc);
        for (int r = 0; r < t; ++r) sel_idx[out + r] = it[r].i;
        qsort(sel_idx + out, (size_t)t, sizeof(int32_t), cmp_i32);
        out += t;
        base += n;
        free(it);
    }
    return PO_OK;
}

/* ------------------------------------------------------------------------
 * Pack (Fig. 6b: evicted positions are removed, not stored as zeros) with the
 * spatially preserving rebase (Eq. 9): row r of the packed history is source
 * row sel_idx[r]; its (h, w) and tag are copied, its t has delta_t subtracted.
 * ------------------------------------------------------------------------ */
void po_pack(const float *src_k, const float *src_v, const int32_t *src_pos, int row_elems,
             const int32_t *sel_idx, int64_t n_sel, int32_t delta_t,
             float *dst_k, float *dst_v, int32_t *dst_pos) {
    for (int64_t r = 0; r < n_sel; ++r) {
        int64_t s = sel_idx[r];
        for (int c = 0; c < row_elems; ++c) {
            dst_k[(size_t)r * row_elems + c] = src_k[(size_t)s * row_elems + c];
            dst_v[(size_t)r * row_elems + c] = src_v[(size_t)s * row_elems + c];
        }
        dst_pos[4 * r + 0] = src_pos[4 * s + 0] - delta_t;
        dst_pos[4 * r + 1] = src_pos[4 * s + 1];
        dst_pos[4 * r + 2] = src_pos[4 * s + 2];
        dst_pos[4 * r + 3] = src_pos[4 * s + 3];
    }
}

/* ------------------------------------------------------------------------
 * Attention of query rows over a key set (Eq. 2 with every key visible):
 *   out_ih = sum_j softmax_j( (R q_ih).(R k_j,g(h)) / sqrt(d) ) v_j,g(h)
 * The key set is the concatenation of up to three segments (anchors, packed
 * history, current frame).  rows == NULL computes all (i, h); otherwise the
 * listed (i, h) pairs (rows[2e], rows[2e+1]), written to out[e][d], lse[e].
 * lse = log sum_j exp(logit_j) (natural log).
 * ------------------------------------------------------------------------ */
int po_attend(const float *q, const int32_t *q_pos, int n_q, int n_q_heads, int n_kv_heads, int d,
              double base, int n_seg, const float *const *seg_k, const float *const *seg_v,
              const int32_t *const *seg_pos, const int64_t *seg_n,
              const int32_t *rows, int64_t n_rows, double *out, double *lse) {
    if (n_q_heads % n_kv_heads) return PO_ERR_ARG;
    int G = n_q_heads / n_kv_heads;
    int64_t n_k = 0;
    for (int s = 0; s < n_seg; ++s) n_k += seg_n[s];
    if (n_k <= 0) return PO_ERR_ARG;
    /* rotated keys of every segment, concatenated; values by pointer */
    double *rk = (double *)malloc(sizeof(double) * (size_t)n_k * n_kv_heads * d);
    const float **vrow = (const float **)malloc(sizeof(float *) * (size_t)n_k);
    if (!rk || !vrow) { free(rk); free(vrow); return PO_ERR_ARG; }
    int64_t off = 0;
    for (int s = 0; s < n_seg; ++s) {
        double *r = rope_all(seg_k[s], seg_pos[s], seg_n[s], n_kv_heads, d, base);
        memcpy(rk + (size_t)off * n_kv_heads * d, r, sizeof(double) * (size_t)seg_n[s] * n_kv_heads * d);
        free(r);
        for (int64_t j = 0; j < seg_n[s]; ++j) vrow[off + j] = seg_v[s] + (size_t)j * n_kv_heads * d;
        off += seg_n[s];
    }
    int64_t total = rows ? n_rows : (int64_t)n_q * n_q_heads;
    double inv_sqrt_d = 1.0 / sqrt((double)d);
#pragma omp parallel
    {
        double *logit = (double *)malloc(sizeof(double) * (size_t)n_k);
        double rq[1024];
#pragma omp for schedule(dynamic, 8)
        for (int64_t e = 0; e < total; ++e) {
            int i = rows ? rows[2 * e] : (int)(e / n_q_heads);
            int h = rows ? rows[2 * e + 1] : (int)(e % n_q_heads);
            int g = h / G;
            po_rope(q + ((size_t)i * n_q_heads + h) * d, q_pos + 4 * i, d, base, rq);
            double mx = -INFINITY;
            for (int64_t j = 0; j < n_k; ++j) {
                const double *kk = rk + ((size_t)j * n_kv_heads + g) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += rq[c] * kk[c];
                logit[j] = dot * inv_sqrt_d;
                if (logit[j] > mx) mx = logit[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < n_k; ++j) {
                logit[j] = exp(logit[j] - mx);
                denom += logit[j];
            }
            double *o = out + (size_t)e * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j < n_k; ++j) {
                double p = logit[j] / denom;
                const float *vv = vrow[j] + (size_t)g * d;
                for (int c = 0; c < d; ++c) o[c] += p * (double)vv[c];
            }
            if (lse) lse[e] = mx + log(denom);
        }
        free(logit);
    }
    free(rk);
    free(vrow);
    return PO_OK;
}

/* ------------------------------------------------------------------------
 * Attention over a whole sequence with the block mask of Eq. 2: token i may
 * look at token j when block[j] <= block[i] (both directions inside a block,
 * causal between blocks).  out [n][Hq][d].
 * ------------------------------------------------------------------------ */
int po_full_block_causal_attention(const float *q, const float *k, const float *v, const int32_t *pos,
                                   const int32_t *block, int64_t n, int n_q_heads, int n_kv_heads,
                                   int d, double base, double *out) {
    if (n_q_heads % n_kv_heads) return PO_ERR_ARG;
    int G = n_q_heads / n_kv_heads;
    double *rq = rope_all(q, pos, n, n_q_heads, d, base);
    double *rk = rope_all(k, pos, n, n_kv_heads, d, base);
    if (!rq || !rk) { free(rq); free(rk); return PO_ERR_ARG; }
    double inv_sqrt_d = 1.0 / sqrt((double)d);
#pragma omp parallel
    {
        double *logit = (double *)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(dynamic, 8)
        for (int64_t e = 0; e < n * n_q_heads; ++e) {
            int64_t i = e / n_q_heads;
            int h = (int)(e % n_q_heads), g = h / G;
            const double *qq = rq + ((size_t)i * n_q_heads + h) * d;
            double mx = -INFINITY;
            for (int64_t j = 0; j < n; ++j) {
                if (block[j] > block[i]) { logit[j] = -INFINITY; continue; }
                const double *kk = rk + ((size_t)j * n_kv_heads + g) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += qq[c] * kk[c];
                logit[j] = dot * inv_sqrt_d;
                if (logit[j] > mx) mx = logit[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                logit[j] = exp(logit[j] - mx); /* exp(-inf) = 0 for masked keys */
                denom += logit[j];
            }
            double *o = out + (size_t)e * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                double p = logit[j] / denom;
                const float *vv = v + ((size_t)j * n_kv_heads + g) * d;
                for (int c = 0; c < d; ++c) o[c] += p * (double)vv[c];
            }
        }
        free(logit);
    }
    free(rq);
    free(rk);
    return PO_OK;
}

/* ------------------------------------------------------------------------
 * Attention mass of every key (Sec. 3.4: the mean attention score a cached
 * token receives, the quantity "attention-guided" retention ranks by):
 *   mass_j = 1/(n_q*Hq) * sum_i sum_h softmax_j( (R q_ih).(R k_j,g(h)) / sqrt(d) )
 * over the same key set as po_attend (every key visible, Eq. 2).  The masses
 * of all keys sum to one.  mass [n_k], keys in segment order.
 * ------------------------------------------------------------------------ */
int po_attend_mass(const float *q, const int32_t *q_pos, int n_q, int n_q_heads, int n_kv_heads, int d,
                   double base, int n_seg, const float *const *seg_k, const int32_t *const *seg_pos,
                   const int64_t *seg_n, double *mass) {
    if (n_q_heads % n_kv_heads || n_q <= 0) return PO_ERR_ARG;
    int G = n_q_heads / n_kv_heads;
    int64_t n_k = 0;
    for (int s = 0; s < n_seg; ++s) n_k += seg_n[s];
    if (n_k <= 0) return PO_ERR_ARG;
    double *rk = (double *)malloc(sizeof(double) * (size_t)n_k * n_kv_heads * d);
    if (!rk) return PO_ERR_ARG;
    int64_t off = 0;
    for (int s = 0; s < n_seg; ++s) {
        double *r = rope_all(seg_k[s], seg_pos[s], seg_n[s], n_kv_heads, d, base);
        memcpy(rk + (size_t)off * n_kv_heads * d, r, sizeof(double) * (size_t)seg_n[s] * n_kv_heads * d);
        free(r);
        off += seg_n[s];
    }
    double *rq = rope_all(q, q_pos, n_q, n_q_heads, d, base);
    int64_t total = (int64_t)n_q * n_q_heads;
    double *lse = (double *)malloc(sizeof(double) * (size_t)total);
    if (!rq || !lse) { free(rk); free(rq); free(lse); return PO_ERR_ARG; }
    double inv_sqrt_d = 1.0 / sqrt((double)d);
    /* first the normaliser of every query row: lse_e = log sum_j exp(logit_ej) */
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t e = 0; e < total; ++e) {
        int g = (int)(e % n_q_heads) / G;
        const double *qq = rq + (size_t)e * d;
        double mx = -INFINITY;
        for (int64_t j = 0; j < n_k; ++j) {
            const double *kk = rk + ((size_t)j * n_kv_heads + g) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qq[c] * kk[c];
            if (dot * inv_sqrt_d > mx) mx = dot * inv_sqrt_d;
        }
        double denom = 0.0;
        for (int64_t j = 0; j < n_k; ++j) {
            const double *kk = rk + ((size_t)j * n_kv_heads + g) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qq[c] * kk[c];
            denom += exp(dot * inv_sqrt_d - mx);
        }
        lse[e] = mx + log(denom);
    }
    /* then every key's mean probability over the rows, rows in index order */
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t j = 0; j < n_k; ++j) {
        double s = 0.0;
        for (int64_t e = 0; e < total; ++e) {
            int g = (int)(e % n_q_heads) / G;
            const double *qq = rq + (size_t)e * d;
            const double *kk = rk + ((size_t)j * n_kv_heads + g) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qq[c] * kk[c];
            s += exp(dot * inv_sqrt_d - lse[e]);
        }
        mass[j] = s / (double)total;
    }
    free(rq);
    free(lse);
    free(rk);
    return PO_OK;
}
