/*
 * CPU oracle for budgeted KV-cache decode attention (Scissorhands).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step
 * statement of what the method computes, used to check the CUDA library and
 * timed as a reported CPU baseline.  It shares no code with the CUDA path and
 * nothing in the product may call it.
 *
 * Everything is fp64, one unit ((sequence, head) pair) at a time; units are
 * independent (Section 4.1 drops the layer and batch indices), so the only
 * parallelism is an OpenMP loop over units.  No blocking, no fusion.
 *
 * What a step does, in the paper's order (Algorithm 1, with Algorithm 2 as the
 * compression):
 *   1. t <- t+1; the new token's key/value are appended, n <- n+1
 *      (Algorithm 1, "Model update K,V such that n <- n+1").
 *   2. scores over the n cached tokens, the new one included:
 *        alpha_j = exp(scale*<q,K[j]>) / sum_i exp(scale*<q,K[i]>),
 *        out     = sum_j alpha_j V[j]          (estimator of Section 4.1).
 *   3. record: low_j = [alpha_j < 1/t], remembered per cached token together
 *      with the step number (Algorithm 2's loop body, kept online as the
 *      "Overhead Tradeoff" paragraph allows; 1/t is the significance threshold
 *      of Section 3.1 with t the position of the querying token).
 *   4. if the cache is full (n == B): Algorithm 2 -
 *        I_j = number of the last w steps (t-w, t] at which token j was low,
 *        the r most recent tokens are not candidates,
 *        the m candidates first in the order (I descending, position
 *        ascending) are dropped, the rest keep their order; n <- n-m.
 *
 * Readings taken where the paper is silent or garbled (all listed in the
 * design notes of the repository): the record lives per cached token; the
 * window is the last w steps including the current one; ties in I drop the
 * oldest token first; "I[:-r] <- 0" is read as excluding the r newest tokens
 * from eviction; compression triggers when n reaches B so storage never
 * exceeds B rows; the softmax scale defaults to 1/sqrt(d) (caller-supplied).
 *
 * 4-bit store (quant = 1): symmetric int4, groups of 64 along head_dim, one
 * fp16 scale per group, applied to a token when it is appended.  The rounding
 * rule is carried out in IEEE float32 so that it is reproducible:
 *   a = max|x| over the group; sc = fp16(a / 7.0f); sc == 0 -> all codes 0;
 *   code = clamp(rintf(x / (float)sc), -7, 7); stored value = code * sc.
 * The paper only says "4-bit quantization following FlexGen"; the format is
 * the benchmark definition's.
 *
 * Pins (tests/test_oracle_*.py, none of which re-use this file's formulas):
 * full-cache equivalence when B >= T, the renormalisation identity and output
 * bound from the proof of Theorem 4.1, closed forms for equal keys, a
 * from-the-definition brute force with exhaustive subset search on tiny
 * streams, the budget saw-tooth, and an independent scalar int4 quantiser.
 * Which of the alternative readings the authors used is "parity unpinned":
 * the paper prints no numbers that would decide it.
 *
 * Alternative readings (sho_create_reading; the CUDA library implements the
 * defaults only).  Each is what another reader could take from the same lines:
 *   threshold 1: Algorithm 2 literally compares every step of the window with
 *                1/t of the compression step, not of the step itself;
 *   threshold 2: 1/n, the mean of the scores actually normalised over n tokens;
 *   window    1: Algorithm 2's range [t-w, t] taken literally has w+1 steps;
 *   tie       1: a stable ascending argsort cut at [:-m] drops, among equal
 *                counters, the newest tokens instead of the oldest;
 *   trigger   1: Algorithm 1's "if n > B" literally: the cache may hold B+1
 *                tokens for one step, and compression leaves B+1-m.
 *   prompt    1: the prompting stage of Section 2 read as a bulk operation (see
 *                sho_prefill_bulk) instead of the token stream of Definition 4.1.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int n;            /* live tokens */
    double *K, *V;    /* [B][d] stored (already rounded / dequantised) values */
    int *pos;         /* [B] 1-based stream position of each live token, ascending */
    int *h_cnt;       /* [cap] how many (step, low) pairs the token has received */
    int *h_step;      /* [cap][hw] the last hw pairs: step numbers */
    uint8_t *h_low;   /* [cap][hw] the last hw pairs: low flags */
    double *h_alpha;  /* [cap][hw] the last hw pairs: the score itself (threshold reading 1 needs it) */
    double *last_alpha; /* [cap] scores of the step just attended, until sho_record files them */
    double *Q;        /* [w][d] queries of the last w steps (slot = step mod w) */
    int *q_step;      /* [w] step of each stored query, 0 = none */
} unit_t;

typedef struct {
    int U, B, r, w, m, d, quant;
    int cap;          /* rows of storage per unit: B, or B+1 under trigger reading 1 */
    int hw;           /* history entries kept per token: w, or w+1 under window reading 1 */
    int thr_mode, win_plus1, tie_newest, trig_literal;   /* alternative readings, all 0 by default */
    double scale;
    long t;           /* tokens streamed so far */
    unit_t *unit;
} sho_t;

double sho_amb_window(void) { return 1e-6; }

int sho_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void sho_destroy(sho_t *o) {
    if (!o) return;
    if (o->unit) {
        for (int u = 0; u < o->U; ++u) {
            unit_t *x = &o->unit[u];
            free(x->K); free(x->V); free(x->pos); free(x->h_cnt); free(x->h_step); free(x->h_low); free(x->Q); free(x->q_step);
            free(x->h_alpha); free(x->last_alpha);
        }
        free(o->unit);
    }
    free(o);
}

sho_t *sho_create_reading(int U, int B, int r, int w, int m, int d, double scale, int quant,
                          int thr_mode, int win_plus1, int tie_newest, int trig_literal) {
    if (U < 1 || B < 1 || r < 0 || w < 1 || m < 1 || m > B - r || d < 1) return NULL;
    if (quant && d % 64) return NULL;
    if (thr_mode < 0 || thr_mode > 2) return NULL;
    sho_t *o = calloc(1, sizeof *o);
    if (!o) return NULL;
    o->U = U; o->B = B; o->r = r; o->w = w; o->m = m; o->d = d; o->quant = quant; o->scale = scale;
    o->thr_mode = thr_mode; o->win_plus1 = !!win_plus1; o->tie_newest = !!tie_newest; o->trig_literal = !!trig_literal;
    o->cap = B + o->trig_literal;
    o->hw = w + o->win_plus1;
    o->t = 0;
    o->unit = calloc((size_t)U, sizeof(unit_t));
    if (!o->unit) { free(o); return NULL; }
    for (int u = 0; u < U; ++u) {
        unit_t *x = &o->unit[u];
        x->n = 0;
        const size_t cap = (size_t)o->cap, hw = (size_t)o->hw;
        x->K = calloc(cap * d, sizeof(double));
        x->V = calloc(cap * d, sizeof(double));
        x->pos = calloc(cap, sizeof(int));
        x->h_cnt = calloc(cap, sizeof(int));
        x->h_step = calloc(cap * hw, sizeof(int));
        x->h_low = calloc(cap * hw, 1);
        x->h_alpha = calloc(cap * hw, sizeof(double));
        x->last_alpha = calloc(cap, sizeof(double));
        x->Q = calloc((size_t)w * d, sizeof(double));
        x->q_step = calloc((size_t)w, sizeof(int));
        if (!x->K || !x->V || !x->pos || !x->h_cnt || !x->h_step || !x->h_low || !x->h_alpha || !x->last_alpha || !x->Q ||
            !x->q_step) { sho_destroy(o); return NULL; }
    }
    return o;
}

sho_t *sho_create(int U, int B, int r, int w, int m, int d, double scale, int quant) {
    return sho_create_reading(U, B, r, w, m, d, scale, quant, 0, 0, 0, 0);
}

int sho_cap(const sho_t *o) { return o->cap; }

/* int4 group-64 round trip of one row, float32 rule stated in the header. */
static void quant_row(const double *x, int d, double *stored, int8_t *codes, float *scales) {
    for (int g0 = 0; g0 < d; g0 += 64) {
        float a = 0.0f;
        for (int i = g0; i < g0 + 64; ++i) {
            float xi = fabsf((float)x[i]);
            if (xi > a) a = xi;
        }
        _Float16 sc16 = (_Float16)(a / 7.0f);
        float sc = (float)sc16;
        if (scales) scales[g0 / 64] = sc;
        for (int i = g0; i < g0 + 64; ++i) {
            float c = 0.0f;
            if (sc != 0.0f) {
                c = rintf((float)x[i] / sc);
                if (c > 7.0f) c = 7.0f;
                if (c < -7.0f) c = -7.0f;
            }
            if (codes) codes[i] = (int8_t)c;
            stored[i] = (double)c * (double)sc;
        }
    }
}

/* Stand-alone quantiser for tests: x[rows][d] -> stored values, codes, scales. */
void sho_quantize(const double *x, int rows, int d, double *stored, int8_t *codes, float *scales) {
    for (int i = 0; i < rows; ++i)
        quant_row(x + (size_t)i * d, d, stored + (size_t)i * d, codes ? codes + (size_t)i * d : NULL,
                  scales ? scales + (size_t)i * (d / 64) : NULL);
}

int sho_n(const sho_t *o) { return o->unit[0].n; }
long sho_t_now(const sho_t *o) { return o->t; }
/* Is a compression due?  n == B by default (so n < B holds between steps, Definition 4.1);
 * under trigger reading 1, Algorithm 1's literal n > B, i.e. n == B+1. */
int sho_full(const sho_t *o) { return o->unit[0].n == o->cap; }

/*
 * Steps 1 and 2 (and the comparison of step 3, not yet recorded).
 * q, k, v: [U][d].  out: [U][d].  alpha: [U][cap] (first n entries of each row
 * valid; cap = sho_cap() = B unless trigger reading 1).  low, amb: [U][cap] bytes; amb_j = 1 when alpha_j lies within
 * sho_amb_window() of the threshold, where an fp32 implementation may
 * legitimately decide the comparison the other way.
 * Returns -1 if the cache is already full (the caller forgot to compress).
 */
int sho_attend(sho_t *o, const double *q, const double *k, const double *v,
               double *out, double *alpha, uint8_t *low, uint8_t *amb) {
    const int B = o->cap, d = o->d;
    if (o->unit[0].n >= B) return -1;
    o->t += 1;
    const long t = o->t;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < o->U; ++u) {
        unit_t *x = &o->unit[u];
        /* 1. append */
        int j = x->n;
        if (o->quant) {
            quant_row(k + (size_t)u * d, d, x->K + (size_t)j * d, NULL, NULL);
            quant_row(v + (size_t)u * d, d, x->V + (size_t)j * d, NULL, NULL);
        } else {
            memcpy(x->K + (size_t)j * d, k + (size_t)u * d, sizeof(double) * d);
            memcpy(x->V + (size_t)j * d, v + (size_t)u * d, sizeof(double) * d);
        }
        x->pos[j] = (int)t;
        x->h_cnt[j] = 0;
        x->n = j + 1;
        const int n = x->n;
        /* 2. scores and output */
        double *a = alpha + (size_t)u * B;
        const double *qu = q + (size_t)u * d;
        memcpy(x->Q + (size_t)(t % o->w) * d, qu, sizeof(double) * d);   /* kept for the recompute variant */
        x->q_step[t % o->w] = (int)t;
        double smax = -INFINITY;
        for (j = 0; j < n; ++j) {
            double s = 0.0;
            for (int i = 0; i < d; ++i) s += qu[i] * x->K[(size_t)j * d + i];
            s *= o->scale;
            a[j] = s;
            if (s > smax) smax = s;
        }
        double L = 0.0;
        for (j = 0; j < n; ++j) { a[j] = exp(a[j] - smax); L += a[j]; }
        for (j = 0; j < n; ++j) a[j] /= L;
        for (j = n; j < B; ++j) a[j] = 0.0;
        double *ou = out + (size_t)u * d;
        for (int i = 0; i < d; ++i) ou[i] = 0.0;
        for (j = 0; j < n; ++j)
            for (int i = 0; i < d; ++i) ou[i] += a[j] * x->V[(size_t)j * d + i];
        /* 3. the comparison against 1/t (threshold reading 2: against 1/n, the mean score) */
        const double thr = o->thr_mode == 2 ? 1.0 / (double)n : 1.0 / (double)t;
        for (j = 0; j < n; ++j) x->last_alpha[j] = a[j];
        for (j = 0; j < B; ++j) {
            low[(size_t)u * B + j] = (j < n) && (a[j] < thr);
            amb[(size_t)u * B + j] = (j < n) && (fabs(a[j] - thr) <= sho_amb_window());
        }
    }
    return 0;
}

/* Step 3: remember this step's low flags, [U][B], for every live token. */
void sho_record(sho_t *o, const uint8_t *low) {
    const int B = o->cap, w = o->hw;
    const long t = o->t;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < o->U; ++u) {
        unit_t *x = &o->unit[u];
        for (int j = 0; j < x->n; ++j) {
            int slot = x->h_cnt[j] % w;
            x->h_step[(size_t)j * w + slot] = (int)t;
            x->h_low[(size_t)j * w + slot] = low[(size_t)u * B + j] ? 1 : 0;
            x->h_alpha[(size_t)j * w + slot] = x->last_alpha[j];
            x->h_cnt[j] += 1;
        }
    }
}

/* I_j of Algorithm 2 at the current t: low flags among steps (t-w, t] (window reading 1: [t-w, t]).
 * Threshold reading 1 decides every step of the window against 1/t of the present step instead of
 * using the flag taken at that step. */
static int counter_of(const sho_t *o, const unit_t *x, int j) {
    const int hw = o->hw;
    const long first = o->t - o->w + (o->win_plus1 ? 0 : 1);     /* first step of the window */
    int have = x->h_cnt[j] < hw ? x->h_cnt[j] : hw;
    int c = 0;
    for (int s = 0; s < have; ++s) {
        if ((long)x->h_step[(size_t)j * hw + s] < first) continue;
        if (o->thr_mode == 1) c += x->h_alpha[(size_t)j * hw + s] < 1.0 / (double)o->t;
        else c += x->h_low[(size_t)j * hw + s] ? 1 : 0;
    }
    return c;
}

/* Counters of all live tokens, [U][cap] (entries past n are 0). */
void sho_counters(const sho_t *o, int *I) {
    for (int u = 0; u < o->U; ++u) {
        const unit_t *x = &o->unit[u];
        for (int j = 0; j < o->cap; ++j) I[(size_t)u * o->cap + j] = j < x->n ? counter_of(o, x, j) : 0;
    }
}

/* Positions of all live tokens, [U][cap] (entries past n are 0). */
void sho_positions(const sho_t *o, int *pos) {
    for (int u = 0; u < o->U; ++u) {
        const unit_t *x = &o->unit[u];
        for (int j = 0; j < o->cap; ++j) pos[(size_t)u * o->cap + j] = j < x->n ? x->pos[j] : 0;
    }
}

/* Stored K and V rows of one unit, [cap][d] each (rows past n are 0). */
void sho_cache(const sho_t *o, int u, double *K, double *V) {
    const unit_t *x = &o->unit[u];
    memset(K, 0, sizeof(double) * o->cap * o->d);
    memset(V, 0, sizeof(double) * o->cap * o->d);
    memcpy(K, x->K, sizeof(double) * x->n * o->d);
    memcpy(V, x->V, sizeof(double) * x->n * o->d);
}

/*
 * The selection of Algorithm 2 on given counters: tokens are in position
 * order, the last r are protected, and m times over the not-yet-chosen
 * candidate with the largest counter is taken, the oldest among equals.
 * evict[] receives the chosen indices in the order chosen.
 */
static void select_tie(const int *I, int n, int r, int m, int *evict, int tie_newest) {
    uint8_t *gone = calloc((size_t)n, 1);
    for (int e = 0; e < m; ++e) {
        int best = -1;
        for (int j = 0; j < n - r; ++j) {
            if (gone[j]) continue;
            /* strict >: the earlier index wins ties; tie reading 1 (>=): the later one does */
            if (best < 0 || I[j] > I[best] || (tie_newest && I[j] == I[best])) best = j;
        }
        evict[e] = best;
        if (best >= 0) gone[best] = 1;
    }
    free(gone);
}

void sho_select(const int *I, int n, int r, int m, int *evict) { select_tie(I, n, r, m, evict, 0); }
void sho_select_newest_first(const int *I, int n, int r, int m, int *evict) { select_tie(I, n, r, m, evict, 1); }

/* Algorithm 2 on one unit as it stands: counters at the present t, the r newest protected, the m
 * candidates first in the order dropped, the rest moved up in order.  evicted_pos: [m] or NULL. */
static void compress_unit(const sho_t *o, unit_t *x, int m, int r, int *evicted_pos) {
    const int d = o->d, w = o->hw;
    const int n = x->n;
    int *I = malloc(sizeof(int) * n);
    int *ev = malloc(sizeof(int) * m);
    uint8_t *drop = calloc((size_t)n, 1);
    for (int j = 0; j < n; ++j) I[j] = counter_of(o, x, j);
    select_tie(I, n, r, m, ev, o->tie_newest);
    for (int e = 0; e < m; ++e) drop[ev[e]] = 1;
    int keep = 0, ne = 0;
    for (int j = 0; j < n; ++j) {
        if (drop[j]) {
            if (evicted_pos) evicted_pos[ne] = x->pos[j];
            ne += 1;
            continue;
        }
        if (keep != j) {
            memcpy(x->K + (size_t)keep * d, x->K + (size_t)j * d, sizeof(double) * d);
            memcpy(x->V + (size_t)keep * d, x->V + (size_t)j * d, sizeof(double) * d);
            x->pos[keep] = x->pos[j];
            x->h_cnt[keep] = x->h_cnt[j];
            memcpy(x->h_step + (size_t)keep * w, x->h_step + (size_t)j * w, sizeof(int) * w);
            memcpy(x->h_low + (size_t)keep * w, x->h_low + (size_t)j * w, w);
            memcpy(x->h_alpha + (size_t)keep * w, x->h_alpha + (size_t)j * w, sizeof(double) * w);
        }
        keep += 1;
    }
    x->n = keep;
    free(I); free(ev); free(drop);
}

/*
 * Step 4: Algorithm 2 when the cache is full.  evicted_pos: [U][m] stream
 * positions dropped, ascending (untouched when nothing happens).
 * Returns the number of tokens dropped per unit (m or 0).
 */
int sho_compress(sho_t *o, int *evicted_pos) {
    if (o->unit[0].n < o->cap) return 0;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < o->U; ++u)
        compress_unit(o, &o->unit[u], o->m, o->r, evicted_pos ? evicted_pos + (size_t)u * o->m : NULL);
    return o->m;
}

/*
 * The prompting stage read as a bulk operation (Section 2: the prompt's keys and values are computed
 * and cached in full before generation starts) instead of Definition 4.1's token stream: `src` has
 * streamed the whole prompt under a budget that never made it compress, so its outputs are full causal
 * attention and its record holds the prompt's last w steps.  The prompt's cache is then brought under
 * dst's budget by Algorithm 2 applied as often as needed - same record, m tokens per round, the r
 * newest protected, until fewer than B tokens remain (trigger reading 1: no more than B) - and what
 * survives, with its record, becomes dst's cache; dst continues at t = src's t.
 * src and dst must agree in U, d, w, quant and readings; dst must be fresh.  Returns the number of
 * rounds, or -1 on a mismatch.  src is left compressed.
 */
int sho_import_compressed(sho_t *dst, sho_t *src) {
    if (dst->U != src->U || dst->d != src->d || dst->w != src->w || dst->hw != src->hw || dst->quant != src->quant ||
        dst->thr_mode != src->thr_mode || dst->tie_newest != src->tie_newest || dst->t != 0)
        return -1;
    const int stop = dst->cap;            /* compress while n >= stop */
    int rounds = 0;
    while (src->unit[0].n >= stop) {
        if (src->unit[0].n - dst->r < dst->m) return -1;
#pragma omp parallel for schedule(static)
        for (int u = 0; u < src->U; ++u) compress_unit(src, &src->unit[u], dst->m, dst->r, NULL);
        rounds += 1;
    }
    const int d = dst->d, hw = dst->hw;
    for (int u = 0; u < src->U; ++u) {
        unit_t *a = &dst->unit[u];
        const unit_t *b = &src->unit[u];
        a->n = b->n;
        memcpy(a->K, b->K, sizeof(double) * b->n * d);
        memcpy(a->V, b->V, sizeof(double) * b->n * d);
        memcpy(a->pos, b->pos, sizeof(int) * b->n);
        memcpy(a->h_cnt, b->h_cnt, sizeof(int) * b->n);
        memcpy(a->h_step, b->h_step, sizeof(int) * b->n * hw);
        memcpy(a->h_low, b->h_low, (size_t)b->n * hw);
        memcpy(a->h_alpha, b->h_alpha, sizeof(double) * b->n * hw);
        memcpy(a->Q, b->Q, sizeof(double) * dst->w * d);
        memcpy(a->q_step, b->q_step, sizeof(int) * dst->w);
    }
    dst->t = src->t;
    return rounds;
}

/*
 * The record as Algorithm 2 states it, computed at compression time ("an extra
 * attention computation ... to collect the importance measurements over a
 * history window", Section 4.1, Overhead Tradeoff) instead of being kept
 * online: every query of the last w steps (t-w, t] is scored again against the
 * cache as it is now, restricted to the tokens that already existed at that
 * query's step (pos <= step: attention is causal), and compared with 1/step.
 * Tokens evicted since then are gone, so the scores are normalised over the
 * survivors.  alpha, low, amb: [U][w][cap], row (step mod w); steps: [w] (0 = no query).
 */
void sho_recount(const sho_t *o, double *alpha, uint8_t *low, uint8_t *amb, int *steps) {
    const int B = o->cap, d = o->d, w = o->w;
    for (int s = 0; s < w; ++s) {
        int st = o->unit[0].q_step[s];
        steps[s] = (st > 0 && (long)st > o->t - w && (long)st <= o->t) ? st : 0;
    }
#pragma omp parallel for schedule(static)
    for (int u = 0; u < o->U; ++u) {
        const unit_t *x = &o->unit[u];
        for (int s = 0; s < w; ++s) {
            double *a = alpha + ((size_t)u * w + s) * B;
            uint8_t *lo = low + ((size_t)u * w + s) * B, *am = amb + ((size_t)u * w + s) * B;
            for (int j = 0; j < B; ++j) { a[j] = 0.0; lo[j] = 0; am[j] = 0; }
            const int st = steps[s];
            if (!st) continue;
            const double *qu = x->Q + (size_t)s * d;
            int nv = 0;                                   /* tokens that existed at step st (positions ascend) */
            while (nv < x->n && x->pos[nv] <= st) ++nv;
            if (!nv) continue;
            double smax = -INFINITY, L = 0.0;
            for (int j = 0; j < nv; ++j) {
                double sc = 0.0;
                for (int i = 0; i < d; ++i) sc += qu[i] * x->K[(size_t)j * d + i];
                a[j] = sc * o->scale;
                if (a[j] > smax) smax = a[j];
            }
            for (int j = 0; j < nv; ++j) { a[j] = exp(a[j] - smax); L += a[j]; }
            const double thr = 1.0 / (double)st;
            for (int j = 0; j < nv; ++j) {
                a[j] /= L;
                lo[j] = a[j] < thr;
                am[j] = fabs(a[j] - thr) <= sho_amb_window();
            }
        }
    }
}

/* Replace every live token's history by the given recomputed flags
 * ([U][w][cap], row = step mod w, steps as returned by sho_recount). */
void sho_set_record(sho_t *o, const uint8_t *low, const int *steps) {
    const int B = o->cap, w = o->w, hw = o->hw;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < o->U; ++u) {
        unit_t *x = &o->unit[u];
        for (int j = 0; j < x->n; ++j) {
            x->h_cnt[j] = 0;
            for (long st = o->t - w + 1; st <= o->t; ++st) {     /* ascending steps */
                if (st < 1) continue;
                const int s = (int)(st % w);
                if (steps[s] != (int)st || x->pos[j] > st) continue;
                const int slot = x->h_cnt[j] % hw;
                x->h_step[(size_t)j * hw + slot] = (int)st;
                x->h_low[(size_t)j * hw + slot] = low[((size_t)u * w + s) * B + j] ? 1 : 0;
                x->h_alpha[(size_t)j * hw + slot] = low[((size_t)u * w + s) * B + j] ? 0.0 : 1.0;   /* only the flag is known */
                x->h_cnt[j] += 1;
            }
        }
    }
}

/* One whole step for callers that do not intervene: 1-4 above. */
int sho_step(sho_t *o, const double *q, const double *k, const double *v, double *out,
             double *alpha, uint8_t *low, uint8_t *amb, int *evicted_pos) {
    int rc = sho_attend(o, q, k, v, out, alpha, low, amb);
    if (rc) return rc;
    sho_record(o, low);
    return sho_compress(o, evicted_pos);
}
