/*
 * MorphKV reference oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, fp64, single-threaded CPU statement of what one MorphKV
 * "unit" (one layer x batch row x KV head, serving G grouped query heads)
 * computes per decode step, written from the paper's definitions:
 *
 *   Eq. 1          causal soft-max attention of the new query over the cache
 *   Eq. 4, 5, 6    fused score F[k] of an older token k from the attention
 *                  weights that the R window tokens assigned to it
 *   Algorithm 1    S_r = sum over the GQA group of AW_r, F = f(S_r ...),
 *                  next cache = Top_C(F) united with the window
 *   Eq. 7          the cache stays at C + R entries
 *   Implementation section ("lightweight KV cache extension"): the attention
 *                  profile of each window token is STORED when the token is
 *                  generated; rows are appended and the oldest discarded.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * this file.  It shares no code, header, table or helper with the CUDA path.
 *
 * Readings of points the paper leaves open (each also listed in the design
 * notes of the repository):
 *   - attention is self-inclusive: token t attends to the cache and to itself;
 *   - after step t the window is {t, ..., t-R+1}; the token t-R that just left
 *     the window joins the C distant tokens as a candidate, so exactly one
 *     token is evicted per step once the cache is full;
 *   - AW_r[k] is the weight token r assigned WHEN IT WAS GENERATED (stored);
 *     mode `recompute` re-derives the same number from the stored query and
 *     that row's frozen soft-max statistics (max, denominator) instead;
 *   - GQA: sum over the group first, then sum/max over the window, for both
 *     fusions;
 *   - scale 1/sqrt(head_dim);
 *   - ties in Top_C: the lower position is kept;
 *   - prefill: one application of Algorithm 1 with the whole prompt as G_i and
 *     the last min(R,P) prompt tokens (full causal profiles) as the window;
 *   - evict_interval T > 1 (coarse-grained eviction appendix): the policy runs
 *     on every T-th decode step only; the cache peaks at C + R + T - 1;
 *   - norm_mode CURRENT (the other reading of Eq. 4's AW_r): each window row's
 *     stored weights are renormalised over the tokens that are still cached
 *     when the scores are taken (a row never saw tokens newer than itself, so
 *     this is causal inside the window); the default FROZEN uses them as stored.
 *
 * Pinned by tests/test_oracle_pins.py (full-attention special case against an
 * independent causal attention, the paper's worked 0.3/0.05 example, cache
 * invariants, brute-force ranking on tiny inputs, R=1 and G=1 reductions,
 * stored == recompute, shift / permutation / scaling metamorphic checks, and
 * for evict_interval > 1 which tokens are dropped on which steps against a
 * dictionary restatement that ranks all candidates with a plain sort).
 * The readings themselves (window membership, stored weights, prefill
 * procedure) have no printed value in the paper to pin them: parity unpinned
 * for those choices.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

enum { ORA_SUM = 0, ORA_MAX = 1 };

typedef struct ora_unit {
    int G, d, C, R, fusion, T, recompute;
    int norm_current; /* 1: renormalise each window row over the tokens still cached (see header) */
    int cap;        /* physical slots: C + R + T (one transient slot for the new token) */
    int n;          /* occupied slots */
    long t;         /* position of the next token to decode */
    long steps;     /* decode steps taken */
    long *pos;      /* [cap] position held by a slot, -1 = free */
    double *K, *V;  /* [cap][d] */
    /* window rows: R + 1 physical rows so that "append, then discard the oldest" is literal */
    int nw;         /* rows in use */
    long *wpos;     /* [R+1] position of a row, -1 = free */
    double *A;      /* [R+1][G][cap] stored profile, indexed by slot (stored mode) */
    double *Q;      /* [R+1][G][d]   window queries   (recompute mode) */
    double *wm, *wl;/* [R+1][G]      frozen max / denominator of the row's soft-max */
    /* results of the last scoring, for the harness */
    int n_cand;
    long *cand_pos;   /* [cap] */
    double *cand_F;   /* [cap] */
    int n_evicted;
    long *evicted;    /* [cap] */
    double kth, k1th; /* C-th and (C+1)-th largest fused score at the last selection */
} ora_unit;

ora_unit *ora_create(int G, int d, int C, int R, int fusion, int evict_interval, int recompute)
{
    if (G < 1 || d < 1 || C < 1 || R < 1 || evict_interval < 1) return NULL;
    if (fusion != ORA_SUM && fusion != ORA_MAX) return NULL;
    ora_unit *u = (ora_unit *)calloc(1, sizeof(*u));
    if (!u) return NULL;
    u->G = G; u->d = d; u->C = C; u->R = R; u->fusion = fusion; u->T = evict_interval;
    u->recompute = recompute;
    u->cap = C + R + evict_interval;
    size_t cap = (size_t)u->cap, rows = (size_t)R + 1;
    u->pos = (long *)malloc(cap * sizeof(long));
    u->K = (double *)calloc(cap * d, sizeof(double));
    u->V = (double *)calloc(cap * d, sizeof(double));
    u->wpos = (long *)malloc(rows * sizeof(long));
    u->A = (double *)calloc(rows * G * cap, sizeof(double));
    u->Q = (double *)calloc(rows * G * d, sizeof(double));
    u->wm = (double *)calloc(rows * G, sizeof(double));
    u->wl = (double *)calloc(rows * G, sizeof(double));
    u->cand_pos = (long *)malloc(cap * sizeof(long));
    u->cand_F = (double *)malloc(cap * sizeof(double));
    u->evicted = (long *)malloc(cap * sizeof(long));
    for (size_t i = 0; i < cap; ++i) u->pos[i] = -1;
    for (size_t i = 0; i < rows; ++i) u->wpos[i] = -1;
    return u;
}

void ora_destroy(ora_unit *u)
{
    if (!u) return;
    free(u->pos); free(u->K); free(u->V); free(u->wpos); free(u->A); free(u->Q);
    free(u->wm); free(u->wl); free(u->cand_pos); free(u->cand_F); free(u->evicted);
    free(u);
}

/* 0 = FROZEN (default), 1 = CURRENT */
void ora_set_norm_mode(ora_unit *u, int current) { if (u) u->norm_current = current != 0; }

static int free_slot(const ora_unit *u)
{
    for (int s = 0; s < u->cap; ++s) if (u->pos[s] < 0) return s;
    return -1;
}

static int free_row(const ora_unit *u)
{
    for (int r = 0; r <= u->R; ++r) if (u->wpos[r] < 0) return r;
    return -1;
}

static int in_window(const ora_unit *u, long p)
{
    for (int r = 0; r <= u->R; ++r) if (u->wpos[r] == p) return 1;
    return 0;
}

static double dot(const double *a, const double *b, int d)
{
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += a[i] * b[i];
    return s;
}

/* AW_r^g[k]: the weight window row `r` (head g) assigned to the token in `slot`
 * when r was generated (0 for a token newer than r: it was not there). */
static double profile_weight(const ora_unit *u, int r, int g, int slot)
{
    if (u->pos[slot] > u->wpos[r]) return 0.0;
    if (!u->recompute) return u->A[((size_t)r * u->G + g) * u->cap + slot];
    const double *q = u->Q + ((size_t)r * u->G + g) * u->d;
    double s = dot(q, u->K + (size_t)slot * u->d, u->d) / sqrt((double)u->d);
    return exp(s - u->wm[r * u->G + g]) / u->wl[r * u->G + g];
}

typedef struct { double F; long pos; int slot; } cand_t;

static int cand_cmp(const void *a, const void *b)
{
    const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
    if (x->F > y->F) return -1;            /* larger fused score first */
    if (x->F < y->F) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);  /* ties: lower position first (kept) */
}

static void evict_slot(ora_unit *u, int slot)
{
    u->evicted[u->n_evicted++] = u->pos[slot];
    u->pos[slot] = -1;
    u->n--;
    for (int r = 0; r <= u->R; ++r)
        for (int g = 0; g < u->G; ++g)
            u->A[((size_t)r * u->G + g) * u->cap + slot] = 0.0;
}

/*
 * Algorithm 1 + Eq. 7 on the current state: candidates are the cached tokens
 * outside the window; S_r[k] = sum_g AW_r^g[k]; F[k] = sum_r or max_r S_r[k];
 * keep the C best by (F descending, position ascending).  If `forced` is
 * given, those positions are evicted instead of the oracle's own choice (the
 * harness uses this to follow a legitimate near-tie decision of the device).
 * Returns 0, or -1 if a forced position is not a candidate.
 */
static int score_and_select(ora_unit *u, const long *forced, int n_forced)
{
    cand_t *c = (cand_t *)malloc((size_t)u->cap * sizeof(cand_t));
    int nc = 0;
    /* CURRENT: what is left of each row's weight mass on the tokens still cached (1 under FROZEN) */
    double *mass = (double *)malloc((size_t)(u->R + 1) * u->G * sizeof(double));
    for (int r = 0; r <= u->R; ++r)
        for (int g = 0; g < u->G; ++g) {
            double m = 1.0;
            if (u->norm_current && u->wpos[r] >= 0) {
                m = 0.0;
                for (int s = 0; s < u->cap; ++s) if (u->pos[s] >= 0) m += profile_weight(u, r, g, s);
            }
            mass[r * u->G + g] = m;
        }
    for (int s = 0; s < u->cap; ++s) {
        if (u->pos[s] < 0 || in_window(u, u->pos[s])) continue;
        double F = 0.0;
        int first = 1;
        for (int r = 0; r <= u->R; ++r) {
            if (u->wpos[r] < 0) continue;
            double S = 0.0;                                   /* GQA aggregate */
            for (int g = 0; g < u->G; ++g) S += profile_weight(u, r, g, s) / mass[r * u->G + g];
            if (u->fusion == ORA_SUM) F += S;                 /* Eq. 5 */
            else if (first || S > F) F = S;                   /* Eq. 6 */
            first = 0;
        }
        c[nc].F = F; c[nc].pos = u->pos[s]; c[nc].slot = s; ++nc;
    }
    free(mass);
    qsort(c, (size_t)nc, sizeof(cand_t), cand_cmp);
    u->n_cand = nc;
    for (int i = 0; i < nc; ++i) { u->cand_pos[i] = c[i].pos; u->cand_F[i] = c[i].F; }
    u->kth = nc >= u->C ? c[u->C - 1].F : NAN;
    u->k1th = nc > u->C ? c[u->C].F : NAN;
    int rc = 0;
    if (nc > u->C) {
        if (n_forced > 0) {
            for (int f = 0; f < n_forced && rc == 0; ++f) {
                int hit = -1;
                for (int i = 0; i < nc; ++i) if (c[i].pos == forced[f]) hit = i;
                if (hit < 0) rc = -1; else evict_slot(u, c[hit].slot);
            }
        } else {
            for (int i = u->C; i < nc; ++i) evict_slot(u, c[i].slot);
        }
    }
    free(c);
    return rc;
}

/*
 * Prefill with P prompt tokens: k, v [P][d], q_window [G][Rw][d] (queries of
 * the last Rw = min(R, P) prompt positions, oldest first).  `forced` /
 * `n_forced`: optional list of the prompt positions to evict instead of the
 * oracle's own choice (the harness uses it to follow a legitimate near-tie
 * decision of the device); it must name exactly as many candidates as the
 * policy evicts.  The ranking of all candidates is kept for ora_last_scores.
 */
int ora_prefill_forced(ora_unit *u, const double *k, const double *v, const double *q_window, int P,
                       const long *forced, int n_forced)
{
    if (!u || P < 1 || u->t != 0) return -1;
    const int G = u->G, d = u->d, R = u->R;
    const int Rw = P < R ? P : R;
    const double scale = 1.0 / sqrt((double)d);
    /* full causal profiles of the window rows over ALL prompt keys (Eq. 1) */
    double *Afull = (double *)calloc((size_t)Rw * G * P, sizeof(double));
    double *m = (double *)malloc((size_t)Rw * G * sizeof(double));
    double *l = (double *)malloc((size_t)Rw * G * sizeof(double));
    for (int i = 0; i < Rw; ++i) {
        const long r = P - Rw + i;
        for (int g = 0; g < G; ++g) {
            const double *q = q_window + ((size_t)g * Rw + i) * d;
            double *a = Afull + ((size_t)i * G + g) * P;
            double mx = -INFINITY, den = 0.0;
            for (long j = 0; j <= r; ++j) { a[j] = dot(q, k + (size_t)j * d, d) * scale; if (a[j] > mx) mx = a[j]; }
            for (long j = 0; j <= r; ++j) { a[j] = exp(a[j] - mx); den += a[j]; }
            for (long j = 0; j <= r; ++j) a[j] /= den;
            m[i * G + g] = mx; l[i * G + g] = den;
        }
    }
    /* fused score of every older prompt token (Alg. 1), then Top_C */
    const int ncand = P - Rw;
    char *keep = (char *)malloc((size_t)P);
    memset(keep, 1, (size_t)P);
    u->n_evicted = 0; u->n_cand = 0; u->kth = NAN; u->k1th = NAN;
    if (ncand > u->C) {
        cand_t *c = (cand_t *)malloc((size_t)ncand * sizeof(cand_t));
        for (int j = 0; j < ncand; ++j) {
            double F = 0.0;
            for (int i = 0; i < Rw; ++i) {
                double S = 0.0;
                for (int g = 0; g < G; ++g) S += Afull[((size_t)i * G + g) * P + j];
                if (u->fusion == ORA_SUM) F += S; else if (i == 0 || S > F) F = S;
            }
            c[j].F = F; c[j].pos = j; c[j].slot = j;
        }
        qsort(c, (size_t)ncand, sizeof(cand_t), cand_cmp);
        u->kth = c[u->C - 1].F; u->k1th = c[u->C].F;
        /* the prompt may hold more candidates than the cache has slots: grow the read-back arrays */
        if (ncand > u->cap) {
            u->cand_pos = (long *)realloc(u->cand_pos, (size_t)ncand * sizeof(long));
            u->cand_F = (double *)realloc(u->cand_F, (size_t)ncand * sizeof(double));
        }
        u->n_cand = ncand;
        for (int j = 0; j < ncand; ++j) { u->cand_pos[j] = c[j].pos; u->cand_F[j] = c[j].F; }
        if (n_forced > 0) {
            int bad = n_forced != ncand - u->C;
            for (int f = 0; f < n_forced && !bad; ++f) {
                if (forced[f] < 0 || forced[f] >= ncand || !keep[forced[f]]) bad = 1; else keep[forced[f]] = 0;
            }
            if (bad) { free(c); free(Afull); free(m); free(l); free(keep); return -3; }
        } else {
            for (int j = u->C; j < ncand; ++j) keep[c[j].pos] = 0;
        }
        free(c);
    }
    /* build the cache and the stored profile rows of the window */
    int s = 0;
    for (long j = 0; j < P; ++j) {
        if (!keep[j]) continue;
        u->pos[s] = j;
        memcpy(u->K + (size_t)s * d, k + (size_t)j * d, (size_t)d * sizeof(double));
        memcpy(u->V + (size_t)s * d, v + (size_t)j * d, (size_t)d * sizeof(double));
        for (int i = 0; i < Rw; ++i)
            for (int g = 0; g < G; ++g)
                u->A[((size_t)i * G + g) * u->cap + s] = Afull[((size_t)i * G + g) * P + j];
        ++s;
    }
    u->n = s;
    for (int i = 0; i < Rw; ++i) {
        u->wpos[i] = P - Rw + i;
        for (int g = 0; g < G; ++g) {
            memcpy(u->Q + ((size_t)i * G + g) * d, q_window + ((size_t)g * Rw + i) * d, (size_t)d * sizeof(double));
            u->wm[i * G + g] = m[i * G + g];
            u->wl[i * G + g] = l[i * G + g];
        }
    }
    u->nw = Rw;
    u->t = P;
    free(Afull); free(m); free(l); free(keep);
    return 0;
}

int ora_prefill(ora_unit *u, const double *k, const double *v, const double *q_window, int P)
{
    return ora_prefill_forced(u, k, v, q_window, P, NULL, 0);
}

/*
 * One decode step: q [G][d], k_new, v_new [d] -> out [G][d].
 * `forced`/`n_forced`: optional eviction choice imposed by the harness.
 * Returns 0 on success.
 */
int ora_step(ora_unit *u, const double *q, const double *k_new, const double *v_new, double *out,
             const long *forced, int n_forced)
{
    if (!u || u->t < 1) return -1;
    const int G = u->G, d = u->d, R = u->R;
    const double scale = 1.0 / sqrt((double)d);
    const long t = u->t;

    /* the new token takes a slot first so that "the cache and itself" is one set J (Eq. 1) */
    const int ns = free_slot(u);
    const int nr = free_row(u);
    if (ns < 0 || nr < 0) return -2;
    u->pos[ns] = t;
    memcpy(u->K + (size_t)ns * d, k_new, (size_t)d * sizeof(double));
    memcpy(u->V + (size_t)ns * d, v_new, (size_t)d * sizeof(double));
    u->n++;

    /* 1. attend (Eq. 1) and 2. append the profile row of token t */
    u->wpos[nr] = t;
    u->nw++;
    double *a = (double *)malloc((size_t)u->cap * sizeof(double));
    for (int g = 0; g < G; ++g) {
        const double *qg = q + (size_t)g * d;
        double mx = -INFINITY, den = 0.0;
        for (int s = 0; s < u->cap; ++s) {
            if (u->pos[s] < 0) continue;
            a[s] = dot(qg, u->K + (size_t)s * d, d) * scale;
            if (a[s] > mx) mx = a[s];
        }
        for (int s = 0; s < u->cap; ++s) if (u->pos[s] >= 0) { a[s] = exp(a[s] - mx); den += a[s]; }
        double *o = out + (size_t)g * d;
        for (int i = 0; i < d; ++i) o[i] = 0.0;
        double *row = u->A + ((size_t)nr * G + g) * u->cap;
        for (int s = 0; s < u->cap; ++s) {
            if (u->pos[s] < 0) { row[s] = 0.0; continue; }
            const double w = a[s] / den;
            row[s] = w;
            const double *vs = u->V + (size_t)s * d;
            for (int i = 0; i < d; ++i) o[i] += w * vs[i];
        }
        memcpy(u->Q + ((size_t)nr * G + g) * d, qg, (size_t)d * sizeof(double));
        u->wm[nr * G + g] = mx;
        u->wl[nr * G + g] = den;
    }
    free(a);

    /* 3. window slide (H1): keep the R most recent rows, discard the oldest profile */
    if (u->nw > R) {
        int oldest = -1;
        for (int r = 0; r <= R; ++r)
            if (u->wpos[r] >= 0 && (oldest < 0 || u->wpos[r] < u->wpos[oldest])) oldest = r;
        u->wpos[oldest] = -1;
        u->nw--;
        memset(u->A + (size_t)oldest * G * u->cap, 0, (size_t)G * u->cap * sizeof(double));
    }

    /* 4. score + select (Alg. 1, Eq. 7) on eviction steps when the distant side overflows */
    u->n_evicted = 0; u->n_cand = 0; u->kth = NAN; u->k1th = NAN;
    u->steps++;
    int rc = 0;
    if (u->steps % u->T == 0 && u->n - u->nw > u->C) rc = score_and_select(u, forced, n_forced);
    u->t = t + 1;
    return rc;
}

/* ---- read-back for the harness ---- */
int ora_count(const ora_unit *u) { return u->n; }
long ora_next_pos(const ora_unit *u) { return u->t; }

/* positions currently cached (unordered); returns the count */
int ora_cache_positions(const ora_unit *u, long *out)
{
    int n = 0;
    for (int s = 0; s < u->cap; ++s) if (u->pos[s] >= 0) out[n++] = u->pos[s];
    return n;
}

/* K/V row of a cached position; returns 0 if present */
int ora_cache_row(const ora_unit *u, long p, double *k_out, double *v_out)
{
    for (int s = 0; s < u->cap; ++s)
        if (u->pos[s] == p) {
            memcpy(k_out, u->K + (size_t)s * u->d, (size_t)u->d * sizeof(double));
            memcpy(v_out, u->V + (size_t)s * u->d, (size_t)u->d * sizeof(double));
            return 0;
        }
    return -1;
}

/* candidates of the last selection sorted by (F desc, pos asc); returns their count */
int ora_last_scores(const ora_unit *u, long *pos_out, double *F_out)
{
    for (int i = 0; i < u->n_cand; ++i) { pos_out[i] = u->cand_pos[i]; F_out[i] = u->cand_F[i]; }
    return u->n_cand;
}

int ora_last_evicted(const ora_unit *u, long *out)
{
    for (int i = 0; i < u->n_evicted; ++i) out[i] = u->evicted[i];
    return u->n_evicted;
}

/* C-th and (C+1)-th largest fused scores of the last selection (NaN if none) */
void ora_last_boundary(const ora_unit *u, double *kth, double *k1th) { *kth = u->kth; *k1th = u->k1th; }

/* frozen soft-max statistics of the window row holding position p (head g); returns 0 if present */
int ora_window_stats(const ora_unit *u, long p, int g, double *m, double *l)
{
    for (int r = 0; r <= u->R; ++r)
        if (u->wpos[r] == p) { *m = u->wm[r * u->G + g]; *l = u->wl[r * u->G + g]; return 0; }
    return -1;
}

/*
 * The fuse + select step alone on a caller-given table S[R][n] of group-summed
 * weights (Eq. 5 / Eq. 6 followed by Top_C with ties to the lower index):
 * writes F[n] and keep[n] (1 = retained).  Used to pin the paper's worked
 * example and the brute-force ranking tests.
 */
void ora_fuse_select(const double *S, int R, int n, int C, int fusion, double *F, int *keep)
{
    cand_t *c = (cand_t *)malloc((size_t)(n > 0 ? n : 1) * sizeof(cand_t));
    for (int k = 0; k < n; ++k) {
        double f = 0.0;
        for (int r = 0; r < R; ++r) {
            const double s = S[(size_t)r * n + k];
            if (fusion == ORA_SUM) f += s; else if (r == 0 || s > f) f = s;
        }
        F[k] = f; c[k].F = f; c[k].pos = k; c[k].slot = k;
    }
    qsort(c, (size_t)n, sizeof(cand_t), cand_cmp);
    for (int k = 0; k < n; ++k) keep[c[k].pos] = k < C;
    free(c);
}
