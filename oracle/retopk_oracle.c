/*
 * ReTopK decode step and Exact Top-K attention: plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, step-by-step restatement of the
 * method against which the CUDA library is checked.  It shares no code, header, table
 * or helper with the CUDA path, and only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may build or call it.
 *
 * ReTopK is a heuristic (it approximates the Exact Top-K support), so the oracle follows
 * the algorithm's steps in the paper's order and notation:
 *   Sec. 3.2 / Eq. 4, Eq. 1   full scores e_i = q.k_i / sqrt(d), exact support S_t
 *   Sec. 3.3 / Eq. 5          per-query-head FIFO cache of (normalised query, support)
 *   Eq. 6, Eq. 7              cosine similarities rho_c, Top-R recall, rho_max
 *   Eq. 8, Eq. 9              recent window, candidate set A_t = Unique(union)
 *   Eq. 10, Eq. 11            candidate scores and reranked support
 *   Eq. 12                    softmax . V over the selected support
 *   Sec. 3.4 / Eq. 13         path decision (refresh, similarity fallback, reuse)
 *   Sec. 3.4, last sentence   cache insert after either path
 *
 * Symbols: the paper's cache capacity C, recall count R and refresh period T_r are
 * called M, r and R here (the names of the library's C interface).
 *
 * Readings taken where the paper is silent (each is exercised by a test):
 *   - the cache is empty after create/reset; an empty cache gives rho_max = -inf and
 *     therefore the exact path;
 *   - with fewer than r cached entries, all of them are recalled;
 *   - t_dec is a 0-based offset: refresh iff R > 0, t_dec > 0 and t_dec % R == 0;
 *     refresh is tested before the similarity threshold; rho_max == tau reuses;
 *   - ties: larger value first, then lower index (keys) / lower slot (cache entries);
 *     -0.0 and +0.0 are equal;
 *   - the FIFO is a ring: entry number n is written to slot n % M, after recall;
 *   - supports are stored ascending; when fewer than K keys are selectable the support
 *     is padded with -1;
 *   - indices are 0-based; the window is [max(0, L - W), L - 1]; seq_len L includes the
 *     current token;
 *   - grouped-query attention: cache, decision and support per query head h, keys and
 *     values of KV head h / (H_q / H_kv);
 *   - a zero query normalises to zero;
 *   - "recent" recall (the component study's Recent-R row, Table 3): the min(r, fill) most
 *     recently inserted entries are recalled instead of the most similar ones, and rho_max is
 *     the largest similarity among THOSE entries (the paper gives no formula; the row's
 *     higher exact-path share fits a maximum taken over fewer entries);
 *   - prefill seeding (Sec. 3.3, cache paragraph: the cache starts from the last C prompt
 *     tokens): the paper does not say which support a prompt token gets; here each of the last
 *     n_tail <= M prompt positions p contributes its normalised query and its CAUSAL Exact
 *     Top-K support over keys 0..p, oldest first; the decode offset stays 0;
 *   - bf16 query cache (a storage variant; the paper runs everything in BF16 and does not say
 *     how the cached queries are kept): each element of the normalised query is rounded once,
 *     to nearest even, to bf16 when it is stored; the similarity of a later step is the dot
 *     product of that step's unrounded normalised query with the stored rounded one.
 *
 * Inputs are bf16 bit patterns, widened exactly to double; every sum is a plain
 * left-to-right fp64 loop; selection is a full sort.  OpenMP only spreads independent
 * (sequence, head) pairs over threads.
 *
 * Parity unpinned by the paper (fixed only by this file's readings, which the hand trace and
 * the integer-tie tests pin): the tie-breaks of Top-r and Top-K, whether the first decode
 * step has offset 0 or 1 for the refresh schedule, the recent-recall rule, the supports of
 * prompt tokens in prefill seeding, and the bf16 storage rule of cached queries.
 *
 * Pins (tests/test_oracle_pins.py): brute-force selection on small inputs, dense softmax
 * attention when K >= L, closed forms for K = 1 and K = 2, exact-path equality when
 * tau > 1 or W >= L, the hand-enumerated six-step trace in tests/golden, counter
 * identities, the candidate bound of Eq. 14, and tie cases with integer inputs; the fidelity
 * quantities (oracle_fidelity) by the hand trace, the W >= L case and a numpy restatement.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { PATH_REUSE = 0, PATH_FALLBACK = 1, PATH_REFRESH = 2 };

typedef struct {
    int B, Hq, Hkv, d, M, r, W, K, R;
    int recall_mode; /* 0: the r most similar cached queries (Eq. 7); 1: the r most recent ones */
    int qbar_bf16;   /* 1: cached normalised queries are rounded to bf16 when stored */
    double tau;
    int64_t max_seq_len;
    int64_t n_ins;   /* entries inserted so far (same for every head) */
    int64_t t_dec;   /* decode-step offset */
    double *qbar;    /* [B*Hq][M][d] */
    int32_t *sup;    /* [B*Hq][M][K], ascending, -1 padded */
    /* counters, summed over (sequence, head) */
    int64_t n_steps, n_reuse, n_fallback, n_refresh, cand_sum;
    /* record of the most recent step, per (sequence, head) */
    int32_t *last_sup;   /* [B*Hq][K] */
    uint8_t *last_path;  /* [B*Hq] */
    double *last_rho;    /* [B*Hq] rho_max (-inf when the cache was empty) */
    int32_t *last_ncand; /* [B*Hq] candidates scored (seq_len on exact steps) */
    double *last_kth;    /* [B*Hq] smallest selected score */
    int32_t *last_cand;  /* [B*Hq][r*K+W] candidate list of reuse steps */
    int32_t *last_sel;   /* [B*Hq][r] recalled slots, -1 padded */
    double *last_out;    /* [B*Hq][d] attention output of the step */
    int32_t *last_uni;   /* [B*Hq][r*K] union of the recalled supports U_t (Eq. 3), ascending */
    int32_t *last_nuni;  /* [B*Hq] its size (reuse steps only) */
} oracle_t;

static double bf16_to_double(uint16_t bits) {
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---- ordering used by every selection: larger value first, then lower index ---- */
typedef struct { double val; int32_t idx; } scored_t;

static int cmp_scored(const void *pa, const void *pb) {
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    if (a->val > b->val) return -1;
    if (a->val < b->val) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static int cmp_by_index(const void *pa, const void *pb) {
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static int cmp_int32(const void *pa, const void *pb) {
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

int oracle_create(oracle_t **out, int B, int Hq, int Hkv, int d, int M, int r, int W, int K,
                  double tau, int R, int64_t max_seq_len) {
    if (!out || B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || d < 1 || M < 1 || r < 1 || r > M ||
        W < 0 || K < 1 || R < 0 || max_seq_len < 1)
        return -1;
    oracle_t *o = (oracle_t *)calloc(1, sizeof *o);
    if (!o) return -2;
    o->B = B; o->Hq = Hq; o->Hkv = Hkv; o->d = d; o->M = M; o->r = r; o->W = W; o->K = K;
    o->tau = tau; o->R = R; o->max_seq_len = max_seq_len;
    size_t nh = (size_t)B * Hq;
    o->qbar = (double *)calloc(nh * M * d, sizeof(double));
    o->sup = (int32_t *)malloc(nh * M * K * sizeof(int32_t));
    o->last_sup = (int32_t *)malloc(nh * K * sizeof(int32_t));
    o->last_path = (uint8_t *)calloc(nh, 1);
    o->last_rho = (double *)calloc(nh, sizeof(double));
    o->last_ncand = (int32_t *)calloc(nh, sizeof(int32_t));
    o->last_kth = (double *)calloc(nh, sizeof(double));
    o->last_cand = (int32_t *)malloc(nh * ((size_t)r * K + W + 1) * sizeof(int32_t));
    o->last_sel = (int32_t *)malloc(nh * r * sizeof(int32_t));
    o->last_out = (double *)calloc(nh * d, sizeof(double));
    o->last_uni = (int32_t *)malloc(nh * ((size_t)r * K + 1) * sizeof(int32_t));
    o->last_nuni = (int32_t *)calloc(nh, sizeof(int32_t));
    if (!o->last_out || !o->last_uni || !o->last_nuni) return -2;
    if (!o->qbar || !o->sup || !o->last_sup || !o->last_path || !o->last_rho || !o->last_ncand ||
        !o->last_kth || !o->last_cand || !o->last_sel)
        return -2;
    memset(o->sup, 0xFF, nh * M * K * sizeof(int32_t));
    memset(o->last_sup, 0xFF, nh * K * sizeof(int32_t));
    memset(o->last_sel, 0xFF, nh * r * sizeof(int32_t));
    *out = o;
    return 0;
}

/* 0: similarity recall (the method); 1: recency recall (the Recent-R ablation row); r <= 64 then. */
int oracle_set_recall_mode(oracle_t *o, int mode) {
    if ((mode != 0 && mode != 1) || (mode == 1 && o->r > 64)) return -1;
    o->recall_mode = mode;
    return 0;
}

/* Nearest bf16 value (8 significand bits, ties to even) of a double, as a double. */
static double round_to_bf16(double x) {
    if (x == 0.0 || !isfinite(x)) return x;
    int e;
    frexp(x, &e);                 /* |x| = f * 2^e with f in [0.5, 1) */
    if (e < -125) e = -125;       /* below the normal range the spacing stays 2^-133 */
    return ldexp(nearbyint(ldexp(x, 8 - e)), e - 8);   /* nearbyint: round half to even */
}

/* 0: cached queries kept as computed (default); 1: rounded to bf16 when stored.  Only while
 * the cache is empty. */
int oracle_set_qbar_format(oracle_t *o, int fmt) {
    if ((fmt != 0 && fmt != 1) || o->n_ins != 0) return -1;
    o->qbar_bf16 = fmt;
    return 0;
}

void oracle_destroy(oracle_t *o) {
    if (!o) return;
    free(o->qbar); free(o->sup); free(o->last_sup); free(o->last_path); free(o->last_rho);
    free(o->last_ncand); free(o->last_kth); free(o->last_cand); free(o->last_sel);
    free(o->last_out); free(o->last_uni); free(o->last_nuni);
    free(o);
}

void oracle_reset(oracle_t *o) {
    size_t nh = (size_t)o->B * o->Hq;
    memset(o->qbar, 0, nh * o->M * o->d * sizeof(double));
    memset(o->sup, 0xFF, nh * o->M * o->K * sizeof(int32_t));
    o->n_ins = 0; o->t_dec = 0;
    o->n_steps = o->n_reuse = o->n_fallback = o->n_refresh = o->cand_sum = 0;
}

/* e_i = q.k_i / sqrt(d) (Eq. 4 and Eq. 10 are the same expression on different index sets). */
static double score_key(const double *q, const uint16_t *krow, int d) {
    double acc = 0.0;
    for (int j = 0; j < d; ++j) acc += q[j] * bf16_to_double(krow[j]);
    return acc / sqrt((double)d);
}

/*
 * Take the min(K, n) best of cand[0..n) under (score desc, index asc), return them
 * ascending by index in sup[0..K) (-1 padded) with their scores in sup_score, and
 * compute Eq. 12 over them.  Returns the number selected.
 */
static int select_and_attend(scored_t *cand, int n, int K, const uint16_t *vhead, int d,
                             int32_t *sup, double *out, double *kth) {
    qsort(cand, (size_t)n, sizeof *cand, cmp_scored);
    int ns = n < K ? n : K;
    *kth = ns > 0 ? cand[ns - 1].val : 0.0;
    /* Eq. 12 with the maximum subtracted (identical in exact arithmetic). */
    double m = ns > 0 ? cand[0].val : 0.0;
    double denom = 0.0;
    for (int j = 0; j < d; ++j) out[j] = 0.0;
    /* accumulate in ascending index order so the summation order is fixed */
    scored_t *chosen = (scored_t *)malloc((size_t)(ns > 0 ? ns : 1) * sizeof *chosen);
    for (int i = 0; i < ns; ++i) chosen[i] = cand[i];
    qsort(chosen, (size_t)ns, sizeof *chosen, cmp_by_index);
    for (int i = 0; i < ns; ++i) {
        double w = exp(chosen[i].val - m);
        denom += w;
        const uint16_t *vrow = vhead + (size_t)chosen[i].idx * d;
        for (int j = 0; j < d; ++j) out[j] += w * bf16_to_double(vrow[j]);
        sup[i] = chosen[i].idx;
    }
    for (int i = ns; i < K; ++i) sup[i] = -1;
    if (ns > 0)
        for (int j = 0; j < d; ++j) out[j] /= denom;
    free(chosen);
    return ns;
}

/* Exact Top-K attention for one head: Eq. 4, Eq. 1, Eq. 12. */
static void exact_head(const double *q, const uint16_t *khead, const uint16_t *vhead, int64_t L,
                       int d, int K, int32_t *sup, double *out, double *kth) {
    scored_t *all = (scored_t *)malloc((size_t)L * sizeof *all);
    for (int64_t i = 0; i < L; ++i) {
        all[i].val = score_key(q, khead + (size_t)i * d, d);
        all[i].idx = (int32_t)i;
    }
    select_and_attend(all, (int)L, K, vhead, d, sup, out, kth);
    free(all);
}

/*
 * Stateless Exact Top-K attention for every (sequence, head).
 * q [B,Hq,d], k/v [B,Hkv,max_seq_len,d] bf16 bits; out [B,Hq,d] double; idx [B,Hq,K] or NULL.
 */
int oracle_exact_topk(const oracle_t *o, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      int64_t L, double *out, int32_t *idx) {
    if (L < 1 || L > o->max_seq_len) return -1;
    const int d = o->d, G = o->Hq / o->Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < o->B; ++b)
        for (int h = 0; h < o->Hq; ++h) {
            size_t bh = (size_t)b * o->Hq + h;
            size_t kv = ((size_t)b * o->Hkv + h / G) * (size_t)o->max_seq_len * d;
            double *qd = (double *)malloc((size_t)d * sizeof(double));
            int32_t *sup = (int32_t *)malloc((size_t)o->K * sizeof(int32_t));
            double kth;
            for (int j = 0; j < d; ++j) qd[j] = bf16_to_double(q[bh * d + j]);
            exact_head(qd, k + kv, v + kv, L, d, o->K, sup, out + bh * d, &kth);
            if (idx) memcpy(idx + bh * o->K, sup, (size_t)o->K * sizeof(int32_t));
            free(qd); free(sup);
        }
    return 0;
}

/* One ReTopK decode step for one (sequence, head). */
static void retopk_head(oracle_t *o, size_t bh, const double *q, const uint16_t *khead,
                        const uint16_t *vhead, int64_t L, double *out) {
    const int d = o->d, M = o->M, K = o->K, r = o->r, W = o->W;
    double *cache_q = o->qbar + bh * M * d;
    int32_t *cache_s = o->sup + bh * (size_t)M * K;
    const int cap = r * K + W;

    /* normalised query (Eq. 5 / text above Eq. 6) */
    double *qbar = (double *)malloc((size_t)d * sizeof(double));
    double nrm2 = 0.0;
    for (int j = 0; j < d; ++j) nrm2 += q[j] * q[j];
    double nrm = sqrt(nrm2);
    for (int j = 0; j < d; ++j) qbar[j] = nrm > 0.0 ? q[j] / nrm : 0.0;

    /* Eq. 6: similarities to the cached queries; Eq. 7: rho_max and Top-R */
    int fill = (int)(o->n_ins < M ? o->n_ins : M);
    scored_t *rho = (scored_t *)malloc((size_t)(fill > 0 ? fill : 1) * sizeof *rho);
    double rho_max = -INFINITY;
    for (int c = 0; c < fill; ++c) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j) acc += qbar[j] * cache_q[(size_t)c * d + j];
        rho[c].val = acc;
        rho[c].idx = c;
        if (acc > rho_max) rho_max = acc;
    }

    /* recall set: all entries ranked by similarity, or just the newest min(r, fill) */
    const int n_recall = r < fill ? r : fill;
    int recent[64];
    if (o->recall_mode == 1) {
        rho_max = -INFINITY;
        for (int j = 0; j < n_recall; ++j) {
            recent[j] = (int)(((o->n_ins - 1 - j) % M + M) % M);      /* j = 0 is the newest */
            if (rho[recent[j]].val > rho_max) rho_max = rho[recent[j]].val;
        }
    }

    /* Eq. 13 */
    int path;
    if (o->R > 0 && o->t_dec > 0 && o->t_dec % o->R == 0) path = PATH_REFRESH;
    else if (rho_max < o->tau) path = PATH_FALLBACK;
    else path = PATH_REUSE;

    int32_t *sup = o->last_sup + bh * K;
    int32_t *sel = o->last_sel + bh * r;
    for (int i = 0; i < r; ++i) sel[i] = -1;
    double kth = 0.0;
    int n_scored;

    if (path == PATH_REUSE) {
        int n_sel = n_recall;
        if (o->recall_mode == 1) {
            scored_t tmp[64];
            for (int j = 0; j < n_sel; ++j) tmp[j] = rho[recent[j]];
            for (int j = 0; j < n_sel; ++j) rho[j] = tmp[j];          /* newest first */
        } else {
            qsort(rho, (size_t)fill, sizeof *rho, cmp_scored);
        }
        /* Eq. 8-9: union of recalled supports and the recent window, sorted, unique */
        int32_t *raw = (int32_t *)malloc((size_t)(cap + 1) * sizeof(int32_t));
        int n_raw = 0;
        for (int s = 0; s < n_sel; ++s) {
            sel[s] = rho[s].idx;
            const int32_t *stored = cache_s + (size_t)rho[s].idx * K;
            for (int i = 0; i < K; ++i)
                if (stored[i] >= 0) raw[n_raw++] = stored[i];
        }
        /* U_t of Eq. 3: the recalled supports alone, before the window joins them */
        {
            int32_t *uni = o->last_uni + bh * ((size_t)r * K + 1);
            int n_uni = 0;
            qsort(raw, (size_t)n_raw, sizeof(int32_t), cmp_int32);
            for (int i = 0; i < n_raw; ++i)
                if (i == 0 || raw[i] != raw[i - 1]) uni[n_uni++] = raw[i];
            o->last_nuni[bh] = n_uni;
        }
        int64_t w_lo = L - W > 0 ? L - W : 0;
        for (int64_t i = w_lo; i < L; ++i) raw[n_raw++] = (int32_t)i;
        qsort(raw, (size_t)n_raw, sizeof(int32_t), cmp_int32);
        int32_t *cand = o->last_cand + bh * (size_t)(cap + 1);
        int n_cand = 0;
        for (int i = 0; i < n_raw; ++i)
            if (i == 0 || raw[i] != raw[i - 1]) cand[n_cand++] = raw[i];
        /* Eq. 10: exact current-query scores on the candidates only */
        scored_t *sc = (scored_t *)malloc((size_t)(n_cand > 0 ? n_cand : 1) * sizeof *sc);
        for (int i = 0; i < n_cand; ++i) {
            sc[i].idx = cand[i];
            sc[i].val = score_key(q, khead + (size_t)cand[i] * d, d);
        }
        /* Eq. 11 and Eq. 12 */
        select_and_attend(sc, n_cand, K, vhead, d, sup, out, &kth);
        n_scored = n_cand;
        free(sc); free(raw);
    } else {
        exact_head(q, khead, vhead, L, d, K, sup, out, &kth);
        n_scored = (int)L;
    }

    /* insert (qbar_t, S_t) at the ring position; happens after recall on either path */
    int slot = (int)(o->n_ins % M);
    for (int j = 0; j < d; ++j)
        cache_q[(size_t)slot * d + j] = o->qbar_bf16 ? round_to_bf16(qbar[j]) : qbar[j];
    memcpy(cache_s + (size_t)slot * K, sup, (size_t)K * sizeof(int32_t));

    o->last_path[bh] = (uint8_t)path;
    o->last_rho[bh] = rho_max;
    o->last_ncand[bh] = n_scored;
    o->last_kth[bh] = kth;
    for (int j = 0; j < d; ++j) o->last_out[bh * d + j] = out[j];
    free(rho); free(qbar);
}

/*
 * One decode step for every (sequence, head).  L = seq_len includes the current token.
 * q [B,Hq,d], k/v [B,Hkv,max_seq_len,d] bf16 bits; out [B,Hq,d] double.
 */
int oracle_decode_step(oracle_t *o, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       int64_t L, double *out) {
    if (L < 1 || L > o->max_seq_len) return -1;
    const int d = o->d, G = o->Hq / o->Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < o->B; ++b)
        for (int h = 0; h < o->Hq; ++h) {
            size_t bh = (size_t)b * o->Hq + h;
            size_t kv = ((size_t)b * o->Hkv + h / G) * (size_t)o->max_seq_len * d;
            double *qd = (double *)malloc((size_t)d * sizeof(double));
            for (int j = 0; j < d; ++j) qd[j] = bf16_to_double(q[bh * d + j]);
            retopk_head(o, bh, qd, k + kv, v + kv, L, out + bh * d);
            free(qd);
        }
    size_t nh = (size_t)o->B * o->Hq;
    for (size_t bh = 0; bh < nh; ++bh) {
        o->n_steps += 1;
        if (o->last_path[bh] == PATH_REUSE) { o->n_reuse += 1; o->cand_sum += o->last_ncand[bh]; }
        else if (o->last_path[bh] == PATH_FALLBACK) o->n_fallback += 1;
        else o->n_refresh += 1;
    }
    o->n_ins += 1;
    o->t_dec += 1;
    return 0;
}

/*
 * Seed the caches from the last n_tail prompt positions (Sec. 3.3, first paragraph).
 * q_tail [n_tail,B,Hq,d]: query of prompt position prompt_len - n_tail + j in slab j.
 * Entry j gets the causal Exact Top-K support over keys 0 .. prompt_len - n_tail + j (Eq. 1).
 */
int oracle_prefill(oracle_t *o, const uint16_t *q_tail, const uint16_t *k, const uint16_t *v,
                   int64_t prompt_len, int n_tail) {
    if (n_tail < 1 || n_tail > o->M || n_tail > prompt_len || prompt_len > o->max_seq_len) return -1;
    const int d = o->d, G = o->Hq / o->Hkv, K = o->K, M = o->M;
    const size_t nh = (size_t)o->B * o->Hq;
    for (int j = 0; j < n_tail; ++j) {
        const int64_t L = prompt_len - n_tail + j + 1;
        const int slot = (int)(o->n_ins % M);
#pragma omp parallel for schedule(dynamic, 1)
        for (long bh = 0; bh < (long)nh; ++bh) {
            const int b = (int)(bh / o->Hq), h = (int)(bh % o->Hq);
            const size_t kv = ((size_t)b * o->Hkv + h / G) * (size_t)o->max_seq_len * d;
            double *qd = (double *)malloc((size_t)d * sizeof(double));
            double *out = (double *)malloc((size_t)d * sizeof(double));
            int32_t *sup = (int32_t *)malloc((size_t)K * sizeof(int32_t));
            double kth, nrm2 = 0.0;
            for (int t = 0; t < d; ++t) {
                qd[t] = bf16_to_double(q_tail[((size_t)j * nh + bh) * d + t]);
                nrm2 += qd[t] * qd[t];
            }
            exact_head(qd, k + kv, v + kv, L, d, K, sup, out, &kth);
            const double nrm = sqrt(nrm2);
            double *cq = o->qbar + ((size_t)bh * M + slot) * d;
            for (int t = 0; t < d; ++t) {
                cq[t] = nrm > 0.0 ? qd[t] / nrm : 0.0;
                if (o->qbar_bf16) cq[t] = round_to_bf16(cq[t]);
            }
            memcpy(o->sup + ((size_t)bh * M + slot) * K, sup, (size_t)K * sizeof(int32_t));
            free(qd); free(out); free(sup);
        }
        o->n_ins += 1;
    }
    return 0;
}

/*
 * Fidelity of the most recent decode step against Exact Top-K attention on the same inputs
 * (the quantities of Eq. 2-3 and of the fidelity paragraph of Sec. 4).  Call right after
 * oracle_decode_step with that step's q, k, v and L.  Per (sequence, head), four doubles:
 *   [0] support recall   |S^_t & S_t| / |S_t|   (S_t exact support of Eq. 1, S^_t the step's support)
 *   [1] retained mass    sum over i in S_t & S^_t of softmax(e restricted to S_t)_i
 *   [2] output cosine    <o^_t, o_t> / (|o^_t| |o_t|), o_t the Exact Top-K output (Eq. 12 over S_t)
 *   [3] coverage         |S_t & U_t| / |S_t| with U_t the union of the recalled supports (Eq. 3);
 *                        -1 on steps that did not take the reuse path
 * Plain definitions: one membership scan per index, left-to-right sums.
 */
int oracle_fidelity(const oracle_t *o, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                    int64_t L, double *four) {
    if (L < 1 || L > o->max_seq_len) return -1;
    const int d = o->d, G = o->Hq / o->Hkv, K = o->K;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < o->B; ++b)
        for (int h = 0; h < o->Hq; ++h) {
            size_t bh = (size_t)b * o->Hq + h;
            size_t kv = ((size_t)b * o->Hkv + h / G) * (size_t)o->max_seq_len * d;
            double *qd = (double *)malloc((size_t)d * sizeof(double));
            double *oe = (double *)malloc((size_t)d * sizeof(double));
            int32_t *se = (int32_t *)malloc((size_t)K * sizeof(int32_t));
            double kth;
            for (int j = 0; j < d; ++j) qd[j] = bf16_to_double(q[bh * d + j]);
            exact_head(qd, k + kv, v + kv, L, d, K, se, oe, &kth);
            const int32_t *sr = o->last_sup + bh * K;
            const int32_t *uni = o->last_uni + bh * ((size_t)o->r * K + 1);
            const int n_uni = o->last_nuni[bh];
            int ne = 0, both = 0, covered = 0;
            double m = -INFINITY;
            for (int i = 0; i < K && se[i] >= 0; ++i) {
                double e = score_key(qd, k + kv + (size_t)se[i] * d, d);
                if (e > m) m = e;
                ++ne;
            }
            double denom = 0.0, kept = 0.0;
            for (int i = 0; i < ne; ++i) {
                double w = exp(score_key(qd, k + kv + (size_t)se[i] * d, d) - m);
                int in_r = 0, in_u = 0;
                for (int j = 0; j < K; ++j) if (sr[j] == se[i]) in_r = 1;
                for (int j = 0; j < n_uni; ++j) if (uni[j] == se[i]) in_u = 1;
                denom += w;
                if (in_r) { kept += w; ++both; }
                covered += in_u;
            }
            double dot = 0.0, na = 0.0, nb = 0.0;
            for (int j = 0; j < d; ++j) {
                double a = o->last_out[bh * d + j];
                dot += a * oe[j]; na += a * a; nb += oe[j] * oe[j];
            }
            double *f = four + bh * 4;
            f[0] = ne > 0 ? (double)both / ne : 0.0;
            f[1] = denom > 0.0 ? kept / denom : 0.0;
            f[2] = (na > 0.0 && nb > 0.0) ? dot / (sqrt(na) * sqrt(nb)) : 0.0;
            f[3] = o->last_path[bh] == PATH_REUSE && ne > 0 ? (double)covered / ne : -1.0;
            free(qd); free(oe); free(se);
        }
    return 0;
}

/* counters: steps, reuse, fallback, refresh, cand_sum */
void oracle_stats(const oracle_t *o, int64_t *five) {
    five[0] = o->n_steps; five[1] = o->n_reuse; five[2] = o->n_fallback;
    five[3] = o->n_refresh; five[4] = o->cand_sum;
}

/* Record of the most recent step; any pointer may be NULL. */
void oracle_last_step(const oracle_t *o, int32_t *support, uint8_t *path, double *rho_max,
                      int32_t *n_cand, double *kth_score, int32_t *sel) {
    size_t nh = (size_t)o->B * o->Hq;
    if (support) memcpy(support, o->last_sup, nh * o->K * sizeof(int32_t));
    if (path) memcpy(path, o->last_path, nh);
    if (rho_max) memcpy(rho_max, o->last_rho, nh * sizeof(double));
    if (n_cand) memcpy(n_cand, o->last_ncand, nh * sizeof(int32_t));
    if (kth_score) memcpy(kth_score, o->last_kth, nh * sizeof(double));
    if (sel) memcpy(sel, o->last_sel, nh * o->r * sizeof(int32_t));
}

/* Candidate list of head bh at the most recent step (valid only if that step reused). */
int oracle_last_candidates(const oracle_t *o, int bh, int32_t *cand) {
    if (o->last_path[bh] != PATH_REUSE) return -1;
    size_t cap1 = (size_t)o->r * o->K + o->W + 1;
    memcpy(cand, o->last_cand + (size_t)bh * cap1, (size_t)o->last_ncand[bh] * sizeof(int32_t));
    return o->last_ncand[bh];
}

void oracle_export_state(const oracle_t *o, double *qbar, int32_t *sup, int64_t *n_ins,
                         int64_t *t_dec) {
    size_t nh = (size_t)o->B * o->Hq;
    if (qbar) memcpy(qbar, o->qbar, nh * o->M * o->d * sizeof(double));
    if (sup) memcpy(sup, o->sup, nh * o->M * o->K * sizeof(int32_t));
    if (n_ins) *n_ins = o->n_ins;
    if (t_dec) *t_dec = o->t_dec;
}

void oracle_import_state(oracle_t *o, const double *qbar, const int32_t *sup, int64_t n_ins,
                         int64_t t_dec) {
    size_t nh = (size_t)o->B * o->Hq;
    memcpy(o->qbar, qbar, nh * o->M * o->d * sizeof(double));
    memcpy(o->sup, sup, nh * o->M * o->K * sizeof(int32_t));
    o->n_ins = n_ins;
    o->t_dec = t_dec;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
