/*
 * DynaKV oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, double-precision CPU restatement of cluster-based KV-cache retrieval
 * with migration-free adaptation (arXiv 2511.07427, Section 4 and Algorithm 1), one
 * unit (= one KV head of one layer of one sequence) at a time.  Only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no code
 * with the CUDA library.
 *
 * Conventions (where the paper is silent the reading is stated at the function):
 *   - all distances are the direct sum of squared differences, all sums run in index
 *     order, all ties go to the lowest index;
 *   - a "hint" is another implementation's answer to a discrete decision.  The oracle
 *     always computes its own answer first; it adopts the hint only if, measured with
 *     the oracle's own numbers, the two candidates differ by less than `tol` relative
 *     (|a-b| / max(|a|,|b|)), counting a tie; otherwise it keeps its own answer and
 *     counts a violation.  With no hint the oracle is self-contained.
 *
 * Pins (tests, CPU only): brute-force argmin, inertia monotonicity, blob recovery,
 * scikit-learn Lloyd cross-check, D^2-sampling frequencies, Welford vs two-pass,
 * full-budget retrieval == dense softmax attention, split invariants, the round cap of
 * the split's 2-means (hand-worked fixture), validity of a selection hint (including the
 * over-budget single-cluster case), the static and local update modes (frozen build, brute-force
 * append targets, separation of two new blobs).
 * Conventions the paper leaves open (score metric, GQA reduction, threshold
 * calibration, split seeding, id rule, budget boundary) are "parity unpinned" by the
 * paper: they are pinned only to their stated definitions.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORK_INIT_KMEANSPP 0
#define ORK_INIT_RANDOM 1

/* How the partition follows the decode stream (Section 3.1 and the baselines of Section 8.1):
 *   ADAPTIVE  append to the nearest cluster, split clusters that grow too large or too spread out (the paper's method);
 *   STATIC    append to the nearest cluster, never split ("static update");
 *   LOCAL     new entries are clustered among themselves only ("local update"): clusters of the prefill build never
 *             change; a new entry joins the nearest cluster born during decoding (the first one founds it), and such a
 *             cluster is split by the same 2-means once it holds more than local_max entries;
 *   DELAYED   the adaptive rule with Algorithm 1's delayed split (Section 4.2): a cluster whose trigger fires is split
 *             at once only if it is among the clusters the step's query retrieved; otherwise it is flagged, entries
 *             it takes from then on count as buffered, and it is split at the first later check at which it is among
 *             the retrieved clusters.  When the buffered entries of all flagged clusters reach buf_max, the flagged
 *             cluster with the most buffered entries (lowest id among equals) is split as well, after the others. */
#define ORK_MODE_ADAPTIVE 0
#define ORK_MODE_STATIC 1
#define ORK_MODE_LOCAL 2
#define ORK_MODE_DELAYED 3

#define ORK_ST_BUDGET_EXCEEDED 1u
#define ORK_ST_MAX_CLUSTERS 2u
#define ORK_ST_MAX_TOKENS 4u

typedef struct {
    int d, G, max_tokens, max_clusters;
    int n;              /* tokens stored; token id = arrival position */
    int M;              /* cluster ids handed out so far (live or dead) */
    double *K, *V;      /* [max_tokens][d] in token-id order */
    int *assign;        /* [max_tokens] cluster id of each token */
    double *r;          /* [max_clusters][d] representatives (Eq. 4) */
    double *M2;         /* [max_clusters] sum of squared distances of members to r */
    int *cnt;           /* [max_clusters] n_j */
    unsigned char *live, *hold;
    double tau;         /* variance threshold of this unit */
    double gamma, alpha;
    int split_min_size, split_iters;
    double tol;
    long ties, violations;
    unsigned status;
    long n_splits;
    int mode, local_max;  /* update mode; LOCAL: size above which a decode-born cluster splits */
    int M_build;          /* ids handed out by the build (or installed): the "old" clusters of LOCAL mode */
    /* DELAYED mode */
    int buf_max;          /* B_max: buffered entries over all flagged clusters that force a split */
    unsigned char *flag;  /* [max_clusters] f_j: a split of cluster j is owed */
    int *buf;             /* [max_clusters] |Buf_j|: the entry that raised the flag and every entry taken since */
    int *req;             /* the clusters the last decode step retrieved, n_req of them */
    int n_req;
} ork_unit;

/* ---------------------------------------------------------------- helpers */

static double sqdist(const double *a, const double *b, int d) {
    double s = 0.0;
    for (int t = 0; t < d; t++) { double e = a[t] - b[t]; s += e * e; }
    return s;
}

static double dot(const double *a, const double *b, int d) {
    double s = 0.0;
    for (int t = 0; t < d; t++) s += a[t] * b[t];
    return s;
}

static int near_tie(double a, double b, double tol) {
    double m = fmax(fabs(a), fabs(b));
    if (m == 0.0) return 1;
    return fabs(a - b) / m < tol;
}

/* Counter-based uniform in (0,1) with 23 random bits: u = (bits + 1/2) / 2^23.
 * The 64-bit counter built from (seed, unit, round, i) goes through the splitmix64
 * finaliser; the CUDA side implements the same published mixer on its own. */
double ork_uniform(uint64_t seed, int unit, int round, int64_t i) {
    uint64_t x = seed ^ ((uint64_t)(unit + 1) * 0x9E3779B97F4A7C15ULL);
    x += (uint64_t)round * 0xBF58476D1CE4E5B9ULL + (uint64_t)i * 0x94D049BB133111EBULL;
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27; x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    uint64_t bits = x >> 41;
    return ((double)bits + 0.5) / 8388608.0;
}

/* ------------------------------------------------- prefill: init (NewCluster) */

/* Seeded k-means++ written as an exponential race: with E_i = -ln u_i i.i.d. Exp(1),
 * argmax_i D2_i / E_i picks index i with probability D2_i / sum D2 (D^2 sampling),
 * and round 0 (argmin E_i) is a uniform pick.  The paper says only "K-Means"
 * (Section 4.1); the seeded k-means++ start is the benchmark configuration's. */
void ork_init_kmeanspp(const double *K, int n, int d, int M, uint64_t seed, int unit,
                       const int *hint, double tol, int *picks, long *ties, long *viol) {
    double *D2 = (double *)malloc(sizeof(double) * (size_t)n);
    for (int r = 0; r < M; r++) {
        int best = 0; double bestv = 0.0;
        for (int i = 0; i < n; i++) {
            double E = -log(ork_uniform(seed, unit, r, i));
            double v = (r == 0) ? -E : D2[i] / E;
            if (i == 0 || v > bestv) { bestv = v; best = i; }
        }
        if (hint && hint[r] != best && hint[r] >= 0 && hint[r] < n) {
            double E = -log(ork_uniform(seed, unit, r, hint[r]));
            double v = (r == 0) ? -E : D2[hint[r]] / E;
            if (near_tie(v, bestv, tol)) { best = hint[r]; if (ties) (*ties)++; }
            else if (viol) (*viol)++;
        }
        picks[r] = best;
        for (int i = 0; i < n; i++) {
            double dd = sqdist(K + (size_t)i * d, K + (size_t)best * d, d);
            if (r == 0 || dd < D2[i]) D2[i] = dd;
        }
    }
    free(D2);
}

/* Random distinct start: the M keys with the smallest (u(seed,unit,0,i), i), listed in
 * index order.  The uniforms are 23-bit integers in disguise, so this is exact. */
void ork_init_random(int n, int M, uint64_t seed, int unit, int *picks) {
    double *u = (double *)malloc(sizeof(double) * (size_t)n);
    unsigned char *taken = (unsigned char *)calloc((size_t)n, 1);
    for (int i = 0; i < n; i++) u[i] = ork_uniform(seed, unit, 0, i);
    for (int r = 0; r < M && r < n; r++) {
        int best = -1;
        for (int i = 0; i < n; i++)
            if (!taken[i] && (best < 0 || u[i] < u[best])) best = i;
        taken[best] = 1;
    }
    int c = 0;
    for (int i = 0; i < n && c < M; i++) if (taken[i]) picks[c++] = i;
    free(u); free(taken);
}

/* ------------------------------------------------- prefill: Lloyd iterations */

/* a_i = argmin_j ||k_i - c_j||^2 over the candidate clusters (Section 4.1, Eq. 3:
 * every entry belongs to exactly one cluster).  `live` NULL = all M are candidates. */
void ork_assign(const double *K, int n, int d, const double *C, int M, const unsigned char *live,
                const int *hint, double tol, int *assign, long *ties, long *viol) {
    for (int i = 0; i < n; i++) {
        const double *k = K + (size_t)i * d;
        int best = -1; double bd = 0.0;
        for (int j = 0; j < M; j++) {
            if (live && !live[j]) continue;
            double dd = sqdist(k, C + (size_t)j * d, d);
            if (best < 0 || dd < bd) { bd = dd; best = j; }
        }
        if (hint && hint[i] != best) {
            int h = hint[i];
            if (h >= 0 && h < M && (!live || live[h]) && near_tie(sqdist(k, C + (size_t)h * d, d), bd, tol)) {
                best = h; if (ties) (*ties)++;
            } else if (viol) (*viol)++;
        }
        assign[i] = best;
    }
}

/* c_j = mean of the keys assigned to j (Eq. 4).  A cluster with no member keeps its
 * previous centre (the reading taken for Section 7's remark that the k-means copes with empty clusters). */
void ork_update(const double *K, int n, int d, const int *assign, int M, double *C, int *cnt) {
    double *sum = (double *)calloc((size_t)M * d, sizeof(double));
    for (int j = 0; j < M; j++) cnt[j] = 0;
    for (int i = 0; i < n; i++) {
        int j = assign[i];
        cnt[j]++;
        for (int t = 0; t < d; t++) sum[(size_t)j * d + t] += K[(size_t)i * d + t];
    }
    for (int j = 0; j < M; j++)
        if (cnt[j] > 0)
            for (int t = 0; t < d; t++) C[(size_t)j * d + t] = sum[(size_t)j * d + t] / cnt[j];
    free(sum);
}

/* Sum over keys of the squared distance to the assigned centre (k-means inertia). */
double ork_inertia(const double *K, int n, int d, const double *C, const int *assign) {
    double s = 0.0;
    for (int i = 0; i < n; i++) s += sqdist(K + (size_t)i * d, C + (size_t)assign[i] * d, d);
    return s;
}

/* ---------------------------------------------------------------- unit state */

ork_unit *ork_create(int d, int G, int max_tokens, int max_clusters, double gamma, double alpha,
                     int split_min_size, int split_iters, double tol) {
    ork_unit *u = (ork_unit *)calloc(1, sizeof(ork_unit));
    u->d = d; u->G = G; u->max_tokens = max_tokens; u->max_clusters = max_clusters;
    u->K = (double *)calloc((size_t)max_tokens * d, sizeof(double));
    u->V = (double *)calloc((size_t)max_tokens * d, sizeof(double));
    u->assign = (int *)calloc((size_t)max_tokens, sizeof(int));
    u->r = (double *)calloc((size_t)max_clusters * d, sizeof(double));
    u->M2 = (double *)calloc((size_t)max_clusters, sizeof(double));
    u->cnt = (int *)calloc((size_t)max_clusters, sizeof(int));
    u->live = (unsigned char *)calloc((size_t)max_clusters, 1);
    u->hold = (unsigned char *)calloc((size_t)max_clusters, 1);
    u->flag = (unsigned char *)calloc((size_t)max_clusters, 1);
    u->buf = (int *)calloc((size_t)max_clusters, sizeof(int));
    u->req = (int *)calloc((size_t)max_clusters, sizeof(int));
    u->buf_max = 1 << 30;
    u->gamma = gamma; u->alpha = alpha;
    u->split_min_size = split_min_size; u->split_iters = split_iters;
    u->tol = tol;
    return u;
}

void ork_destroy(ork_unit *u) {
    if (!u) return;
    free(u->K); free(u->V); free(u->assign); free(u->r); free(u->M2); free(u->cnt);
    free(u->live); free(u->hold); free(u->flag); free(u->buf); free(u->req); free(u);
}

/* UpdateStats (Algorithm 1): n_j, r_j = member mean, M2_j = sum ||k - r_j||^2 recomputed
 * from the members of cluster j, members visited in token-id order. */
static void recompute_stats(ork_unit *u, int j) {
    int d = u->d, c = 0;
    double *r = u->r + (size_t)j * d;
    double *sum = (double *)calloc((size_t)d, sizeof(double));
    for (int i = 0; i < u->n; i++)
        if (u->assign[i] == j) { c++; for (int t = 0; t < d; t++) sum[t] += u->K[(size_t)i * d + t]; }
    u->cnt[j] = c;
    if (c > 0) for (int t = 0; t < d; t++) r[t] = sum[t] / c;
    double m2 = 0.0;
    for (int i = 0; i < u->n; i++)
        if (u->assign[i] == j) m2 += sqdist(u->K + (size_t)i * d, r, d);
    u->M2[j] = m2;
    free(sum);
}

/* Prefill (Algorithm 1, NewCluster on the prefill cache): init, then exactly T rounds of
 * assign + update; membership is the T-th assignment and the representatives are its
 * means, so Eq. 4 holds exactly.  Clusters empty at the end are dead: never scored,
 * never appended to; their ids stay reserved.  The unit's variance threshold is
 * tau = alpha * mean over live clusters of sigma_j^2, sigma_j^2 = M2_j / n_j (the paper
 * calls the thresholds head-specific but does not say how they are set).
 * hint_picks [M] and hint_assign [T][n] are optional. */
int ork_build(ork_unit *u, const double *K, const double *V, int n, int n_clusters, int T,
              uint64_t seed, int unit_index, int init_mode, const int *hint_picks,
              const int *hint_assign) {
    int d = u->d, M = n_clusters;
    if (n > u->max_tokens || M > u->max_clusters || n < M || M < 1) return -1;
    memcpy(u->K, K, sizeof(double) * (size_t)n * d);
    memcpy(u->V, V, sizeof(double) * (size_t)n * d);
    u->n = n; u->M = M; u->M_build = M;
    int *picks = (int *)malloc(sizeof(int) * (size_t)M);
    if (init_mode == ORK_INIT_KMEANSPP)
        ork_init_kmeanspp(u->K, n, d, M, seed, unit_index, hint_picks, u->tol, picks, &u->ties, &u->violations);
    else
        ork_init_random(n, M, seed, unit_index, picks);
    for (int j = 0; j < M; j++) memcpy(u->r + (size_t)j * d, u->K + (size_t)picks[j] * d, sizeof(double) * d);
    free(picks);
    for (int it = 0; it < T; it++) {
        ork_assign(u->K, n, d, u->r, M, NULL, hint_assign ? hint_assign + (size_t)it * n : NULL,
                   u->tol, u->assign, &u->ties, &u->violations);
        ork_update(u->K, n, d, u->assign, M, u->r, u->cnt);
    }
    double vs = 0.0; int nl = 0;
    for (int j = 0; j < M; j++) {
        u->live[j] = u->cnt[j] > 0; u->hold[j] = 0; u->M2[j] = 0.0;
        if (!u->live[j]) continue;
        for (int i = 0; i < n; i++)
            if (u->assign[i] == j) u->M2[j] += sqdist(u->K + (size_t)i * d, u->r + (size_t)j * d, d);
        vs += u->M2[j] / u->cnt[j]; nl++;
    }
    u->tau = u->alpha * (vs / nl);
    return 0;
}

/* ------------------------------------------------------ decode: score, select */

/* s_j = (1/G) sum_g q_g . r_j for live clusters (Section 4.1: the query is scored against
 * every representative).  Inner product, averaged over the G query heads that
 * share this KV head so the group retrieves one set.  Dead clusters get -infinity. */
void ork_score(const ork_unit *u, const double *q, double *scores) {
    int d = u->d;
    for (int j = 0; j < u->M; j++) {
        if (!u->live[j]) { scores[j] = -INFINITY; continue; }
        double s = 0.0;
        for (int g = 0; g < u->G; g++) s += dot(q + (size_t)g * d, u->r + (size_t)j * d, d);
        scores[j] = s / u->G;
    }
}

/* Top clusters under a token budget: order live clusters by (score descending, id
 * ascending) and take the longest prefix whose sizes sum to <= budget; if the first
 * cluster alone is larger it is taken whole and BUDGET_EXCEEDED is raised (the budget
 * form of the paper's top-k active set, Section 4.1 / Algorithm 1, the step that loads the top clusters).
 * Returns the selection in that order.
 * With a hint (another implementation's ordered selection) the hint is accepted, and a
 * tie counted, if it is a valid answer up to `tol` on the scores: non-increasing up to
 * tol, within budget, no unselected cluster scoring above the last selected one by more
 * than tol, and some unselected cluster tied for next place does not fit.  A hint that
 * exceeds the budget is valid only as one cluster that ties the best live score, when the
 * oracle's own answer is the over-budget case as well. */
int ork_select(ork_unit *u, const double *scores, int budget, const int *hint_ids, int hint_n,
               int *out_ids, int *out_tokens) {
    int M = u->M, nsel = 0, tokens = 0;
    unsigned char *used = (unsigned char *)calloc((size_t)M, 1);
    for (;;) {
        int best = -1;
        for (int j = 0; j < M; j++)
            if (u->live[j] && !used[j] && (best < 0 || scores[j] > scores[best])) best = j;
        if (best < 0) break;
        if (tokens + u->cnt[best] > budget) {
            if (nsel == 0 && budget > 0) { out_ids[nsel++] = best; tokens += u->cnt[best]; u->status |= ORK_ST_BUDGET_EXCEEDED; }
            break;
        }
        used[best] = 1; out_ids[nsel++] = best; tokens += u->cnt[best];
    }
    free(used);
    if (hint_ids && hint_n >= 0) {
        int same = (hint_n == nsel);
        for (int a = 0; same && a < nsel; a++) same = (hint_ids[a] == out_ids[a]);
        if (!same) {
            /* is the hint a valid selection up to tol? */
            int ok = 1, htok = 0;
            unsigned char *in = (unsigned char *)calloc((size_t)M, 1);
            for (int a = 0; a < hint_n && ok; a++) {
                int j = hint_ids[a];
                if (j < 0 || j >= M || !u->live[j] || in[j]) { ok = 0; break; }
                in[j] = 1; htok += u->cnt[j];
                if (a > 0) {
                    double sp = scores[hint_ids[a - 1]], sc = scores[j];
                    if (sc > sp && !near_tie(sc, sp, u->tol)) ok = 0;
                }
            }
            int over = ok && htok > budget;
            if (over) {
                /* Over budget: valid only as the "best cluster taken alone" case.  The hint must be a single
                 * cluster, the oracle's own answer must be that case too, and the hinted cluster must tie the
                 * best live score. */
                int own_over = (nsel == 1 && tokens > budget);
                if (hint_n != 1 || !own_over) ok = 0;
                else {
                    double sh = scores[hint_ids[0]], sb = scores[out_ids[0]];
                    if (!(sh == sb || near_tie(sh, sb, u->tol))) ok = 0;
                }
            }
            if (ok && hint_n == 0) {
                /* nothing selected: valid only if nothing fits at the top */
                int any = 0; for (int j = 0; j < M; j++) any |= u->live[j];
                if (any && budget > 0) ok = 0;
            }
            if (ok && hint_n > 0 && !over) {
                double slast = scores[hint_ids[hint_n - 1]];
                double snext = -INFINITY; int have = 0;
                for (int j = 0; j < M; j++)
                    if (u->live[j] && !in[j]) { if (!have || scores[j] > snext) snext = scores[j]; have = 1; }
                if (have) {
                    if (snext > slast && !near_tie(snext, slast, u->tol)) ok = 0;
                    int blocked = 0;
                    for (int j = 0; j < M; j++)
                        if (u->live[j] && !in[j] && (scores[j] == snext || near_tie(scores[j], snext, u->tol)) &&
                            htok + u->cnt[j] > budget) blocked = 1;
                    if (!blocked) ok = 0;
                }
            }
            free(in);
            if (ok) {
                u->ties++;
                nsel = hint_n; tokens = htok;
                for (int a = 0; a < nsel; a++) out_ids[a] = hint_ids[a];
            } else u->violations++;
        }
    }
    if (out_tokens) *out_tokens = tokens;
    return nsel;
}

/* ------------------------------------------------------ decode: attention */

/* Attention restricted to the retrieved entries (Section 2.1: attention reads
 * only the retrieved part of the cache): for each of the G heads, logits q_g.k_i / sqrt(d) over the
 * members of the selected clusters (token-id order), softmax, weighted sum of values.
 * Written as the definition: max, exponentials, normalise.  Empty selection -> zeros. */
void ork_attend(const ork_unit *u, const double *q, const int *ids, int n_ids, double *out) {
    int d = u->d;
    unsigned char *sel = (unsigned char *)calloc((size_t)u->max_clusters, 1);
    for (int a = 0; a < n_ids; a++) sel[ids[a]] = 1;
    double *logit = (double *)malloc(sizeof(double) * (size_t)(u->n > 0 ? u->n : 1));
    double scale = 1.0 / sqrt((double)d);
    for (int g = 0; g < u->G; g++) {
        double *o = out + (size_t)g * d;
        for (int t = 0; t < d; t++) o[t] = 0.0;
        double mx = -INFINITY; int any = 0;
        for (int i = 0; i < u->n; i++) {
            if (!sel[u->assign[i]]) continue;
            logit[i] = dot(q + (size_t)g * d, u->K + (size_t)i * d, d) * scale;
            if (!any || logit[i] > mx) mx = logit[i];
            any = 1;
        }
        if (!any) continue;
        double den = 0.0;
        for (int i = 0; i < u->n; i++) if (sel[u->assign[i]]) den += exp(logit[i] - mx);
        for (int i = 0; i < u->n; i++) {
            if (!sel[u->assign[i]]) continue;
            double p = exp(logit[i] - mx) / den;
            for (int t = 0; t < d; t++) o[t] += p * u->V[(size_t)i * d + t];
        }
    }
    free(logit); free(sel);
}

/* One retrieval step: score, select, attend.  Returns the number of selected clusters;
 * ids (score order) go to out_ids, the attention output [G][d] to out. */
int ork_decode_step(ork_unit *u, const double *q, int budget, const int *hint_ids, int hint_n,
                    double *out, int *out_ids, int *out_tokens) {
    double *scores = (double *)malloc(sizeof(double) * (size_t)(u->M > 0 ? u->M : 1));
    ork_score(u, q, scores);
    int nsel = ork_select(u, scores, budget, hint_ids, hint_n, out_ids, out_tokens);
    ork_attend(u, q, out_ids, nsel, out);
    /* the retrieved set of this step, for the delayed split */
    u->n_req = nsel;
    for (int i = 0; i < nsel; i++) u->req[i] = out_ids[i];
    free(scores);
    return nsel;
}

/* ------------------------------------------------------ decode: append */

/* Algorithm 1, the nearest-cluster assignment of the new entry, UpdateVar, AddEntry,
 * UpdateStats: nearest live representative in squared Euclidean distance, then the
 * incremental mean / sum-of-squares update
 *     n <- n+1;  delta = k - r;  r <- r + delta/n;  M2 <- M2 + delta.(k - r_new),
 * which needs only the centroid, the running sum of squares and the new entry, as Section 4.2 says the update should.
 * Returns the cluster id, or -1 if the unit is full. */
int ork_append(ork_unit *u, const double *k, const double *v, int hint_cluster) {
    int d = u->d;
    if (u->n >= u->max_tokens) { u->status |= ORK_ST_MAX_TOKENS; return -1; }
    int best = -1; double bd = 0.0;
    /* LOCAL mode: only clusters born during decoding are candidates */
    int j0 = (u->mode == ORK_MODE_LOCAL) ? u->M_build : 0;
    for (int j = j0; j < u->M; j++) {
        if (!u->live[j]) continue;
        double dd = sqdist(k, u->r + (size_t)j * d, d);
        if (best < 0 || dd < bd) { bd = dd; best = j; }
    }
    if (best < 0 && u->mode == ORK_MODE_LOCAL) {
        if (u->M < u->max_clusters) {
            /* the first new entry founds a cluster of its own: r = k, M2 = 0 */
            int id = u->M++;
            int i = u->n++;
            memcpy(u->K + (size_t)i * d, k, sizeof(double) * d);
            memcpy(u->V + (size_t)i * d, v, sizeof(double) * d);
            u->assign[i] = id;
            memcpy(u->r + (size_t)id * d, k, sizeof(double) * d);
            u->M2[id] = 0.0; u->cnt[id] = 1; u->live[id] = 1; u->hold[id] = 0;
            return id;
        }
        /* no id left: fall back to the nearest cluster of all */
        u->status |= ORK_ST_MAX_CLUSTERS;
        for (int j = 0; j < u->M; j++) {
            if (!u->live[j]) continue;
            double dd = sqdist(k, u->r + (size_t)j * d, d);
            if (best < 0 || dd < bd) { bd = dd; best = j; }
        }
        j0 = 0;
    }
    if (best < 0) return -1;
    if (hint_cluster >= 0 && hint_cluster != best) {
        if (hint_cluster >= j0 && hint_cluster < u->M && u->live[hint_cluster] &&
            near_tie(sqdist(k, u->r + (size_t)hint_cluster * d, d), bd, u->tol)) { best = hint_cluster; u->ties++; }
        else u->violations++;
    }
    int i = u->n++;
    memcpy(u->K + (size_t)i * d, k, sizeof(double) * d);
    memcpy(u->V + (size_t)i * d, v, sizeof(double) * d);
    u->assign[i] = best;
    double *r = u->r + (size_t)best * d;
    int nn = ++u->cnt[best];
    double add = 0.0;
    for (int t = 0; t < d; t++) {
        double delta = k[t] - r[t];
        r[t] += delta / nn;
        add += delta * (k[t] - r[t]);
    }
    u->M2[best] += add;
    u->hold[best] = 0;
    if (u->mode == ORK_MODE_DELAYED && u->flag[best]) u->buf[best]++;     /* an entry for a flagged cluster is buffered */
    return best;
}

/* ------------------------------------------------------ decode: split check */

/* SplitCluster (Algorithm 1; Section 4.2: a flagged cluster is re-clustered locally; Section 5.2: one child keeps
 * growing where the parent was, the other is written elsewhere).  Two-means over the members of cluster j, members in
 * token-id order: centre A = the member farthest from r_j, centre B = the member
 * farthest from A; at most split_iters rounds of (label by nearer centre, ties to A;
 * recompute the two means), stopping early when no label changes.  labels[m] = 0 for A,
 * 1 for B.  Returns 0 if one side ended empty (split abandoned), else 1, and leaves
 * the final centres in cA, cB. */
static int two_means(const ork_unit *u, const int *mem, int nm, unsigned char *labels, double *cA, double *cB) {
    int d = u->d;
    int a = 0, b = 0; double fa = -1.0, fb = -1.0;
    const double *rj = u->r + (size_t)u->assign[mem[0]] * d;
    for (int m = 0; m < nm; m++) { double dd = sqdist(u->K + (size_t)mem[m] * d, rj, d); if (dd > fa) { fa = dd; a = m; } }
    for (int m = 0; m < nm; m++) { double dd = sqdist(u->K + (size_t)mem[m] * d, u->K + (size_t)mem[a] * d, d); if (dd > fb) { fb = dd; b = m; } }
    memcpy(cA, u->K + (size_t)mem[a] * d, sizeof(double) * d);
    memcpy(cB, u->K + (size_t)mem[b] * d, sizeof(double) * d);
    for (int m = 0; m < nm; m++) labels[m] = 255;
    for (int it = 0; it < u->split_iters; it++) {
        int changed = 0, nA = 0, nB = 0;
        for (int m = 0; m < nm; m++) {
            const double *k = u->K + (size_t)mem[m] * d;
            unsigned char l = sqdist(k, cB, d) < sqdist(k, cA, d) ? 1 : 0;
            if (l != labels[m]) changed = 1;
            labels[m] = l;
            if (l) nB++; else nA++;
        }
        if (nA == 0 || nB == 0) return 0;
        if (!changed) break;
        for (int t = 0; t < d; t++) { cA[t] = 0.0; cB[t] = 0.0; }
        for (int m = 0; m < nm; m++) {
            const double *k = u->K + (size_t)mem[m] * d;
            double *c = labels[m] ? cB : cA;
            for (int t = 0; t < d; t++) c[t] += k[t];
        }
        for (int t = 0; t < d; t++) { cA[t] /= nA; cB[t] /= nB; }
    }
    int nA = 0, nB = 0;
    for (int m = 0; m < nm; m++) { if (labels[m]) nB++; else nA++; }
    return nA > 0 && nB > 0;
}

/* Split check over the whole unit.  Snapshot N (tokens) and M_live; a live cluster j is
 * triggered when n_j >= split_min_size, it is not on hold, and
 *     sigma_j^2 = M2_j / n_j > tau                      (the paper's variance rule), or
 *     n_j * M_live > gamma * N                           (size above gamma x the mean size,
 *                                                         the benchmark configuration's rule).
 * Triggered clusters are processed in ascending id, each split once.  The child that
 * contains the smallest token id keeps id j; the other child takes the next free id.
 * Children's n, r, M2 are recomputed from their members.  A split whose 2-means leaves a
 * side empty is abandoned and the cluster is put on hold until its next append.  When
 * max_clusters ids are in use the remaining splits are skipped and a status bit is set.
 * hint_assign_after (optional, [n]) is another implementation's token->cluster map after
 * its own split check.  Returns the number of splits performed. */
int ork_split_check(ork_unit *u, const int *hint_assign_after) {
    int d = u->d, n = u->n, M0 = u->M, done = 0;
    if (u->mode == ORK_MODE_STATIC) return 0;
    int Mlive = 0;
    for (int j = 0; j < M0; j++) Mlive += u->live[j];
    int *mem = (int *)malloc(sizeof(int) * (size_t)(n > 0 ? n : 1));
    unsigned char *labels = (unsigned char *)malloc((size_t)(n > 0 ? n : 1));
    double *cA = (double *)malloc(sizeof(double) * d), *cB = (double *)malloc(sizeof(double) * d);
    /* triggers are evaluated on the state at entry */
    unsigned char *trig = (unsigned char *)calloc((size_t)M0, 1);
    unsigned char *vartie = (unsigned char *)calloc((size_t)M0, 1);
    for (int j = 0; j < M0; j++) {
        if (!u->live[j] || u->hold[j] || u->cnt[j] < u->split_min_size) continue;
        if (u->mode == ORK_MODE_LOCAL) {
            /* only decode-born clusters split, and only by their absolute size */
            trig[j] = j >= u->M_build && u->cnt[j] > u->local_max;
            continue;
        }
        double var = u->M2[j] / u->cnt[j];
        int by_var = u->alpha > 0.0 && var > u->tau;
        int by_size = u->gamma > 0.0 && (double)u->cnt[j] * (double)Mlive > u->gamma * (double)n;
        trig[j] = by_var || by_size;
        vartie[j] = u->alpha > 0.0 && !by_size && near_tie(var, u->tau, u->tol);
    }
    int *order = (int *)malloc(sizeof(int) * (size_t)(M0 + 1));
    int n_order = 0;
    if (u->mode == ORK_MODE_DELAYED) {
        /* Algorithm 1, delayed split.  In the retrieved set: split now, whether the trigger fires at this check or
         * the flag is owed from an earlier one.  Outside it: a firing trigger raises the flag (that entry is the first
         * buffered one).  Then, if the buffered entries of the clusters still flagged reach buf_max, the one with the
         * most of them follows. */
        unsigned char *inreq = (unsigned char *)calloc((size_t)M0, 1);
        for (int i = 0; i < u->n_req; i++) if (u->req[i] >= 0 && u->req[i] < M0) inreq[u->req[i]] = 1;
        for (int j = 0; j < M0; j++) {
            int owed = u->live[j] && u->flag[j];
            if ((trig[j] || owed) && inreq[j]) { trig[j] = 1; order[n_order++] = j; continue; }
            if (trig[j] && !u->flag[j]) { u->flag[j] = 1; u->buf[j] = 1; }
            trig[j] = 0;
        }
        long total = 0; int jmax = -1;
        for (int j = 0; j < M0; j++) {
            if (!u->live[j] || !u->flag[j] || trig[j]) continue;
            total += u->buf[j];
            if (jmax < 0 || u->buf[j] > u->buf[jmax]) jmax = j;
        }
        if (jmax >= 0 && total >= u->buf_max) { trig[jmax] = 1; order[n_order++] = jmax; }
        free(inreq);
    } else {
        for (int j = 0; j < M0; j++) order[n_order++] = j;
    }
    for (int oi = 0; oi < n_order; oi++) {
        int j = order[oi];
        if (!u->live[j]) continue;
        int hinted = 0, hint_split = 0;
        if (hint_assign_after) {
            hinted = 1;
            for (int i = 0; i < n; i++) if (u->assign[i] == j && hint_assign_after[i] != j) { hint_split = 1; break; }
        }
        int want = trig[j];
        if (hinted && hint_split && !want) {
            if (vartie[j] && !u->hold[j] && u->cnt[j] >= u->split_min_size) { want = 1; u->ties++; }
            else { u->violations++; continue; }
        }
        if (!want) continue;
        if (u->M >= u->max_clusters) { u->status |= ORK_ST_MAX_CLUSTERS; continue; }
        int nm = 0;
        for (int i = 0; i < n; i++) if (u->assign[i] == j) mem[nm++] = i;
        int ok = two_means(u, mem, nm, labels, cA, cB);
        if (hinted && !hint_split) {
            /* the other side did not split j: acceptable only as a trigger tie */
            if (!ok) { u->hold[j] = 1; u->flag[j] = 0; u->buf[j] = 0; continue; }
            if (vartie[j]) { u->ties++; continue; }
            u->violations++;
        }
        if (!ok) { u->hold[j] = 1; u->flag[j] = 0; u->buf[j] = 0; continue; }
        /* stay = the side holding the smallest token id (mem[0]) */
        unsigned char stay = labels[0];
        if (hinted && hint_split) {
            for (int m = 0; m < nm; m++) {
                int hint_moves = hint_assign_after[mem[m]] != j;
                int mine_moves = labels[m] != stay;
                if (hint_moves == mine_moves) continue;
                const double *k = u->K + (size_t)mem[m] * d;
                if (near_tie(sqdist(k, cA, d), sqdist(k, cB, d), u->tol)) {
                    labels[m] = hint_moves ? (unsigned char)(1 - stay) : stay; u->ties++;
                } else u->violations++;
            }
        }
        int id = u->M++;
        u->live[id] = 1; u->hold[id] = 0; u->hold[j] = 0;
        u->flag[j] = 0; u->buf[j] = 0; u->flag[id] = 0; u->buf[id] = 0;
        for (int m = 0; m < nm; m++) if (labels[m] != stay) u->assign[mem[m]] = id;
        recompute_stats(u, j);
        recompute_stats(u, id);
        done++; u->n_splits++;
    }
    free(mem); free(labels); free(cA); free(cB); free(trig); free(vartie); free(order);
    return done;
}

/* Install a given partition instead of building one: keys and values in token-id order, the cluster id of
 * every token, and the number of ids in use.  Representatives are recomputed as member means (Eq. 4), M2 as the
 * sum of squared distances to them, both from the members in token-id order (UpdateStats of Algorithm 1); ids
 * without members are dead; tau = alpha * mean live variance, as after a build.  Lets a test continue from
 * another implementation's partition at sizes where running the oracle's own k-means would take minutes. */
int ork_install(ork_unit *u, const double *K, const double *V, int n, const int *assign, int M) {
    int d = u->d;
    if (n > u->max_tokens || M > u->max_clusters || M < 1 || n < 1) return -1;
    for (int i = 0; i < n; i++) if (assign[i] < 0 || assign[i] >= M) return -1;
    memcpy(u->K, K, sizeof(double) * (size_t)n * d);
    memcpy(u->V, V, sizeof(double) * (size_t)n * d);
    memcpy(u->assign, assign, sizeof(int) * (size_t)n);
    u->n = n; u->M = M; u->M_build = M;
    double vs = 0.0; int nl = 0;
    for (int j = 0; j < M; j++) {
        u->hold[j] = 0;
        recompute_stats(u, j);
        u->live[j] = u->cnt[j] > 0;
        if (u->live[j]) { vs += u->M2[j] / u->cnt[j]; nl++; }
    }
    u->tau = nl ? u->alpha * (vs / nl) : 0.0;
    return 0;
}

/* ---------------------------------------------------------------- getters */

int ork_n(const ork_unit *u) { return u->n; }
int ork_M(const ork_unit *u) { return u->M; }
double ork_tau(const ork_unit *u) { return u->tau; }
long ork_ties(const ork_unit *u) { return u->ties; }
long ork_violations(const ork_unit *u) { return u->violations; }
unsigned ork_status(const ork_unit *u) { return u->status; }
long ork_n_splits(const ork_unit *u) { return u->n_splits; }
void ork_get_assign(const ork_unit *u, int *out) { memcpy(out, u->assign, sizeof(int) * (size_t)u->n); }
void ork_get_centroids(const ork_unit *u, double *out) { memcpy(out, u->r, sizeof(double) * (size_t)u->M * u->d); }
void ork_get_counts(const ork_unit *u, int *out) { memcpy(out, u->cnt, sizeof(int) * (size_t)u->M); }
void ork_get_M2(const ork_unit *u, double *out) { memcpy(out, u->M2, sizeof(double) * (size_t)u->M); }
void ork_get_live(const ork_unit *u, unsigned char *out) { memcpy(out, u->live, (size_t)u->M); }
void ork_set_tau(ork_unit *u, double tau) { u->tau = tau; }
void ork_set_mode(ork_unit *u, int mode, int local_max) { u->mode = mode; u->local_max = local_max; }
void ork_set_buf_max(ork_unit *u, int buf_max) { u->buf_max = buf_max; }
void ork_get_flags(const ork_unit *u, unsigned char *flag, int *buf) {
    memcpy(flag, u->flag, (size_t)u->M); memcpy(buf, u->buf, sizeof(int) * (size_t)u->M);
}
