/*
 * pg_oracle.c - plain fp64 CPU restatement of PowerGossip, for CHECKING ONLY.
 *
 * TEST INFRASTRUCTURE.  Nothing in the product path may include, link or call
 * this file: it exists so that the tests, the smoke check and the benchmark's
 * CPU-baseline leg have an independent implementation to compare against.  It
 * shares no code with the CUDA library (own topology builder, own random
 * numbers, own arithmetic) and is deliberately slow and direct: dense loops in
 * double precision, no blocking, no fusion, steps in the order the paper gives.
 *
 * What it follows (Vogels, Karimireddy, Jaggi, "Practical Low-Rank
 * Communication Compression in Decentralized Deep Learning"):
 *   - Section 4, compressor C_v(X) = (X v) v^T and the compressed gossip update
 *     X_i <- X_i + sum_j W_ij C_{v_ij}(X_j - X_i)            (Eq. 2)
 *   - Eq. 3, warm-started power iteration on the pairwise difference
 *   - Algorithm 2, rank-1 s-step PowerGossip: normalise the stored vector, two
 *     local mat-vecs (one per endpoint), subtract, store the result as the next
 *     vector; the next iteration does the same with X transposed
 *   - Assumption A4 on the mixing matrix W (symmetric, doubly stochastic,
 *     non-zero only on edges)
 *   - Appendix "Changing rank vs changing # power iterations": for rank > 1 the
 *     projection matrices are orthogonalised instead of normalised.
 *
 * One "power step" here is two consecutive iterations of Algorithm 2 on an
 * unchanged difference D = X_i - X_j (i < j), the first with the stored right
 * vector(s) Q, the second with X transposed:
 *     Qh = Q with unit columns;  Pm = X_i Qh - X_j Qh;  Ph = orthonormalise(Pm)
 *     Q' = X_i^T Ph - X_j^T Ph;  correction = Ph Q'^T  (= Ph Ph^T D)
 *     X_i <- X_i - W_ij Ph Q'^T,  X_j <- X_j + W_ij Ph Q'^T,  Q <- Q'
 * All edges of a step read the same pre-update X (every neighbour term in
 * Algorithm 1 uses X^(t-1)); with several power steps per round X is updated
 * after every step.
 *
 * Pinned (tests/test_oracle_pins.py): average conservation (Lemma 1), exact
 * removal of a rank-1 difference, brute-force SVD limits, identical workers as
 * a fixed point, full rank == plain gossip W X, monotone consensus distance,
 * schedule structure, Philox known-answer vectors, the paper's printed
 * per-tensor compression ratios.  The numeric trajectory of X over many rounds
 * on generic inputs has no printed worked example in the paper: beyond those
 * pins it is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PGO_RING 0
#define PGO_TORUS 1
#define PGO_MATCHING 2
#define PGO_CUSTOM 3

#define PGO_W_UNIFORM 0
#define PGO_W_METROPOLIS 1
#define PGO_W_EXPLICIT 2

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), from its definition.    */
/* ------------------------------------------------------------------------- */
void pgo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Algorithm 2, initialisation: every entry of the per-edge vector is standard
 * normal.  Entry e of column k of the vector that the pair (i<j) keeps for
 * layer l is a pure function of (seed, i, j, l, k, e): Philox block e/4 with
 * counter (e/4, l, i, j*256+k), two Box-Muller pairs per block, rounded to
 * fp32 (the CUDA side stores fp32, and both sides must start from equal bits). */
void pgo_init_q(uint64_t seed, int i, int j, int layer, int col, int m, float *out)
{
    const double two_pi = 6.283185307179586476925286766559;
    const double scale = 1.0 / 4294967296.0;
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int b = 0; 4 * b < m; ++b) {
        uint32_t ctr[4] = { (uint32_t)b, (uint32_t)layer, (uint32_t)i,
                            (uint32_t)j * 256u + (uint32_t)col };
        uint32_t x[4];
        double z[4];
        pgo_philox4x32_10(ctr, key, x);
        for (int h = 0; h < 2; ++h) {
            double u1 = ((double)x[2 * h] + 0.5) * scale;
            double u2 = ((double)x[2 * h + 1] + 0.5) * scale;
            double r = sqrt(-2.0 * log(u1));
            z[2 * h] = r * cos(two_pi * u2);
            z[2 * h + 1] = r * sin(two_pi * u2);
        }
        for (int t = 0; t < 4 && 4 * b + t < m; ++t) out[4 * b + t] = (float)z[t];
    }
}

/* ------------------------------------------------------------------------- */
/* Topology: canonical edge lists ((min,max) pairs, sorted lexicographically). */
/* ------------------------------------------------------------------------- */
static int cmp_edge(const void *a, const void *b)
{
    const int *x = (const int *)a, *y = (const int *)b;
    if (x[0] != y[0]) return x[0] < y[0] ? -1 : 1;
    if (x[1] != y[1]) return x[1] < y[1] ? -1 : 1;
    return 0;
}

static int canonicalise(int *edges, int n)
{
    /* order each pair, drop self loops, sort, drop duplicates */
    int k = 0;
    for (int e = 0; e < n; ++e) {
        int a = edges[2 * e], b = edges[2 * e + 1];
        if (a == b) continue;
        edges[2 * k] = a < b ? a : b;
        edges[2 * k + 1] = a < b ? b : a;
        ++k;
    }
    qsort(edges, (size_t)k, 2 * sizeof(int), cmp_edge);
    int u = 0;
    for (int e = 0; e < k; ++e) {
        if (u > 0 && edges[2 * (u - 1)] == edges[2 * e] && edges[2 * (u - 1) + 1] == edges[2 * e + 1]) continue;
        edges[2 * u] = edges[2 * e];
        edges[2 * u + 1] = edges[2 * e + 1];
        ++u;
    }
    return u;
}

/* Edge list of round `round`.  edges_out must hold 2*max(2*N, n_custom) ints.
 * Returns the number of edges, or -1 for an invalid request.
 *   ring      : {i, (i+1) mod N}
 *   torus RxC : worker id = r*C + c; right and down neighbours with wrap-around
 *   matching  : Fisher-Yates shuffle of 0..N-1 (position k from N-1 down to 1
 *               swaps with index  r mod (k+1),  r = the low 64 bits of Philox
 *               at counter (k, round_lo, round_hi, 0xFFFFFFFF) keyed by the
 *               seed); consecutive entries are paired.  N must be even.
 *   custom    : the caller's list, canonicalised. */
int pgo_schedule(int kind, int N, int trows, int tcols, const int *custom, int n_custom,
                 uint64_t seed, int64_t round, int *edges_out)
{
    int n = 0;
    if (N < 1) return -1;
    if (kind == PGO_RING) {
        for (int i = 0; i < N; ++i) { edges_out[2 * n] = i; edges_out[2 * n + 1] = (i + 1) % N; ++n; }
    } else if (kind == PGO_TORUS) {
        if (trows < 1 || tcols < 1 || trows * tcols != N) return -1;
        for (int r = 0; r < trows; ++r)
            for (int c = 0; c < tcols; ++c) {
                int id = r * tcols + c;
                edges_out[2 * n] = id; edges_out[2 * n + 1] = r * tcols + (c + 1) % tcols; ++n;
                edges_out[2 * n] = id; edges_out[2 * n + 1] = ((r + 1) % trows) * tcols + c; ++n;
            }
    } else if (kind == PGO_MATCHING) {
        if (N % 2 != 0) return -1;
        int *perm = (int *)malloc(sizeof(int) * (size_t)N);
        uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
        for (int i = 0; i < N; ++i) perm[i] = i;
        for (int k = N - 1; k >= 1; --k) {
            uint32_t ctr[4] = { (uint32_t)k, (uint32_t)((uint64_t)round & 0xFFFFFFFFu),
                                (uint32_t)((uint64_t)round >> 32), 0xFFFFFFFFu };
            uint32_t x[4];
            pgo_philox4x32_10(ctr, key, x);
            uint64_t r = (uint64_t)x[0] | ((uint64_t)x[1] << 32);
            int j = (int)(r % (uint64_t)(k + 1));
            int t = perm[k]; perm[k] = perm[j]; perm[j] = t;
        }
        for (int a = 0; a < N / 2; ++a) { edges_out[2 * n] = perm[2 * a]; edges_out[2 * n + 1] = perm[2 * a + 1]; ++n; }
        free(perm);
    } else if (kind == PGO_CUSTOM) {
        for (int e = 0; e < n_custom; ++e) {
            if (custom[2 * e] < 0 || custom[2 * e] >= N || custom[2 * e + 1] < 0 || custom[2 * e + 1] >= N) return -1;
            edges_out[2 * n] = custom[2 * e]; edges_out[2 * n + 1] = custom[2 * e + 1]; ++n;
        }
    } else {
        return -1;
    }
    return canonicalise(edges_out, n);
}

/* Gossip weight of every edge of a list (Assumption A4: symmetric, rows sum to
 * one with the self weight making up the rest).
 *   uniform    : 1 / (max degree + 1)
 *   Metropolis : 1 / (1 + max(deg_i, deg_j))
 *   explicit   : W[i*N + j]; must be symmetric, >= 0 off the diagonal, zero off
 *                the edge list and every row must sum to 1 (1e-5).
 * Returns 0, or -1 when an explicit matrix breaks A4. */
int pgo_edge_weights(int rule, int N, const int *edges, int E, const float *W, int allow_zero, double *w_out)
{
    int *deg = (int *)calloc((size_t)N, sizeof(int));
    int maxdeg = 0, rc = 0;
    for (int e = 0; e < E; ++e) { deg[edges[2 * e]]++; deg[edges[2 * e + 1]]++; }
    for (int i = 0; i < N; ++i) if (deg[i] > maxdeg) maxdeg = deg[i];
    if (rule == PGO_W_UNIFORM) {
        for (int e = 0; e < E; ++e) w_out[e] = 1.0 / (double)(maxdeg + 1);
    } else if (rule == PGO_W_METROPOLIS) {
        for (int e = 0; e < E; ++e) {
            int a = deg[edges[2 * e]], b = deg[edges[2 * e + 1]];
            w_out[e] = 1.0 / (double)(1 + (a > b ? a : b));
        }
    } else if (rule == PGO_W_EXPLICIT && W != NULL) {
        char *is_edge = (char *)calloc((size_t)N * (size_t)N, 1);
        for (int e = 0; e < E; ++e) {
            int i = edges[2 * e], j = edges[2 * e + 1];
            is_edge[(size_t)i * N + j] = is_edge[(size_t)j * N + i] = 1;
            w_out[e] = (double)W[(size_t)i * N + j];
            if (!allow_zero && !(W[(size_t)i * N + j] > 0.0f)) rc = -1;
        }
        for (int i = 0; i < N; ++i) {
            double s = 0.0;
            for (int j = 0; j < N; ++j) {
                float a = W[(size_t)i * N + j];
                s += (double)a;
                if (a != W[(size_t)j * N + i]) rc = -1;
                if (i != j && a != 0.0f && !is_edge[(size_t)i * N + j]) rc = -1;
                if (i != j && a < 0.0f) rc = -1;
            }
            if (fabs(s - 1.0) > 1e-5) rc = -1;
        }
        free(is_edge);
    } else {
        rc = -1;
    }
    free(deg);
    return rc;
}

/* ------------------------------------------------------------------------- */
/* The network state and one gossip round.                                    */
/* ------------------------------------------------------------------------- */
typedef struct pgo_ctx {
    int N, L, rank, power_steps;
    int kind, trows, tcols, rule;
    int n_custom;
    int *custom;
    float *W;            /* explicit mixing matrix or NULL */
    uint64_t seed;
    int64_t round;
    int *rows, *cols;
    double **X;          /* X[i*L + l]: rows x cols, row-major */
    double **Q;          /* Q[pair*L + l]: rank columns of length cols, NULL until first met */
    double **Ph;         /* last orthonormal left factor of the pair: rank columns of length rows */
    int max_edges;
    int half_step;       /* 1: Algorithm 2 read literally, one mat-vec per iteration */
    int random_proj;     /* 0: power iteration; 1: random right projections R_k; 2: random left projections */
    int64_t step;        /* random projections: steps taken so far (keys the directions) */
    int64_t iteration;   /* half-step mode: Algorithm 2's counter k (shared: all pairs move in lockstep) */
    /* diagnostics and test aids; neither changes what a power step computes */
    double min_resid_ratio;  /* smallest (residual norm / norm before projection)^2 met at a column k > 0 */
    int fp32_storage;        /* 1: X and Q are rounded to fp32 after every power step (see pgo_set_fp32_storage) */
} pgo_ctx;

static size_t pair_index(int N, int i, int j)  /* i < j, over all N(N-1)/2 pairs */
{
    return (size_t)i * (size_t)N - (size_t)i * ((size_t)i + 1) / 2 + (size_t)(j - i - 1);
}

void pgo_destroy(pgo_ctx *c);

pgo_ctx *pgo_create(int kind, int N, int trows, int tcols, const int *custom, int n_custom,
                    int rule, const float *W, const int *shapes, int L, int rank,
                    int power_steps, uint64_t seed)
{
    if (N < 2 || L < 1 || rank < 1 || power_steps < 1) return NULL;
    pgo_ctx *c = (pgo_ctx *)calloc(1, sizeof(pgo_ctx));
    c->N = N; c->L = L; c->rank = rank; c->power_steps = power_steps;
    c->kind = kind; c->trows = trows; c->tcols = tcols; c->rule = rule;
    c->seed = seed; c->round = 0;
    c->min_resid_ratio = INFINITY;
    c->n_custom = n_custom;
    if (n_custom > 0) {
        c->custom = (int *)malloc(sizeof(int) * 2 * (size_t)n_custom);
        memcpy(c->custom, custom, sizeof(int) * 2 * (size_t)n_custom);
    }
    if (W != NULL) {
        c->W = (float *)malloc(sizeof(float) * (size_t)N * (size_t)N);
        memcpy(c->W, W, sizeof(float) * (size_t)N * (size_t)N);
    }
    c->rows = (int *)malloc(sizeof(int) * (size_t)L);
    c->cols = (int *)malloc(sizeof(int) * (size_t)L);
    for (int l = 0; l < L; ++l) { c->rows[l] = shapes[2 * l]; c->cols[l] = shapes[2 * l + 1]; }
    c->X = (double **)calloc((size_t)N * (size_t)L, sizeof(double *));
    for (int i = 0; i < N; ++i)
        for (int l = 0; l < L; ++l)
            c->X[(size_t)i * L + l] = (double *)calloc((size_t)c->rows[l] * (size_t)c->cols[l], sizeof(double));
    size_t n_pairs = (size_t)N * (size_t)(N - 1) / 2;
    c->Q = (double **)calloc(n_pairs * (size_t)L, sizeof(double *));
    c->Ph = (double **)calloc(n_pairs * (size_t)L, sizeof(double *));
    c->max_edges = 2 * N > n_custom ? 2 * N : n_custom;
    /* reject invalid topologies / mixing matrices up front */
    int *edges = (int *)malloc(sizeof(int) * 2 * (size_t)c->max_edges);
    double *w = (double *)malloc(sizeof(double) * (size_t)c->max_edges);
    int E = pgo_schedule(kind, N, trows, tcols, c->custom, n_custom, seed, 0, edges);
    int ok = E >= 0;
    if (ok && kind != PGO_MATCHING)
        ok = pgo_edge_weights(rule, N, edges, E, c->W, kind == PGO_CUSTOM, w) == 0;
    free(edges); free(w);
    if (!ok) { pgo_destroy(c); return NULL; }
    return c;
}

void pgo_destroy(pgo_ctx *c)
{
    if (!c) return;
    size_t n_pairs = (size_t)c->N * (size_t)(c->N - 1) / 2;
    for (size_t t = 0; t < (size_t)c->N * (size_t)c->L; ++t) free(c->X[t]);
    for (size_t t = 0; t < n_pairs * (size_t)c->L; ++t) { free(c->Q[t]); free(c->Ph[t]); }
    free(c->X); free(c->Q); free(c->Ph); free(c->rows); free(c->cols); free(c->custom); free(c->W);
    free(c);
}

static double *q_of(pgo_ctx *c, int i, int j, int l)   /* i < j; drawn on first use */
{
    size_t t = pair_index(c->N, i, j) * (size_t)c->L + (size_t)l;
    if (c->Q[t] == NULL) {
        int m = c->cols[l];
        float *tmp = (float *)malloc(sizeof(float) * (size_t)m);
        /* in half-step mode the vector alternates between R^cols and R^rows: room for both */
        size_t room = (size_t)m * (size_t)c->rank;
        if (c->half_step && (size_t)c->rows[l] > room) room = (size_t)c->rows[l];
        c->Q[t] = (double *)calloc(room, sizeof(double));
        for (int k = 0; k < c->rank; ++k) {
            pgo_init_q(c->seed, i, j, l, k, m, tmp);
            for (int e = 0; e < m; ++e) c->Q[t][(size_t)k * m + e] = (double)tmp[e];
        }
        free(tmp);
    }
    return c->Q[t];
}

int pgo_set_params(pgo_ctx *c, int i, int l, const float *src)
{
    if (!c || i < 0 || i >= c->N || l < 0 || l >= c->L) return -1;
    size_t cnt = (size_t)c->rows[l] * (size_t)c->cols[l];
    double *x = c->X[(size_t)i * c->L + l];
    for (size_t t = 0; t < cnt; ++t) x[t] = (double)src[t];
    return 0;
}

/* Algorithm 1's local term: X_i <- X_i + delta (the caller passes -eta * G). */
int pgo_add_params(pgo_ctx *c, int i, int l, const double *delta)
{
    if (!c || i < 0 || i >= c->N || l < 0 || l >= c->L) return -1;
    size_t cnt = (size_t)c->rows[l] * (size_t)c->cols[l];
    double *x = c->X[(size_t)i * c->L + l];
    for (size_t t = 0; t < cnt; ++t) x[t] += delta[t];
    return 0;
}

int pgo_get_params(pgo_ctx *c, int i, int l, double *dst)
{
    if (!c || i < 0 || i >= c->N || l < 0 || l >= c->L) return -1;
    memcpy(dst, c->X[(size_t)i * c->L + l], sizeof(double) * (size_t)c->rows[l] * (size_t)c->cols[l]);
    return 0;
}

/* column-major: dst[k*cols + e] */
int pgo_get_q(pgo_ctx *c, int i, int j, int l, double *dst)
{
    if (!c || i == j || i < 0 || j < 0 || i >= c->N || j >= c->N || l < 0 || l >= c->L) return -1;
    int a = i < j ? i : j, b = i < j ? j : i;
    memcpy(dst, q_of(c, a, b, l), sizeof(double) * (size_t)c->cols[l] * (size_t)c->rank);
    return 0;
}

int pgo_set_q(pgo_ctx *c, int i, int j, int l, const double *src)
{
    if (!c || i == j || i < 0 || j < 0 || i >= c->N || j >= c->N || l < 0 || l >= c->L) return -1;
    int a = i < j ? i : j, b = i < j ? j : i;
    memcpy(q_of(c, a, b, l), src, sizeof(double) * (size_t)c->cols[l] * (size_t)c->rank);
    return 0;
}

/* last orthonormal left factor of the pair (rank columns of length rows);
 * returns -1 if the pair has not been an edge yet */
int pgo_get_phat(pgo_ctx *c, int i, int j, int l, double *dst)
{
    if (!c || i == j || i < 0 || j < 0 || i >= c->N || j >= c->N || l < 0 || l >= c->L) return -1;
    int a = i < j ? i : j, b = i < j ? j : i;
    double *p = c->Ph[pair_index(c->N, a, b) * (size_t)c->L + (size_t)l];
    if (!p) return -1;
    memcpy(dst, p, sizeof(double) * (size_t)c->rows[l] * (size_t)c->rank);
    return 0;
}

int64_t pgo_get_round(pgo_ctx *c) { return c ? c->round : -1; }
void pgo_set_round(pgo_ctx *c, int64_t r) { if (c) c->round = r; }

int pgo_round_schedule(pgo_ctx *c, int64_t round, int *edges_out, double *w_out)
{
    int E = pgo_schedule(c->kind, c->N, c->trows, c->tcols, c->custom, c->n_custom, c->seed, round, edges_out);
    if (E < 0) return -1;
    if (c->kind == PGO_MATCHING) {
        /* a matched pair has degree one: Metropolis weight 1/(1+1), self weight 1/2 */
        for (int e = 0; e < E; ++e) w_out[e] = 0.5;
    } else if (pgo_edge_weights(c->rule, c->N, edges_out, E, c->W, c->kind == PGO_CUSTOM, w_out) != 0) {
        return -1;
    }
    return E;
}

/* y (n) = A (n x m, row-major) times v (m) */
static void matvec(const double *A, int n, int m, const double *v, double *y)
{
    for (int r = 0; r < n; ++r) {
        double s = 0.0;
        const double *a = A + (size_t)r * m;
        for (int cidx = 0; cidx < m; ++cidx) s += a[cidx] * v[cidx];
        y[r] = s;
    }
}

/* y (m) = A^T (A is n x m, row-major) times v (n) */
static void matvec_t(const double *A, int n, int m, const double *v, double *y)
{
    for (int cidx = 0; cidx < m; ++cidx) y[cidx] = 0.0;
    for (int r = 0; r < n; ++r) {
        const double *a = A + (size_t)r * m;
        double vr = v[r];
        for (int cidx = 0; cidx < m; ++cidx) y[cidx] += a[cidx] * vr;
    }
}

static double dot(const double *a, const double *b, int n)
{
    double s = 0.0;
    for (int t = 0; t < n; ++t) s += a[t] * b[t];
    return s;
}

/* One power step of one edge on one layer: fills Ph (n x rank, column-major),
 * Qn (m x rank, column-major) and live[k] (0 when column k was degenerate). */
static void edge_power_step(const double *Xi, const double *Xj, int n, int m, int rank,
                            const double *Q, double *Ph, double *Qn, int *live, double *min_ratio)
{
    double *qh = (double *)malloc(sizeof(double) * (size_t)m);
    double *pi = (double *)malloc(sizeof(double) * (size_t)n);
    double *pj = (double *)malloc(sizeof(double) * (size_t)n);
    double *qi = (double *)malloc(sizeof(double) * (size_t)m);
    double *qj = (double *)malloc(sizeof(double) * (size_t)m);
    for (int k = 0; k < rank; ++k) {
        /* Algorithm 2: v_hat = v / ||v|| (a zero vector stays zero) */
        const double *q = Q + (size_t)k * m;
        double nq = sqrt(dot(q, q, m));
        for (int e = 0; e < m; ++e) qh[e] = nq > 0.0 ? q[e] / nq : 0.0;
        /* p_i = X_i v_hat and p_j = X_j v_hat on the two nodes, then the difference */
        matvec(Xi, n, m, qh, pi);
        matvec(Xj, n, m, qh, pj);
        double *p = Ph + (size_t)k * n;
        for (int r = 0; r < n; ++r) p[r] = pi[r] - pj[r];
        /* Eq. 3 normalisation; for rank > 1 orthogonalise against the earlier
         * columns first (modified Gram-Schmidt, column order 0..rank-1) */
        double pre = dot(p, p, n);
        for (int h = 0; h < k; ++h) {
            const double *ph = Ph + (size_t)h * n;
            double a = dot(ph, p, n);
            for (int r = 0; r < n; ++r) p[r] -= a * ph[r];
        }
        double nn = dot(p, p, n);
        /* a column that is zero, or (for k > 0) whose residual has dropped below
         * 1e-5 of its length before projection (it was, to fp32 working accuracy,
         * a linear combination of the earlier columns: what is left has no
         * meaningful direction), contributes nothing and keeps its vector */
        int ok = (nn > 0.0) && isfinite(nn) && (k == 0 || nn > 1e-10 * pre);
        if (k > 0 && pre > 0.0 && isfinite(nn) && nn / pre < *min_ratio) *min_ratio = nn / pre;   /* diagnostic only */
        live[k] = ok;
        double inv = ok ? 1.0 / sqrt(nn) : 0.0;
        for (int r = 0; r < n; ++r) p[r] = ok ? p[r] * inv : 0.0;
    }
    for (int k = 0; k < rank; ++k) {
        /* the even iteration: same with X transposed, starting from the unit vector */
        const double *p = Ph + (size_t)k * n;
        matvec_t(Xi, n, m, p, qi);
        matvec_t(Xj, n, m, p, qj);
        for (int e = 0; e < m; ++e) Qn[(size_t)k * m + e] = qi[e] - qj[e];
    }
    free(qh); free(pi); free(pj); free(qi); free(qj);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2 read literally ("half-step mode").                             */
/*                                                                           */
/* Every iteration is ONE mat-vec and ONE gossip update with that iteration's */
/* approximation; `power_steps` is the algorithm's s, the iterations per      */
/* round.  With D = X_i - X_j (i < j), counter k:                             */
/*   k odd : vh = v/||v|| in R^cols;  p = X_i vh - X_j vh;                     */
/*           X_i -= W p vh^T,  X_j += W p vh^T;   v <- p      (now in R^rows) */
/*   k even: the same with X transposed: vh in R^rows;  q = X_i^T vh - X_j^T vh */
/*           X_i -= W vh q^T,  X_j += W vh q^T;   v <- q      (now in R^cols) */
/* One iteration moves (rows+cols)/2 floats per edge direction on average,    */
/* which is what the paper's per-tensor compression ratios count.  Rank 1 and */
/* static graphs only (all pairs share k).  A zero vector normalises to zero  */
/* (0/||0|| := 0), so an edge whose ends agree exactly stays silent.          */
/* ------------------------------------------------------------------------- */
int pgo_set_half_step(pgo_ctx *c, int on)
{
    if (!c) return -1;
    if (on && (c->rank != 1 || c->kind == PGO_MATCHING || c->round != 0)) return -1;
    c->half_step = on ? 1 : 0;
    c->iteration = 0;
    return 0;
}

/* current vector of the pair: rows entries after an odd iteration, cols after an
 * even one (or before the first); returns its length, or -1 */
int pgo_get_vector(pgo_ctx *c, int i, int j, int l, double *dst)
{
    if (!c || i == j || i < 0 || j < 0 || i >= c->N || j >= c->N || l < 0 || l >= c->L) return -1;
    int a = i < j ? i : j, b = i < j ? j : i;
    int len = (c->half_step && (c->iteration % 2 == 1)) ? c->rows[l] : c->cols[l];
    memcpy(dst, q_of(c, a, b, l), sizeof(double) * (size_t)len);
    return len;
}

static int half_step_round(pgo_ctx *c)
{
    int *edges = (int *)malloc(sizeof(int) * 2 * (size_t)c->max_edges);
    double *w = (double *)malloc(sizeof(double) * (size_t)c->max_edges);
    int E = pgo_round_schedule(c, c->round, edges, w);
    if (E < 0) { free(edges); free(w); return -1; }
    for (int e = 0; e < E; ++e)
        for (int l = 0; l < c->L; ++l) (void)q_of(c, edges[2 * e], edges[2 * e + 1], l);
    double **out = (double **)calloc((size_t)E * (size_t)c->L, sizeof(double *));
    double **vh = (double **)calloc((size_t)E * (size_t)c->L, sizeof(double *));
    for (int it = 0; it < c->power_steps; ++it) {
        c->iteration += 1;
        const int odd = (int)(c->iteration % 2);
        /* every edge forms its vector from the same pre-update X */
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
        for (int l = 0; l < c->L; ++l)
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                int n = c->rows[l], m = c->cols[l];
                int len_in = odd ? m : n, len_out = odd ? n : m;
                size_t t = pair_index(c->N, i, j) * (size_t)c->L + (size_t)l;
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                const double *v = c->Q[t];
                double nv = sqrt(dot(v, v, len_in));
                vh[u] = (double *)malloc(sizeof(double) * (size_t)len_in);
                for (int a = 0; a < len_in; ++a) vh[u][a] = (nv > 0.0 && isfinite(nv)) ? v[a] / nv : 0.0;
                double *pi = (double *)malloc(sizeof(double) * (size_t)len_out);
                double *pj = (double *)malloc(sizeof(double) * (size_t)len_out);
                const double *Xi = c->X[(size_t)i * c->L + l], *Xj = c->X[(size_t)j * c->L + l];
                if (odd) { matvec(Xi, n, m, vh[u], pi); matvec(Xj, n, m, vh[u], pj); }
                else     { matvec_t(Xi, n, m, vh[u], pi); matvec_t(Xj, n, m, vh[u], pj); }
                for (int a = 0; a < len_out; ++a) pi[a] -= pj[a];
                out[u] = pi;
                free(pj);
            }
        /* the update of this iteration, then the vector moves to the other space */
        for (int l = 0; l < c->L; ++l) {
            int n = c->rows[l], m = c->cols[l];
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                size_t t = pair_index(c->N, i, j) * (size_t)c->L + (size_t)l;
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                double *Xi = c->X[(size_t)i * c->L + l], *Xj = c->X[(size_t)j * c->L + l];
                const double *left = odd ? out[u] : vh[u];     /* length rows */
                const double *right = odd ? vh[u] : out[u];    /* length cols */
                for (int r = 0; r < n; ++r) {
                    double a = w[e] * left[r];
                    for (int cidx = 0; cidx < m; ++cidx) {
                        double d = a * right[cidx];
                        Xi[(size_t)r * m + cidx] = Xi[(size_t)r * m + cidx] - d;   /* what i loses ... */
                        Xj[(size_t)r * m + cidx] = Xj[(size_t)r * m + cidx] + d;   /* ... j gains */
                    }
                }
                memcpy(c->Q[t], out[u], sizeof(double) * (size_t)(odd ? n : m));
                free(out[u]); free(vh[u]);
                out[u] = vh[u] = NULL;
            }
        }
    }
    free(out); free(vh); free(edges); free(w);
    c->round += 1;
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Random-projection compressors (Section 5.1, the examples after A5).        */
/*   right:  R_k(X) = (X U) U^T,  U a uniformly drawn orthonormal cols x k      */
/*   left :  L_k(X) = V (V^T X),  V a uniformly drawn orthonormal rows x k      */
/* A fresh direction set per edge, layer and step; nothing is warm-started.    */
/* Directions: entry e of column c for pair (i<j), layer l, step t is the same  */
/* Philox/Box-Muller normal as the initial vectors, with the key               */
/* (seed_lo ^ low32(t+1), seed_hi ^ high32(t+1) ^ 0x52503031), rounded to fp32; */
/* the columns are then orthonormalised (modified Gram-Schmidt, same dependent- */
/* column rule as the power step), which makes them uniform on the Stiefel      */
/* manifold.  delta of A5 is k/cols (right) or k/rows (left).                   */
/* ------------------------------------------------------------------------- */
int pgo_set_random_projection(pgo_ctx *c, int mode)
{
    if (!c || mode < 0 || mode > 2 || c->round != 0 || c->half_step) return -1;
    c->random_proj = mode;
    c->step = 0;
    return 0;
}

/* the orthonormal directions of one (pair, layer, step): len x rank, column-major, fp64 */
void pgo_random_directions(uint64_t seed, int64_t step, int i, int j, int layer, int len, int rank, double *out)
{
    uint64_t t1 = (uint64_t)step + 1u;
    uint64_t key = seed ^ (t1 & 0xFFFFFFFFu) ^ (((t1 >> 32) ^ 0x52503031u) << 32);
    float *tmp = (float *)malloc(sizeof(float) * (size_t)len);
    for (int k = 0; k < rank; ++k) {
        double *u = out + (size_t)k * len;
        pgo_init_q(key, i, j, layer, k, len, tmp);
        for (int e = 0; e < len; ++e) u[e] = (double)tmp[e];
        double pre = dot(u, u, len);
        for (int h = 0; h < k; ++h) {
            const double *uh = out + (size_t)h * len;
            double a = dot(uh, u, len);
            for (int e = 0; e < len; ++e) u[e] -= a * uh[e];
        }
        double nn = dot(u, u, len);
        int ok = (nn > 0.0) && isfinite(nn) && (k == 0 || nn > 1e-10 * pre);
        double inv = ok ? 1.0 / sqrt(nn) : 0.0;
        for (int e = 0; e < len; ++e) u[e] = ok ? u[e] * inv : 0.0;
    }
    free(tmp);
}

static int random_projection_round(pgo_ctx *c)
{
    int *edges = (int *)malloc(sizeof(int) * 2 * (size_t)c->max_edges);
    double *w = (double *)malloc(sizeof(double) * (size_t)c->max_edges);
    int E = pgo_round_schedule(c, c->round, edges, w);
    if (E < 0) { free(edges); free(w); return -1; }
    const int rank = c->rank, right = c->random_proj == 1;
    double **dirs = (double **)calloc((size_t)E * (size_t)c->L, sizeof(double *));
    double **prod = (double **)calloc((size_t)E * (size_t)c->L, sizeof(double *));
    for (int step = 0; step < c->power_steps; ++step) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
        for (int l = 0; l < c->L; ++l)
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                int n = c->rows[l], m = c->cols[l];
                int len_in = right ? m : n, len_out = right ? n : m;
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                dirs[u] = (double *)malloc(sizeof(double) * (size_t)len_in * (size_t)rank);
                prod[u] = (double *)malloc(sizeof(double) * (size_t)len_out * (size_t)rank);
                pgo_random_directions(c->seed, c->step, i, j, l, len_in, rank, dirs[u]);
                double *tmp = (double *)malloc(sizeof(double) * (size_t)len_out);
                const double *Xi = c->X[(size_t)i * c->L + l], *Xj = c->X[(size_t)j * c->L + l];
                for (int k = 0; k < rank; ++k) {
                    double *o = prod[u] + (size_t)k * len_out;
                    const double *d = dirs[u] + (size_t)k * len_in;
                    if (right) { matvec(Xi, n, m, d, o); matvec(Xj, n, m, d, tmp); }
                    else       { matvec_t(Xi, n, m, d, o); matvec_t(Xj, n, m, d, tmp); }
                    for (int a = 0; a < len_out; ++a) o[a] -= tmp[a];
                }
                free(tmp);
            }
        for (int l = 0; l < c->L; ++l) {
            int n = c->rows[l], m = c->cols[l];
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                double *Xi = c->X[(size_t)i * c->L + l], *Xj = c->X[(size_t)j * c->L + l];
                for (int k = 0; k < rank; ++k) {
                    const double *left = right ? prod[u] + (size_t)k * n : dirs[u] + (size_t)k * n;
                    const double *rightv = right ? dirs[u] + (size_t)k * m : prod[u] + (size_t)k * m;
                    for (int r = 0; r < n; ++r) {
                        double a = w[e] * left[r];
                        for (int cidx = 0; cidx < m; ++cidx) {
                            double d = a * rightv[cidx];
                            Xi[(size_t)r * m + cidx] = Xi[(size_t)r * m + cidx] - d;   /* taken from i ...   */
                            Xj[(size_t)r * m + cidx] = d + Xj[(size_t)r * m + cidx];   /* ... and given to j */
                        }
                    }
                }
                free(dirs[u]); free(prod[u]);
                dirs[u] = prod[u] = NULL;
            }
        }
        c->step += 1;
    }
    free(dirs); free(prod); free(edges); free(w);
    c->round += 1;
    return 0;
}

/* Diagnostic: the smallest squared ratio (Gram-Schmidt residual / column before
 * projection) met so far at any column k > 0; +inf if none was met.  The
 * dependent-column rule compares this ratio with 1e-10, so a run whose minimum
 * stays far above that threshold would have taken the same decisions under any
 * smaller threshold. */
double pgo_min_residual_ratio(pgo_ctx *c) { return c ? c->min_resid_ratio : -1.0; }

/* Test aid, NOT part of the method: with this on, every entry of X and of the
 * vectors of this round's pairs is rounded to fp32 and widened again after every
 * power step, while all arithmetic stays in fp64.  That is the least
 * perturbation any implementation that stores its state in fp32 applies to the
 * iteration; a test runs this beside the untouched fp64 run to see how far such
 * an implementation can be expected to drift.  Power-iteration mode only. */
int pgo_set_fp32_storage(pgo_ctx *c, int on)
{
    if (!c || c->half_step || c->random_proj) return -1;
    c->fp32_storage = on ? 1 : 0;
    return 0;
}

static void round_state_to_fp32(pgo_ctx *c, const int *edges, int E)
{
    for (int i = 0; i < c->N; ++i)
        for (int l = 0; l < c->L; ++l) {
            double *x = c->X[(size_t)i * c->L + l];
            size_t cnt = (size_t)c->rows[l] * (size_t)c->cols[l];
            for (size_t t = 0; t < cnt; ++t) x[t] = (double)(float)x[t];
        }
    for (int e = 0; e < E; ++e)
        for (int l = 0; l < c->L; ++l) {
            double *q = c->Q[pair_index(c->N, edges[2 * e], edges[2 * e + 1]) * (size_t)c->L + (size_t)l];
            size_t cnt = (size_t)c->cols[l] * (size_t)c->rank;
            for (size_t t = 0; t < cnt; ++t) q[t] = (double)(float)q[t];
        }
}

/* One gossip round = power_steps power steps on every layer and every edge of
 * this round's graph.  Returns 0, or -1 on an invalid schedule. */
int pgo_round(pgo_ctx *c)
{
    if (c->half_step) return half_step_round(c);
    if (c->random_proj) return random_projection_round(c);
    int *edges = (int *)malloc(sizeof(int) * 2 * (size_t)c->max_edges);
    double *w = (double *)malloc(sizeof(double) * (size_t)c->max_edges);
    int E = pgo_round_schedule(c, c->round, edges, w);
    if (E < 0) { free(edges); free(w); return -1; }
    int rank = c->rank;
    /* make sure every per-pair state exists before the parallel region */
    for (int e = 0; e < E; ++e)
        for (int l = 0; l < c->L; ++l) {
            size_t t = pair_index(c->N, edges[2 * e], edges[2 * e + 1]) * (size_t)c->L + (size_t)l;
            (void)q_of(c, edges[2 * e], edges[2 * e + 1], l);
            if (!c->Ph[t]) c->Ph[t] = (double *)calloc((size_t)c->rows[l] * (size_t)rank, sizeof(double));
        }
    double **Qn = (double **)calloc((size_t)E * (size_t)c->L, sizeof(double *));
    int *live = (int *)calloc((size_t)E * (size_t)c->L * (size_t)rank, sizeof(int));
    for (int step = 0; step < c->power_steps; ++step) {
        /* phase 1: every edge computes its factors from the same pre-update X */
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
        for (int l = 0; l < c->L; ++l)
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                int n = c->rows[l], m = c->cols[l];
                size_t t = pair_index(c->N, i, j) * (size_t)c->L + (size_t)l;
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                Qn[u] = (double *)malloc(sizeof(double) * (size_t)m * (size_t)rank);
                double ratio = INFINITY;
                edge_power_step(c->X[(size_t)i * c->L + l], c->X[(size_t)j * c->L + l], n, m, rank,
                                c->Q[t], c->Ph[t], Qn[u], live + u * (size_t)rank, &ratio);
#pragma omp critical(pgo_min_ratio)
                if (ratio < c->min_resid_ratio) c->min_resid_ratio = ratio;
            }
        /* phase 2: X_i <- X_i - W_ij Ph Q'^T and X_j <- X_j + W_ij Ph Q'^T (what
         * is added to one endpoint is subtracted from the other), Q <- Q' */
        for (int l = 0; l < c->L; ++l) {
            int n = c->rows[l], m = c->cols[l];
            for (int e = 0; e < E; ++e) {
                int i = edges[2 * e], j = edges[2 * e + 1];
                size_t t = pair_index(c->N, i, j) * (size_t)c->L + (size_t)l;
                size_t u = (size_t)e * (size_t)c->L + (size_t)l;
                double *Xi = c->X[(size_t)i * c->L + l], *Xj = c->X[(size_t)j * c->L + l];
                for (int k = 0; k < rank; ++k) {
                    if (!live[u * (size_t)rank + k]) continue;   /* degenerate column: no update, vector kept */
                    const double *p = c->Ph[t] + (size_t)k * n;
                    const double *q = Qn[u] + (size_t)k * m;
#pragma omp parallel for schedule(static) if ((size_t)n * (size_t)m > 65536)
                    for (int r = 0; r < n; ++r) {
                        double a = w[e] * p[r];
                        for (int cidx = 0; cidx < m; ++cidx) {
                            double d = a * q[cidx];
                            Xi[(size_t)r * m + cidx] -= d;
                            Xj[(size_t)r * m + cidx] += d;
                        }
                    }
                    memcpy(c->Q[t] + (size_t)k * m, q, sizeof(double) * (size_t)m);
                }
                free(Qn[u]);
                Qn[u] = NULL;
            }
        }
        if (c->fp32_storage) round_state_to_fp32(c, edges, E);
    }
    free(Qn); free(live); free(edges); free(w);
    c->round += 1;
    return 0;
}

/* Consensus distance (1/N) sum_i ||X_i - mean_j X_j||_F^2 summed over layers. */
double pgo_consensus_distance(pgo_ctx *c)
{
    double total = 0.0;
    for (int l = 0; l < c->L; ++l) {
        size_t cnt = (size_t)c->rows[l] * (size_t)c->cols[l];
        for (size_t t = 0; t < cnt; ++t) {
            double mean = 0.0, s = 0.0;
            for (int i = 0; i < c->N; ++i) mean += c->X[(size_t)i * c->L + l][t];
            mean /= (double)c->N;
            for (int i = 0; i < c->N; ++i) {
                double d = c->X[(size_t)i * c->L + l][t] - mean;
                s += d * d;
            }
            total += s;
        }
    }
    return total / (double)c->N;
}

/* Worker average of one layer (Lemma 1 says it never changes). */
int pgo_average(pgo_ctx *c, int l, double *dst)
{
    if (!c || l < 0 || l >= c->L) return -1;
    size_t cnt = (size_t)c->rows[l] * (size_t)c->cols[l];
    for (size_t t = 0; t < cnt; ++t) {
        double s = 0.0;
        for (int i = 0; i < c->N; ++i) s += c->X[(size_t)i * c->L + l][t];
        dst[t] = s / (double)c->N;
    }
    return 0;
}

/* Floats one endpoint sends per iteration of Algorithm 2 for an n x m tensor at
 * rank `rank`: iterations alternate between an n-vector and an m-vector, so the
 * mean is rank*(n+m)/2; the per-tensor compression ratio of the paper's
 * parameter tables is n*m over that, divided by the number of iterations. */
double pgo_compression_ratio(int n, int m, int rank, int iterations)
{
    double sent = (double)rank * 0.5 * ((double)n + (double)m) * (double)iterations;
    return (double)n * (double)m / sent;
}

/* Threads the parallel loops use from now on (timing aid; results do not depend on it). */
void pgo_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int pgo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
