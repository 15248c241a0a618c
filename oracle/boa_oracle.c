/*
 * boa_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-threaded CPU statement of what the batched adaptive
 * filtered beam search computes.  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference arm may build, load or call it.  It
 * shares no code, header, table or helper with the CUDA library.
 *
 * What each function follows:
 *   orc_phi            filter distance: number of the query's closed range
 *                      predicates a point violates (Background, "Graph
 *                      construction", last paragraph; Eq. 2 gives g = [phi == 0]);
 *                      a column can also hold membership masks (the Conclusion's
 *                      equality / subset filters)
 *   orc_range_penalty  the numeric range distance the same paragraph mentions as the
 *                      alternative to counting (extension: the paper counts)
 *   orc_bruteforce     exact range-filtered k-NN (Definition 1, Definition 2, Eq. 1)
 *   orc_beam_*         filter-aware beam search at one beamwidth (Algorithm 2),
 *                      with exact L2 distances instead of PQ look-ups
 *   orc_uncertain      confidence test gamma(D_i) <= eps (Eq. 3)
 *   orc_prune, orc_build_graph   construction of the proximity graph (Background, "Graph
 *                      construction": Vamana insertion with alpha-dominance pruning, one
 *                      pruning run per attribute threshold)
 *   orc_cos_*          cosine distance (Definition 1 allows the Euclidean norm or cosine distance;
 *                      the paper itself uses the Euclidean norm throughout)
 *   orc_pq_*           product-quantised traversal (Algorithm 2's PQDist line; Section "BOA
 *                      Implementation on a GPU System": the per-query distance table, the
 *                      asymmetric PQ distance as a sum of table look-ups, and the final
 *                      ranking of the candidates by exact distance with invalid ones excluded)
 *   orc_boa_search_wl  multi-phase driver (Algorithm 1)
 *
 * Readings of points the paper leaves open (each is listed in the design notes):
 *   - the score dist + lambda*phi is taken in its lambda -> infinity limit by default:
 *     keys order by (phi, d2, id) lexicographically; id breaks every tie.  A finite
 *     lambda can be set: score = d2 + lambda*phi on squared distances, order (score, id)
 *   - "visited" means two things in Algorithm 2: a node already scored ("seen",
 *     the Bloom filter line, here an exact set) and a node already expanded (a
 *     flag on the worklist entry, the convergence line)
 *   - distances are squared L2 in fp32; two ways to accumulate them are offered:
 *     mode 0 sums in double and rounds once, mode 1 uses the 8-way interleaved
 *     fp32 order described at orc_dist2_lanes
 *   - a query whose beam holds at most k filter-valid entries is uncertain
 *   - restart mode runs every phase from the entry point with pool capacity L;
 *     resume mode keeps pool, flags and seen set, pool capacity Lmax, and only
 *     lengthens the expandable prefix (reading of "redundancy avoidance")
 *   - a phase stops after cap_mult*L + cap_add expansions at the latest
 *   - expansion width W (nodes expanded per iteration) is 1 as in the paper unless a
 *     caller asks for more; see orc_beam_run_w
 *   - with PQ traversal the keys of the search are PQ distances; when a phase has converged
 *     the filter-valid entries of the beam (the first L pool entries, the worklist of
 *     Algorithm 2) are ranked by exact distance, the k nearest are the result, and the
 *     confidence test reads those exact distances
 *
 * parity pins: tests/test_oracle_pins.py (brute force vs. an independent sort,
 * g == 1 vs. a library k-NN, the ring-graph hand trace, full-graph search ==
 * brute force, restart/resume relations, eps special cases, L_avg vs. the
 * paper's Table III).  Unpinned by the paper itself: the exact trajectories on
 * large inputs, the constants alpha, tau, lambda.
 * PQ pins: tests/test_oracle_pq_pins.py (hand-worked table and look-up sums, numpy, a
 * lossless codebook == the exact search, a full-width beam == brute force, properties of
 * the final ranking).  Unpinned by the paper: which candidates the final ranking covers
 * (taken: the filter-valid entries of the beam).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_SENTINEL 0xFFFFFFFFu
#define ORC_MAX_W 64            /* largest expansion width (nodes per iteration) */
#define ORC_F32 0
#define ORC_U8 1
#define ORC_ATTR_I32 0
#define ORC_ATTR_F32 1
#define ORC_ATTR_SET 2          /* cell = 32-bit membership mask of the point */

typedef struct {
    int64_t N;
    int D, m, R, vec_dtype;
    const void *vectors;      /* [N][D] float or uint8_t       */
    const int32_t *attrs;     /* [N][m] 4-byte cells           */
    const int32_t *attr_types; /* [m]                          */
    const uint32_t *graph;    /* [N][R], ORC_SENTINEL = no edge */
    int64_t entry;
    /* metric: 0 = squared Euclidean distance, 1 = cosine distance */
    int metric;
    float *unit;              /* [N][D] rows scaled to unit length (cosine metric, fp32 path) */
    /* product quantisation (optional): D = pq_M * dsub */
    int pq_M, pq_K;
    const float *pq_pivots;   /* [M][K][dsub] centroids of every subspace */
    const uint8_t *pq_codes;  /* [N][M] centroid index of every point in every subspace */
} orc_index;

/* ------------------------------------------------------------------ */
/* element access                                                      */
/* ------------------------------------------------------------------ */
static float orc_elem(const orc_index *ix, int64_t p, int i)
{
    if (ix->vec_dtype == ORC_U8)
        return (float)((const uint8_t *)ix->vectors)[p * ix->D + i];
    return ((const float *)ix->vectors)[p * ix->D + i];
}

/* squared L2 distance, summed in double in index order (mode 0 rounds this to float) */
double orc_dist2_f64(const orc_index *ix, const float *q, int64_t p)
{
    double s = 0.0;
    for (int i = 0; i < ix->D; ++i) {
        double d = (double)orc_elem(ix, p, i) - (double)q[i];
        s += d * d;
    }
    return s;
}

/*
 * Squared L2 distance in fp32, in a fixed order so that a second fp32
 * implementation can reproduce it bit for bit.  The row is cut into chunks of
 * 16 bytes (4 floats or 16 bytes of uint8).  Chunk c belongs to partial sum
 * c mod 8.  Each partial sum runs over its chunks in ascending order and over
 * the elements of a chunk in ascending order with
 *     acc = fmaf(x - q, x - q, acc)        (x - q rounded to fp32 first).
 * The eight partial sums are then added pairwise:
 *     ((p0+p4) + (p2+p6)) + ((p1+p5) + (p3+p7)).
 */
float orc_dist2_lanes(const orc_index *ix, const float *q, int64_t p)
{
    const int per = (ix->vec_dtype == ORC_U8) ? 16 : 4;
    const int nchunks = (ix->D + per - 1) / per;
    float part[8];
    for (int g = 0; g < 8; ++g) {
        float acc = 0.0f;
        for (int c = g; c < nchunks; c += 8) {
            for (int j = 0; j < per; ++j) {
                int i = c * per + j;
                if (i >= ix->D) break;
                float diff = orc_elem(ix, p, i) - q[i];
                acc = fmaf(diff, diff, acc);
            }
        }
        part[g] = acc;
    }
    float a04 = part[0] + part[4], a15 = part[1] + part[5];
    float a26 = part[2] + part[6], a37 = part[3] + part[7];
    float e = a04 + a26, o = a15 + a37;
    return e + o;
}

static float orc_dist2(const orc_index *ix, const float *q, int64_t p, int dist_mode)
{
    if (dist_mode == 1) return orc_dist2_lanes(ix, q, p);
    return (float)orc_dist2_f64(ix, q, p);
}

/* ------------------------------------------------------------------ */
/* cosine distance                                                     */
/* ------------------------------------------------------------------ */
/*
 * Cosine distance, taken as half the squared Euclidean distance of the two vectors scaled to
 * unit length: 0.5 * |x/|x| - q/|q||^2 = 1 - cos(x, q) for non-zero vectors (a zero vector
 * scales to zero).  The norm is the square root of the sum of squares in double, elements in
 * ascending order.
 *   mode 0: everything in double, rounded once to float.
 *   mode 1: the unit vectors are first rounded to float (x_i * (1/|x|) in double, then
 *           rounded), their squared distance is summed in fp32 in the fixed order of
 *           orc_dist2_lanes, and halved (exact).
 */
static double orc_inv_norm(const float *v, int D)
{
    double s = 0.0;
    for (int i = 0; i < D; ++i) s += (double)v[i] * (double)v[i];
    return s > 0.0 ? 1.0 / sqrt(s) : 0.0;
}

/* unit-length copy of v, rounded to float */
void orc_unit_f32(const float *v, int D, float *out)
{
    double inv = orc_inv_norm(v, D);
    for (int i = 0; i < D; ++i) out[i] = (float)((double)v[i] * inv);
}

/* fixed-order fp32 squared distance of two float vectors (the order of orc_dist2_lanes) */
static float orc_lanes_f32(const float *x, const float *q, int D)
{
    const int nchunks = (D + 3) / 4;
    float part[8];
    for (int g = 0; g < 8; ++g) {
        float acc = 0.0f;
        for (int c = g; c < nchunks; c += 8)
            for (int j = 0; j < 4 && c * 4 + j < D; ++j) {
                float diff = x[c * 4 + j] - q[c * 4 + j];
                acc = fmaf(diff, diff, acc);
            }
        part[g] = acc;
    }
    float a04 = part[0] + part[4], a15 = part[1] + part[5];
    float a26 = part[2] + part[6], a37 = part[3] + part[7];
    float e = a04 + a26, o = a15 + a37;
    return e + o;
}

/* q is the query as given (not normalised) */
float orc_cos_dist(const orc_index *ix, const float *q, int64_t p, int dist_mode)
{
    const float *x = (const float *)ix->vectors + p * ix->D;
    if (dist_mode == 1) {
        float *qh = (float *)malloc((size_t)ix->D * sizeof(float));
        orc_unit_f32(q, ix->D, qh);
        float d = 0.5f * orc_lanes_f32(ix->unit + p * ix->D, qh, ix->D);
        free(qh);
        return d;
    }
    double ix_ = orc_inv_norm(x, ix->D), iq = orc_inv_norm(q, ix->D), s = 0.0;
    for (int i = 0; i < ix->D; ++i) {
        double d = (double)x[i] * ix_ - (double)q[i] * iq;
        s += d * d;
    }
    return (float)(0.5 * s);
}

/* Choose the metric (0 = squared Euclidean, 1 = cosine; float vectors only).  Call once, after
   orc_create: the entry point stays the medoid of the vectors as given. */
void orc_set_metric(orc_index *ix, int metric)
{
    ix->metric = metric;
    if (metric == 1 && !ix->unit) {
        ix->unit = (float *)malloc((size_t)ix->N * ix->D * sizeof(float));
        for (int64_t p = 0; p < ix->N; ++p)
            orc_unit_f32((const float *)ix->vectors + p * ix->D, ix->D, ix->unit + p * ix->D);
    }
}

/* the distance of the index's metric, exact (not product-quantised) */
static float orc_metric_dist(const orc_index *ix, const float *q, int64_t p, int dist_mode)
{
    if (ix->metric == 1) return orc_cos_dist(ix, q, p, dist_mode);
    return orc_dist2(ix, q, p, dist_mode);
}

/* number of violated closed range predicates; bounds use the column's own type */
int orc_phi(const orc_index *ix, const int32_t *lo, const int32_t *hi, int64_t p)
{
    int v = 0;
    for (int j = 0; j < ix->m; ++j) {
        int32_t cell = ix->attrs[p * ix->m + j];
        if (ix->attr_types[j] == ORC_ATTR_F32) {
            float a, l, h;
            memcpy(&a, &cell, 4);
            memcpy(&l, &lo[j], 4);
            memcpy(&h, &hi[j], 4);
            if (!(a >= l && a <= h)) v++;      /* NaN violates */
        } else if (ix->attr_types[j] == ORC_ATTR_SET) {
            /* membership predicate: lo = the wanted tags; hi == 0: the point must carry at
               least one of them, hi != 0: all of them */
            uint32_t have = (uint32_t)cell & (uint32_t)lo[j];
            if (hi[j] == 0 ? have == 0u : have != (uint32_t)lo[j]) v++;
        } else {
            if (cell < lo[j] || cell > hi[j]) v++;
        }
    }
    return v;
}

/*
 * Distance-to-range penalty, the numeric alternative to the violation count: for every
 * violated predicate the distance from the cell to the nearer end of its range, times the
 * caller's scale for that attribute, added over the attributes in ascending order in fp32.
 * Integer cells: the distance is taken in double (exact) and rounded once to float; float
 * cells: one fp32 subtraction, a NaN cell counts as infinitely far; a violated membership
 * predicate costs its scale.  Zero exactly when the point is filter-valid.
 */
float orc_range_penalty(const orc_index *ix, const int32_t *lo, const int32_t *hi, int64_t p,
                        const float *scales)
{
    float pen = 0.0f;
    for (int j = 0; j < ix->m; ++j) {
        int32_t cell = ix->attrs[p * ix->m + j];
        float e = 0.0f;
        if (ix->attr_types[j] == ORC_ATTR_F32) {
            float a, l, h;
            memcpy(&a, &cell, 4);
            memcpy(&l, &lo[j], 4);
            memcpy(&h, &hi[j], 4);
            if (a < l) e = l - a;
            else if (a > h) e = a - h;
            else if (!(a >= l && a <= h)) e = INFINITY;
        } else if (ix->attr_types[j] == ORC_ATTR_SET) {
            uint32_t have = (uint32_t)cell & (uint32_t)lo[j];
            if (hi[j] == 0 ? have == 0u : have != (uint32_t)lo[j]) e = 1.0f;
        } else {
            if (cell < lo[j]) e = (float)((double)lo[j] - (double)cell);
            else if (cell > hi[j]) e = (float)((double)cell - (double)hi[j]);
        }
        pen = pen + e * scales[j];
    }
    return pen;
}

/* ------------------------------------------------------------------ */
/* product quantisation                                                */
/* ------------------------------------------------------------------ */
/* The vector space is cut into M subspaces of dsub = D/M consecutive dimensions; every
   subspace has K centroids ("pivots"); a point is stored as the M indices of its nearest
   centroids.  The codebook is an input (trained by whoever built the index). */
void orc_pq_attach(orc_index *ix, const float *pivots, const uint8_t *codes, int M, int K)
{
    ix->pq_M = M; ix->pq_K = K; ix->pq_pivots = pivots; ix->pq_codes = codes;
}

/* The distance table of one query: table[m][c] = squared L2 distance between the m-th
   subvector of q and centroid c of subspace m.  dist_mode 1: fp32, one
   acc = fmaf(q - piv, q - piv, acc) per dimension in ascending order; dist_mode 0: the same
   sum in double, rounded once to float. */
void orc_pq_table(const orc_index *ix, const float *q, int dist_mode, float *table)
{
    const int M = ix->pq_M, K = ix->pq_K, dsub = ix->D / M;
    for (int m = 0; m < M; ++m)
        for (int c = 0; c < K; ++c) {
            const float *piv = ix->pq_pivots + ((size_t)m * K + c) * dsub;
            if (dist_mode == 1) {
                float acc = 0.0f;
                for (int i = 0; i < dsub; ++i) {
                    float diff = q[m * dsub + i] - piv[i];
                    acc = fmaf(diff, diff, acc);
                }
                table[m * K + c] = acc;
            } else {
                double acc = 0.0;
                for (int i = 0; i < dsub; ++i) {
                    double diff = (double)q[m * dsub + i] - (double)piv[i];
                    acc += diff * diff;
                }
                table[m * K + c] = (float)acc;
            }
        }
}

/* Asymmetric PQ distance of point p: the sum over the subspaces of the table entry its
   code selects, added in ascending subspace order (fp32 in mode 1, double rounded once in
   mode 0). */
float orc_pq_dist(const orc_index *ix, const float *table, int dist_mode, int64_t p)
{
    const int M = ix->pq_M, K = ix->pq_K;
    const uint8_t *code = ix->pq_codes + (size_t)p * M;
    if (dist_mode == 1) {
        float acc = 0.0f;
        for (int m = 0; m < M; ++m) acc = acc + table[m * K + code[m]];
        return acc;
    }
    double acc = 0.0;
    for (int m = 0; m < M; ++m) acc += (double)table[m * K + code[m]];
    return (float)acc;
}

/* ------------------------------------------------------------------ */
/* index                                                               */
/* ------------------------------------------------------------------ */
/* point nearest (squared L2 in double, lower id wins ties) to the coordinate mean */
int64_t orc_medoid(const orc_index *ix)
{
    double *mean = (double *)calloc((size_t)ix->D, sizeof(double));
    for (int64_t p = 0; p < ix->N; ++p)
        for (int i = 0; i < ix->D; ++i) mean[i] += (double)orc_elem(ix, p, i);
    for (int i = 0; i < ix->D; ++i) mean[i] /= (double)ix->N;
    int64_t best = 0;
    double bestd = INFINITY;
    for (int64_t p = 0; p < ix->N; ++p) {
        double s = 0.0;
        for (int i = 0; i < ix->D; ++i) {
            double d = (double)orc_elem(ix, p, i) - mean[i];
            s += d * d;
        }
        if (s < bestd) { bestd = s; best = p; }
    }
    free(mean);
    return best;
}

orc_index *orc_create(const void *vectors, int vec_dtype, int64_t N, int D,
                      const int32_t *attrs, const int32_t *attr_types, int m,
                      const uint32_t *graph, int R, int64_t entry)
{
    orc_index *ix = (orc_index *)calloc(1, sizeof(orc_index));
    ix->N = N; ix->D = D; ix->m = m; ix->R = R; ix->vec_dtype = vec_dtype;
    ix->vectors = vectors; ix->attrs = attrs; ix->attr_types = attr_types; ix->graph = graph;
    ix->entry = entry;
    if (entry < 0) ix->entry = orc_medoid(ix);
    return ix;
}
void orc_destroy(orc_index *ix) { free(ix->unit); free(ix); }
int64_t orc_entry(const orc_index *ix) { return ix->entry; }

/* ------------------------------------------------------------------ */
/* exact filtered top-k (Definitions 1 and 2)                          */
/* ------------------------------------------------------------------ */
/* Returns |D_f|.  out_ids/out_d2 receive the min(k,|D_f|) valid points of
   smallest distance, ascending by (d2, id); the rest is padded. */
int64_t orc_bruteforce(const orc_index *ix, const float *q, const int32_t *lo, const int32_t *hi,
                       int k, uint32_t *out_ids, double *out_d2)
{
    int have = 0;
    int64_t nvalid = 0;
    for (int i = 0; i < k; ++i) { out_ids[i] = ORC_SENTINEL; out_d2[i] = INFINITY; }
    for (int64_t p = 0; p < ix->N; ++p) {
        if (orc_phi(ix, lo, hi, p) != 0) continue;
        nvalid++;
        double d = ix->metric == 1 ? (double)orc_cos_dist(ix, q, p, 0) : orc_dist2_f64(ix, q, p);
        /* ids ascend, so a strict < keeps the lower id ahead on equal distance */
        int pos = have;
        while (pos > 0 && d < out_d2[pos - 1]) pos--;
        if (pos >= k) continue;
        int last = (have < k) ? have : k - 1;
        for (int t = last; t > pos; --t) { out_d2[t] = out_d2[t - 1]; out_ids[t] = out_ids[t - 1]; }
        out_d2[pos] = d; out_ids[pos] = (uint32_t)p;
        if (have < k) have++;
    }
    return nvalid;
}

/* ------------------------------------------------------------------ */
/* filter-aware beam search (Algorithm 2)                              */
/* ------------------------------------------------------------------ */
typedef struct {
    int phi;
    float d2;
    float score;         /* d2 + lambda*phi (finite lambda only) */
    float pen;           /* distance-to-range penalty (when it replaces phi in the score) */
    uint32_t id;
    int expanded;
} orc_entry_t;

typedef struct {
    const orc_index *ix;
    int C;               /* pool capacity */
    int size;
    orc_entry_t *pool;   /* ascending by (phi, d2, id), or by (score, id) with a finite lambda */
    float lambda;        /* weight of the filter penalty; INFINITY = lexicographic order */
    uint8_t *seen;       /* [N] */
    uint32_t *touched;   /* ids set in seen, for a cheap reset */
    int64_t ntouched, touched_cap;
    int64_t n_expand, n_scored;
    int hit_cap;
    float *pq_table;     /* [M][K] of the current query when the search runs on PQ distances, else NULL */
    const float *pen_scales; /* [m] when the score uses the distance-to-range penalty, else NULL */
} orc_state;

/* The order the search works by.  The paper's score is dist + lambda*phi with one lambda
   for all attributes.  lambda = INFINITY is its limit: any violated predicate outweighs
   any distance, so keys compare by (phi, d2).  A finite lambda gives score = d2 +
   lambda*phi, one fused multiply-add in fp32.  The node id breaks ties either way. */
static int orc_less(const orc_state *st, const orc_entry_t *a, const orc_entry_t *b)
{
    if (isinf(st->lambda)) {
        if (a->phi != b->phi) return a->phi < b->phi;
        if (a->d2 != b->d2) return a->d2 < b->d2;
    } else {
        if (a->score != b->score) return a->score < b->score;
    }
    return a->id < b->id;
}

orc_state *orc_state_new(const orc_index *ix, int C)
{
    orc_state *st = (orc_state *)calloc(1, sizeof(orc_state));
    st->ix = ix; st->C = C; st->lambda = INFINITY;
    st->pool = (orc_entry_t *)calloc((size_t)C + (size_t)ORC_MAX_W * ix->R + 1, sizeof(orc_entry_t));
    st->seen = (uint8_t *)calloc((size_t)ix->N, 1);
    st->touched_cap = 1024;
    st->touched = (uint32_t *)malloc((size_t)st->touched_cap * sizeof(uint32_t));
    return st;
}
/* set before orc_beam_init; lambda >= 0, INFINITY for the lexicographic order */
void orc_state_set_lambda(orc_state *st, float lambda) { st->lambda = lambda; }
/* score = d2 + lambda * (distance-to-range penalty with these per-attribute scales) instead of
   d2 + lambda * (violation count); needs a finite lambda.  NULL switches back. */
void orc_state_set_penalty(orc_state *st, const float *scales) { st->pen_scales = scales; }
void orc_state_free(orc_state *st)
{
    free(st->pool); free(st->seen); free(st->touched); free(st->pq_table); free(st);
}

/* Switch the state to PQ traversal for query q (on != 0: the distance table is built here),
   or back to exact distances.  Call before orc_beam_init, and again before a resumed run
   of another query. */
void orc_state_use_pq(orc_state *st, int on, const float *q, int dist_mode)
{
    if (!on) { free(st->pq_table); st->pq_table = NULL; return; }
    if (!st->pq_table)
        st->pq_table = (float *)malloc((size_t)st->ix->pq_M * st->ix->pq_K * sizeof(float));
    if (st->ix->metric == 1) {
        /* cosine metric: the codebook lives in the space of unit-length vectors */
        float *qh = (float *)malloc((size_t)st->ix->D * sizeof(float));
        orc_unit_f32(q, st->ix->D, qh);
        orc_pq_table(st->ix, qh, dist_mode, st->pq_table);
        free(qh);
        return;
    }
    orc_pq_table(st->ix, q, dist_mode, st->pq_table);
}

/* the distance the traversal orders by */
static float orc_search_dist(const orc_state *st, const float *q, int64_t p, int dist_mode)
{
    if (st->pq_table) return orc_pq_dist(st->ix, st->pq_table, dist_mode, p);
    return orc_metric_dist(st->ix, q, p, dist_mode);
}

static void orc_mark_seen(orc_state *st, uint32_t id)
{
    st->seen[id] = 1;
    if (st->ntouched == st->touched_cap) {
        st->touched_cap *= 2;
        st->touched = (uint32_t *)realloc(st->touched, (size_t)st->touched_cap * sizeof(uint32_t));
    }
    st->touched[st->ntouched++] = id;
}

static void orc_pool_insert(orc_state *st, orc_entry_t e)
{
    int pos = st->size;
    e.score = isinf(st->lambda) ? e.d2
              : fmaf(st->lambda, st->pen_scales ? e.pen : (float)e.phi, e.d2);
    while (pos > 0 && orc_less(st, &e, &st->pool[pos - 1])) { st->pool[pos] = st->pool[pos - 1]; pos--; }
    st->pool[pos] = e;
    st->size++;
}

/* L_i <- {s}: empty seen set, pool holding only the entry point */
void orc_beam_init(orc_state *st, int C, const float *q, const int32_t *lo, const int32_t *hi, int dist_mode)
{
    const orc_index *ix = st->ix;
    for (int64_t t = 0; t < st->ntouched; ++t) st->seen[st->touched[t]] = 0;
    st->ntouched = 0; st->size = 0; st->C = C;
    st->n_expand = 0; st->n_scored = 0; st->hit_cap = 0;
    orc_entry_t e;
    e.id = (uint32_t)ix->entry; e.expanded = 0;
    e.phi = orc_phi(ix, lo, hi, ix->entry);
    e.pen = st->pen_scales ? orc_range_penalty(ix, lo, hi, ix->entry, st->pen_scales) : 0.0f;
    e.d2 = orc_search_dist(st, q, ix->entry, dist_mode);
    orc_mark_seen(st, e.id);
    orc_pool_insert(st, e);
}

/* run the loop of Algorithm 2 at beamwidth L until every one of the first L
   pool entries is expanded; gives up (hit_cap) when an unexpanded entry is left
   after max_expand expansions of this call.

   W is the expansion width.  The paper expands one node per iteration (W = 1).
   With W > 1 (an extension: the step widening of multi-node expansion in GPU
   graph search) an iteration takes the first W unexpanded entries of the beam,
   fewer when the beam or the expansion cap leaves fewer, marks them expanded,
   and then scores their rows in that order before the pool is looked at again. */
void orc_beam_run_w(orc_state *st, int L, const float *q, const int32_t *lo, const int32_t *hi,
                    int dist_mode, int64_t max_expand, int W)
{
    const orc_index *ix = st->ix;
    int64_t done = 0;
    st->hit_cap = 0;
    if (W < 1) W = 1;
    if (W > ORC_MAX_W) W = ORC_MAX_W;
    for (;;) {
        int lim = st->size < L ? st->size : L;
        uint32_t picked[ORC_MAX_W];
        int np = 0, any = 0;
        for (int t = 0; t < lim; ++t)
            if (!st->pool[t].expanded) { any = 1; break; }
        if (!any) break;                                /* converged */
        if (done >= max_expand) { st->hit_cap = 1; break; }
        for (int t = 0; t < lim && np < W && done + np < max_expand; ++t)
            if (!st->pool[t].expanded) {
                st->pool[t].expanded = 1;
                picked[np++] = st->pool[t].id;
            }
        st->n_expand += np; done += np;
        for (int a = 0; a < np; ++a) {
            uint32_t uid = picked[a];
            for (int j = 0; j < ix->R; ++j) {
                uint32_t n = ix->graph[(int64_t)uid * ix->R + j];
                if (n == ORC_SENTINEL || st->seen[n]) continue;
                orc_mark_seen(st, n);
                st->n_scored++;
                orc_entry_t e;
                e.id = n; e.expanded = 0;
                e.phi = orc_phi(ix, lo, hi, n);
                e.pen = st->pen_scales ? orc_range_penalty(ix, lo, hi, n, st->pen_scales) : 0.0f;
                e.d2 = orc_search_dist(st, q, n, dist_mode);
                orc_pool_insert(st, e);
            }
        }
        if (st->size > st->C) st->size = st->C;          /* keep the C best */
    }
}

/* K_i <- the k nearest filter-valid pool entries; returns how many there are */
int orc_beam_result(const orc_state *st, int k, uint32_t *out_ids, float *out_d2)
{
    int have = 0;
    for (int t = 0; t < st->size && have < k; ++t)
        if (st->pool[t].phi == 0) { out_ids[have] = st->pool[t].id; out_d2[have] = st->pool[t].d2; have++; }
    for (int t = have; t < k; ++t) { out_ids[t] = ORC_SENTINEL; out_d2[t] = INFINITY; }
    return have;
}

int orc_state_size(const orc_state *st) { return st->size; }
int64_t orc_state_expanded(const orc_state *st) { return st->n_expand; }
int64_t orc_state_scored(const orc_state *st) { return st->n_scored; }
int orc_state_hit_cap(const orc_state *st) { return st->hit_cap; }
void orc_state_pool(const orc_state *st, uint32_t *ids, float *d2, int32_t *phi, int32_t *expanded)
{
    for (int t = 0; t < st->size; ++t) {
        ids[t] = st->pool[t].id; d2[t] = st->pool[t].d2;
        phi[t] = st->pool[t].phi; expanded[t] = st->pool[t].expanded;
    }
}

/*
 * Confidence test (Eq. 3).  V = filter-valid entries among the first L pool
 * entries.  gamma = (d_max - d_k)/d_max on Euclidean norms; gamma <= eps is
 * evaluated without square roots as d2_k >= (1-eps)^2 * d2_max, in fp32, the
 * constant rounded once to float.  Returns 1 when the query must escalate.
 */
/* metric 0: the distances are squared norms, gamma is defined on the norms (constant (1-eps)^2);
   metric 1: the distances are cosine distances themselves (constant 1-eps) */
static int orc_gap_uncertain_m(int nv, int k, float d2k, float d2max, double eps, int metric)
{
    if (nv <= k) return 1;
    if (eps < 0.0) return 1;
    if (eps >= 1.0) return 0;
    float c = metric == 1 ? (float)(1.0 - eps) : (float)((1.0 - eps) * (1.0 - eps));
    float rhs = c * d2max;
    return !(d2k >= rhs);
}
static int orc_gap_uncertain(int nv, int k, float d2k, float d2max, double eps)
{
    if (nv <= k) return 1;
    if (eps < 0.0) return 1;
    if (eps >= 1.0) return 0;
    float c = (float)((1.0 - eps) * (1.0 - eps));
    float rhs = c * d2max;
    return !(d2k >= rhs);
}

int orc_uncertain(const orc_state *st, int L, int k, double eps)
{
    int lim = st->size < L ? st->size : L;
    int nv = 0;
    float d2k = 0.0f, d2max = 0.0f;
    for (int t = 0; t < lim; ++t) {
        if (st->pool[t].phi != 0) continue;
        nv++;
        if (nv == k) d2k = st->pool[t].d2;
        d2max = st->pool[t].d2;                           /* entries ascend */
    }
    return orc_gap_uncertain_m(nv, k, d2k, d2max, eps, st->ix->metric);
}

/*
 * End of a PQ search ("Re-rank exact": on convergence the candidates are ranked by exact
 * distance, invalid ones excluded).  V = the filter-valid entries among the first L pool
 * entries.  Every member of V gets its exact squared distance; V is ordered by (d2, id);
 * the first k are the result (padded as usual).  Returns |V|; *d2k and *d2max receive the
 * k-th and the largest exact distance of V (what the confidence test reads), 0 when
 * |V| < k or V is empty.
 */
int orc_beam_rerank(const orc_state *st, int L, int k, const float *q, int dist_mode,
                    uint32_t *out_ids, float *out_d2, float *d2k, float *d2max)
{
    int lim = st->size < L ? st->size : L;
    uint32_t *vid = (uint32_t *)malloc((size_t)(lim + 1) * sizeof(uint32_t));
    float *vd = (float *)calloc((size_t)lim + 1, sizeof(float));
    int nv = 0;
    for (int t = 0; t < lim; ++t) {
        if (st->pool[t].phi != 0) continue;
        uint32_t id = st->pool[t].id;
        float d = orc_metric_dist(st->ix, q, id, dist_mode);
        int pos = nv;                                      /* insertion by (d2, id) */
        while (pos > 0 && (d < vd[pos - 1] || (d == vd[pos - 1] && id < vid[pos - 1]))) {
            vd[pos] = vd[pos - 1]; vid[pos] = vid[pos - 1]; pos--;
        }
        vd[pos] = d; vid[pos] = id; nv++;
    }
    for (int t = 0; t < k; ++t) {
        if (t < nv) { out_ids[t] = vid[t]; out_d2[t] = vd[t]; }
        else { out_ids[t] = ORC_SENTINEL; out_d2[t] = INFINITY; }
    }
    *d2k = nv >= k ? vd[k - 1] : 0.0f;
    *d2max = nv > 0 ? vd[nv - 1] : 0.0f;
    free(vid); free(vd);
    return nv;
}

/* Eq. 3 on the exact distances a PQ search ends with */
int orc_uncertain_reranked(int nv, int k, float d2k, float d2max, double eps)
{
    return orc_gap_uncertain(nv, k, d2k, d2max, eps);
}

/* ------------------------------------------------------------------ */
/* multi-phase driver (Algorithm 1)                                    */
/* ------------------------------------------------------------------ */
/* what resume mode carries from one phase of a query to the next: the pool
   with its expanded flags, and the ids of the seen set */
typedef struct {
    int size;
    orc_entry_t *pool;
    int64_t ntouched;
    uint32_t *touched;
} orc_saved;

static orc_saved *orc_save(const orc_state *st)
{
    orc_saved *sv = (orc_saved *)calloc(1, sizeof(orc_saved));
    sv->size = st->size;
    sv->pool = (orc_entry_t *)malloc((size_t)(st->size + 1) * sizeof(orc_entry_t));
    memcpy(sv->pool, st->pool, (size_t)st->size * sizeof(orc_entry_t));
    sv->ntouched = st->ntouched;
    sv->touched = (uint32_t *)malloc((size_t)(st->ntouched + 1) * sizeof(uint32_t));
    memcpy(sv->touched, st->touched, (size_t)st->ntouched * sizeof(uint32_t));
    return sv;
}
static void orc_saved_free(orc_saved *sv)
{
    if (!sv) return;
    free(sv->pool); free(sv->touched); free(sv);
}
/* put a saved search back into the working state */
static void orc_restore(orc_state *st, const orc_saved *sv, int C)
{
    for (int64_t t = 0; t < st->ntouched; ++t) st->seen[st->touched[t]] = 0;
    st->ntouched = 0; st->C = C;
    st->n_expand = 0; st->n_scored = 0; st->hit_cap = 0;
    for (int64_t t = 0; t < sv->ntouched; ++t) orc_mark_seen(st, sv->touched[t]);
    st->size = sv->size;
    memcpy(st->pool, sv->pool, (size_t)sv->size * sizeof(orc_entry_t));
}

/*
 * widths[0..n_widths): beamwidth of each phase.  mode 0 = restart, 1 = resume.
 * Outputs are indexed by the original query index whatever phase wrote them.
 * phase_active[p] receives |A| at the start of phase p.  n_expand / n_scored
 * add up over the phases a query ran; flags bit 0 = some phase hit its
 * expansion cap.
 */
void orc_boa_search_wl(const orc_index *ix, const float *queries, int64_t Q,
                      const int32_t *lo, const int32_t *hi, int k,
                      const int32_t *widths, int n_widths, double eps, double tau,
                      int mode, int dist_mode, int cap_mult, int cap_add, int W, float lambda,
                      int use_pq, const float *pen_scales,
                      uint32_t *out_ids, float *out_d2,
                      int32_t *final_L, int32_t *n_expand, int32_t *n_scored, int32_t *flags,
                      int64_t *phase_active)
{
    int Cmax = 0;
    for (int p = 0; p < n_widths; ++p) if (widths[p] > Cmax) Cmax = widths[p];
    orc_state *st = orc_state_new(ix, Cmax);
    orc_state_set_lambda(st, lambda);
    orc_state_set_penalty(st, pen_scales);
    for (int p = 0; p < n_widths; ++p) phase_active[p] = 0;

    uint8_t *active = (uint8_t *)malloc((size_t)Q + 1);             /* the set A */
    orc_saved **saved = (orc_saved **)calloc((size_t)Q + 1, sizeof(orc_saved *));
    for (int64_t i = 0; i < Q; ++i) {
        active[i] = 1; final_L[i] = 0; n_expand[i] = 0; n_scored[i] = 0; flags[i] = 0;
        for (int t = 0; t < k; ++t) { out_ids[i * k + t] = ORC_SENTINEL; out_d2[i * k + t] = INFINITY; }
    }
    int64_t n_active = Q;
    for (int p = 0; p < n_widths; ++p) {                            /* one phase per turn */
        if (!((double)n_active > tau * (double)Q)) break;           /* while |A| > tau*rho */
        phase_active[p] = n_active;
        const int L = widths[p];
        const int64_t cap = (int64_t)cap_mult * L + cap_add;
        for (int64_t i = 0; i < Q; ++i) {
            if (!active[i]) continue;
            const float *q = queries + i * ix->D;
            const int32_t *l = lo + i * ix->m, *h = hi + i * ix->m;
            if (use_pq) orc_state_use_pq(st, 1, q, dist_mode);      /* this query's distance table */
            if (mode == 1 && saved[i]) {
                orc_restore(st, saved[i], Cmax);
                orc_saved_free(saved[i]); saved[i] = NULL;
            } else {
                orc_beam_init(st, mode == 1 ? Cmax : L, q, l, h, dist_mode);
            }
            orc_beam_run_w(st, L, q, l, h, dist_mode, cap, W);
            int unc;
            if (use_pq) {
                float d2k, d2max;
                int nv = orc_beam_rerank(st, L, k, q, dist_mode, out_ids + i * k, out_d2 + i * k, &d2k, &d2max);
                unc = orc_gap_uncertain_m(nv, k, d2k, d2max, eps, ix->metric);
            } else {
                orc_beam_result(st, k, out_ids + i * k, out_d2 + i * k);    /* scatter */
                unc = orc_uncertain(st, L, k, eps);
            }
            final_L[i] = L;
            n_expand[i] += (int32_t)st->n_expand;
            n_scored[i] += (int32_t)st->n_scored;
            if (st->hit_cap) flags[i] |= 1;
            if (!unc) {                                             /* F: confident */
                active[i] = 0; n_active--;
            } else if (mode == 1 && p + 1 < n_widths) {
                saved[i] = orc_save(st);
            }
        }
    }
    for (int64_t i = 0; i < Q; ++i) orc_saved_free(saved[i]);
    free(saved);
    free(active);
    orc_state_free(st);
}

/* ------------------------------------------------------------------ */
/* graph construction (Background, "Graph construction")               */
/* ------------------------------------------------------------------ */
/*
 * A Vamana-style build with the threshold pruning the paper adopts: points are inserted in
 * batches; a beam search over the graph built so far collects candidates for each new point;
 * a pruning step keeps at most R out-neighbours by the alpha-dominance rule, run once per
 * attribute threshold with a degree budget of R/|T| each; reverse edges are added, pruning
 * again where a row overflows.  The paper gives the outline only; what is fixed here:
 *   - batches are [start, start + size) in index order, size = min(B, points inserted so
 *     far) (1, 1, 2, 4, ...); every point of a batch searches the graph as it stood before
 *     the batch; `passes` > 1 repeats the sweep with batches of B over the finished graph
 *   - a threshold is a vector t[0..m) over the attributes (thresholds[T][m]); t[j] = +infinity
 *     leaves attribute j free
 *   - candidates of p: for every threshold t one filter-aware beam search (Algorithm 2) at
 *     width Lb from the entry point whose predicate is "attribute position j within t[j] of
 *     p's, for every j" (bounds pos - t[j] and pos + t[j], one fp32 operation each; all
 *     +infinity is the unfiltered search): its filter-valid results, at most Lb; plus p's
 *     current out-neighbours
 *   - distances are squared L2 in the fixed-order fp32 of orc_dist2_lanes; candidates are
 *     ordered by (d2, id); c2 is dominated by a selected c when alpha^2 * d2(c, c2) <=
 *     d2(p, c2) (alpha^2 rounded once to float, one fp32 multiply)
 *   - attribute distance of two points in attribute j = the absolute difference of their
 *     positions (pos[N][m], e.g. rank / N per attribute); threshold pass i takes only
 *     candidates whose capped distance max(dist_j - thresholds[i][j], 0) is zero in every
 *     attribute, forgets the dominance marks of the pass before, and may select
 *     R*(i+1)/T - R*i/T more neighbours
 *   - after a batch every selected edge p -> n asks for n -> p: the requesters of n, in
 *     ascending id order, at most cap_in of them, those not yet in n's row; if they fit
 *     they are appended in that order, else n's row is pruned over row + requesters
 */
typedef struct {
    uint32_t id;
    float d2;
} orc_cand_t;

static int orc_cand_cmp(const void *a, const void *b)
{
    const orc_cand_t *x = (const orc_cand_t *)a, *y = (const orc_cand_t *)b;
    if (x->d2 != y->d2) return x->d2 < y->d2 ? -1 : 1;
    return x->id < y->id ? -1 : (x->id > y->id ? 1 : 0);
}

/* squared distance between two points of the index, fixed-order fp32 */
static float orc_point_dist2(const orc_index *ix, int64_t a, int64_t b)
{
    const int per = (ix->vec_dtype == ORC_U8) ? 16 : 4;
    const int nchunks = (ix->D + per - 1) / per;
    float part[8];
    for (int g = 0; g < 8; ++g) {
        float acc = 0.0f;
        for (int c = g; c < nchunks; c += 8)
            for (int j = 0; j < per && c * per + j < ix->D; ++j) {
                float diff = orc_elem(ix, a, c * per + j) - orc_elem(ix, b, c * per + j);
                acc = fmaf(diff, diff, acc);
            }
        part[g] = acc;
    }
    float a04 = part[0] + part[4], a15 = part[1] + part[5];
    float a26 = part[2] + part[6], a37 = part[3] + part[7];
    float e = a04 + a26, o = a15 + a37;
    return e + o;
}

/* 1 when b is within threshold vector t of a in every attribute */
static int orc_attr_within(const float *pos, int m, int64_t a, int64_t b, const float *t)
{
    for (int j = 0; j < m; ++j) {
        float x = fabsf(pos[a * m + j] - pos[b * m + j]);
        if (x > t[j]) return 0;
    }
    return 1;
}

/* The pruning step.  ids[0..n): candidate ids (any order, repeats and p itself allowed).
   Writes the selected neighbours, in selection order, to row[0..R), padded with the
   sentinel.  Returns how many were selected. */
int orc_prune(const orc_index *ix, const float *pos, int m_pos, int64_t p, const uint32_t *ids, int n,
              int R, float alpha, const float *thresholds, int T, uint32_t *row)
{
    orc_cand_t *c = (orc_cand_t *)malloc((size_t)(n + 1) * sizeof(orc_cand_t));
    int nc = 0;
    for (int i = 0; i < n; ++i) {
        if (ids[i] == ORC_SENTINEL || (int64_t)ids[i] == p) continue;
        c[nc].id = ids[i];
        c[nc].d2 = orc_point_dist2(ix, p, ids[i]);
        nc++;
    }
    qsort(c, (size_t)nc, sizeof(orc_cand_t), orc_cand_cmp);
    int u = 0;                                               /* drop repeats */
    for (int i = 0; i < nc; ++i)
        if (u == 0 || c[i].id != c[u - 1].id) c[u++] = c[i];
    nc = u;
    uint8_t *sel = (uint8_t *)calloc((size_t)nc + 1, 1), *occ = (uint8_t *)malloc((size_t)nc + 1);
    const float alpha2 = alpha * alpha;
    int total = 0;
    for (int ti = 0; ti < T; ++ti) {
        int budget = R * (ti + 1) / T - R * ti / T, taken = 0;
        memset(occ, 0, (size_t)nc + 1);
        for (int i = 0; i < nc && taken < budget; ++i) {
            if (sel[i] || occ[i]) continue;
            if (!orc_attr_within(pos, m_pos, p, c[i].id, thresholds + (size_t)ti * m_pos)) continue;
            sel[i] = 1; taken++;
            row[total++] = c[i].id;
            for (int j = i + 1; j < nc; ++j) {
                if (sel[j]) continue;
                float dcc = orc_point_dist2(ix, c[i].id, c[j].id);
                if (alpha2 * dcc <= c[j].d2) occ[j] = 1;
            }
        }
    }
    for (int i = total; i < R; ++i) row[i] = ORC_SENTINEL;
    free(c); free(sel); free(occ);
    return total;
}

/* graph: [N][R] output (the index's own graph pointer must be this array: the searches of a
   batch read it).  Returns the number of batches. */
int64_t orc_build_graph(orc_index *ix, const float *pos, int m_pos, uint32_t *graph, int R, int Lb,
                        float alpha, const float *thresholds, int T, int B, int passes, int cap_in)
{
    const int64_t N = ix->N;
    for (int64_t i = 0; i < N * R; ++i) graph[i] = ORC_SENTINEL;
    ix->graph = graph; ix->R = R;
    /* the build's searches see the attribute positions as float attribute columns */
    orc_index six = *ix;
    int32_t *ftypes = (int32_t *)malloc((size_t)m_pos * sizeof(int32_t));
    for (int j = 0; j < m_pos; ++j) ftypes[j] = ORC_ATTR_F32;
    six.attrs = (const int32_t *)pos; six.attr_types = ftypes; six.m = m_pos;
    six.metric = 0; six.unit = NULL; six.pq_M = 0;
    orc_state *st = orc_state_new(&six, Lb);
    int32_t *full_lo = (int32_t *)malloc((size_t)m_pos * 4), *full_hi = (int32_t *)malloc((size_t)m_pos * 4);
    float *q = (float *)malloc((size_t)ix->D * sizeof(float));
    const int CW = T * Lb + R;                                 /* candidate slots per point */
    uint32_t *cand = (uint32_t *)malloc((size_t)B * CW * sizeof(uint32_t));
    uint32_t *res_ids = (uint32_t *)malloc((size_t)Lb * sizeof(uint32_t));
    float *res_d2 = (float *)malloc((size_t)Lb * sizeof(float));
    int *ncand = (int *)malloc((size_t)B * sizeof(int));
    uint32_t *req = (uint32_t *)malloc((size_t)B * R * 2 * sizeof(uint32_t));
    uint32_t *tmp = (uint32_t *)malloc((size_t)(R + cap_in + 1) * sizeof(uint32_t));
    int64_t batches = 0, inserted = 0;
    for (int pass = 0; pass < passes; ++pass) {
        int64_t start = 0;
        while (start < N) {
            int64_t bsz = pass == 0 ? (inserted < 1 ? 1 : (inserted < B ? inserted : B)) : B;
            if (start + bsz > N) bsz = N - start;
            /* (a) candidates from the graph as it stands */
            for (int64_t b = 0; b < bsz; ++b) {
                int64_t p = start + b;
                for (int i = 0; i < ix->D; ++i) q[i] = orc_elem(ix, p, i);
                int n = 0;
                for (int ti = 0; ti < T; ++ti) {
                    for (int j = 0; j < m_pos; ++j) {
                        float tj = thresholds[(size_t)ti * m_pos + j];
                        float l = pos[p * m_pos + j] - tj, h = pos[p * m_pos + j] + tj;
                        memcpy(&full_lo[j], &l, 4); memcpy(&full_hi[j], &h, 4);
                    }
                    orc_beam_init(st, Lb, q, full_lo, full_hi, 1);
                    orc_beam_run_w(st, Lb, q, full_lo, full_hi, 1, (int64_t)8 * Lb + 64, 1);
                    int got = orc_beam_result(st, Lb, res_ids, res_d2);
                    for (int t = 0; t < got; ++t) cand[b * CW + n++] = res_ids[t];
                }
                ncand[b] = n;
            }
            /* (b) prune every batch point over candidates + its current row */
            for (int64_t b = 0; b < bsz; ++b) {
                int64_t p = start + b;
                int n = ncand[b];
                for (int j = 0; j < R; ++j) cand[b * CW + n++] = graph[p * R + j];
                orc_prune(ix, pos, m_pos, p, cand + b * CW, n, R, alpha, thresholds, T, graph + p * R);
            }
            /* (c) reverse edges, per target in ascending (target, requester) order */
            int64_t nreq = 0;
            for (int64_t b = 0; b < bsz; ++b)
                for (int j = 0; j < R; ++j) {
                    uint32_t n = graph[(start + b) * R + j];
                    if (n != ORC_SENTINEL) { req[2 * nreq] = n; req[2 * nreq + 1] = (uint32_t)(start + b); nreq++; }
                }
            /* sort the pairs by (target, requester) */
            uint64_t *keys = (uint64_t *)malloc((size_t)(nreq + 1) * sizeof(uint64_t));
            for (int64_t i = 0; i < nreq; ++i) keys[i] = ((uint64_t)req[2 * i] << 32) | req[2 * i + 1];
            for (int64_t i = 1; i < nreq; ++i) {                     /* insertion sort: plain, small */
                uint64_t k = keys[i]; int64_t j = i;
                while (j > 0 && keys[j - 1] > k) { keys[j] = keys[j - 1]; j--; }
                keys[j] = k;
            }
            for (int64_t i = 0; i < nreq;) {
                uint32_t tgt = (uint32_t)(keys[i] >> 32);
                int64_t e = i;
                while (e < nreq && (uint32_t)(keys[e] >> 32) == tgt) e++;
                uint32_t *row = graph + (int64_t)tgt * R;
                int deg = 0, nm = 0;
                while (deg < R && row[deg] != ORC_SENTINEL) deg++;
                for (int64_t r = i; r < e && r < i + cap_in; ++r) {
                    uint32_t rq = (uint32_t)keys[r];
                    int have = 0;
                    for (int j = 0; j < deg; ++j) if (row[j] == rq) have = 1;
                    if (!have) tmp[deg + nm++] = rq;
                }
                if (deg + nm <= R) {
                    for (int j = 0; j < nm; ++j) row[deg + j] = tmp[deg + j];
                } else {
                    for (int j = 0; j < deg; ++j) tmp[j] = row[j];
                    orc_prune(ix, pos, m_pos, tgt, tmp, deg + nm, R, alpha, thresholds, T, row);
                }
                i = e;
            }
            free(keys);
            start += bsz; if (pass == 0) inserted += bsz;
            batches++;
        }
    }
    free(q); free(cand); free(ncand); free(req); free(tmp); free(full_lo); free(full_hi);
    free(res_ids); free(res_d2); free(ftypes);
    orc_state_free(st);
    return batches;
}
