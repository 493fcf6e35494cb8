/* CPU oracle for incremental GNN inference on an evolving graph (RIPPLE++).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path must
 * compute.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it; it
 * shares no code with the CUDA library and the product path never routes through it.
 *
 * Everything floating point is fp64 (the paper does not fix a precision); inputs arrive as fp32
 * and are widened exactly.  Three independent routes to the same per-layer embeddings H^l:
 *
 *   orc_full              whole-graph L-layer inference, the definition (Eq. 1-2, Table 1)
 *   orc_apply_scoped      layer-wise recompute scoped to the affected sets (Sec. 3.2, "RC")
 *   orc_apply_incremental the incremental algorithm (Sec. 3.3): apply, propagation tree,
 *                         delta messages, inbox aggregation, compute
 *
 * Readings taken where the paper is silent (all pinned by the invariant "incremental equals
 * full recomputation", Sec. 3.3.2 / Sec. 5):
 *   - the inbox is kept as a persistent un-normalised aggregate S^l_v = sum_{u in In(v)} c_u h^{l-1}_u;
 *     Update and the activation are re-applied to affected rows (the rule h = h- + W m of
 *     Sec. 3.3.2 is its restriction to the pre-activation);
 *   - mean divides S by the current in-degree at compute time (0 if the in-degree is 0);
 *   - weighted sum uses c_u = deg_out(u)^-1/2 on the source side and deg_in(v)^-1/2 on the sink side,
 *     both from the current graph; a source whose out-degree changed re-sends at every hop;
 *   - "affected" is structural: it follows from the recurrence alone, never from values;
 *   - within a batch the last operation on a pair wins; adding an existing edge or deleting a
 *     missing one changes nothing; the last feature payload of a vertex wins;
 *   - deleting a vertex (Sec. 3.2: all of its incident edges are deleted, then updates propagate
 *     from it as root) removes, at that point of the batch, every edge that has it as an endpoint and
 *     replaces its feature row by zeros; the id stays addressable, so later operations of the same
 *     or a later batch may attach edges or features to it again (a vertex addition, which the
 *     paper models as the edge addition that creates the endpoint, Sec. 4.1);
 *   - attention layers (Sec. 3.4.1, Eq. 3): a vertex with no in-neighbour outputs zeros; the cached
 *     numerator and denominator are the unshifted sums of Eq. 3's terms (the definition route shifts
 *     by the largest logit, the usual evaluation of a softmax); a vertex whose own row changed at hop
 *     l-1 is a hop-l vertex (it recomputes there), so the tree grows with a self term; the layer's
 *     eps is the slope of the logit for negative arguments: 1 gives Eq. 3 as printed, a value below
 *     1 the leaky rectifier of the architecture that Eq. 3 cites; width in = width out;
 *
 * Parity with the authors' own program is unpinned for the mean and weighted-sum degree handling
 * (the paper gives no formula); parity with the definition (orc_full) is pinned for all of it.
 *
 * Edge (u, v): u is the source, v the sink; v aggregates over its in-neighbours.
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { KIND_SAGE = 0, KIND_GRAPHCONV = 1, KIND_GIN = 2, KIND_GAT = 3 };
enum { AGG_SUM = 0, AGG_MEAN = 1, AGG_WSUM_GCN = 2, AGG_MAX = 3, AGG_MIN = 4, AGG_WSUM_EDGE = 5 };
#define MONOTONIC(agg) ((agg) == AGG_MAX || (agg) == AGG_MIN)
enum { ACT_IDENTITY = 0, ACT_RELU = 1 };
enum { OP_ADD_EDGE = 0, OP_DEL_EDGE = 1, OP_SET_FEATURE = 2, OP_DEL_VERTEX = 3 };

typedef struct { int32_t op, u, v; } update_t;

typedef struct {
    int kind, d_in, d_hid, d_out, act;
    double eps;
    double *Wa, *Wb, *ba, *bb; /* input-major: Wa[k * d_next + j] */
} layer_t;

/* ascending neighbour ids; w: the stored weight of each edge (weighted sum with per-edge weights only, else NULL) */
typedef struct { int *a; float *w; int n, cap; } ivec;

typedef struct { int u, v; float w; } pair_t;   /* w: weight of an added edge / weight a deleted edge had */

typedef struct {
    int N, L, agg;
    int weighted;      /* every edge carries a stored weight alpha_uv (Table 1, weighted sum) */
    const float *op_w; /* weights of the batch being applied, one per operation (read for ADD_EDGE only), or NULL = 1 */
    int *d;            /* d[0..L] widths */
    layer_t *layer;    /* layer[1..L] */
    ivec *out, *in;
    double **H;        /* H[0..L]: N x d[l] */
    double **S;        /* S[1..L]: N x d[l-1], un-normalised aggregate (attention: the numerator sum) */
    double **Den;      /* attention layers, Den[1..L]: N, the denominator sum of Eq. 3 */
    double **FH, **FS; /* buffers of orc_full */
    int **A;           /* A[0..L]: affected sets of the last batch, ascending */
    int *nA;
    unsigned char *mark;
    long noop_add, noop_del, superseded;
    long n_added, n_deleted;
    long *active_edges; /* [1..L] out-edges walked at each hop of the last batch */
} oracle_t;

/* ------------------------------------------------------------------------------------------ */
static int cmp_int(const void *a, const void *b) {
    int x = *(const int *)a, y = *(const int *)b;
    return (x > y) - (x < y);
}

static int ivec_find(const ivec *r, int x) { /* index of x or -1 */
    int lo = 0, hi = r->n;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (r->a[mid] < x) lo = mid + 1; else hi = mid;
    }
    return (lo < r->n && r->a[lo] == x) ? lo : -1;
}

static void ivec_insert(ivec *r, int x, int weighted, float w) {
    if (r->n == r->cap) {
        r->cap = r->cap ? 2 * r->cap : 4;
        r->a = (int *)realloc(r->a, sizeof(int) * (size_t)r->cap);
        if (weighted) r->w = (float *)realloc(r->w, sizeof(float) * (size_t)r->cap);
    }
    int i = r->n;
    while (i > 0 && r->a[i - 1] > x) {
        r->a[i] = r->a[i - 1];
        if (weighted) r->w[i] = r->w[i - 1];
        --i;
    }
    r->a[i] = x;
    if (weighted) r->w[i] = w;
    r->n++;
}

static void ivec_erase(ivec *r, int x) {
    int i = ivec_find(r, x);
    if (i < 0) return;
    memmove(r->a + i, r->a + i + 1, sizeof(int) * (size_t)(r->n - i - 1));
    if (r->w) memmove(r->w + i, r->w + i + 1, sizeof(float) * (size_t)(r->n - i - 1));
    r->n--;
}

/* Source-side coefficient c_u (Table 1, weighted sum; 1 for sum and mean). */
static double coef_src(const oracle_t *o, int deg_out) {
    if (o->agg != AGG_WSUM_GCN) return 1.0;
    return deg_out > 0 ? 1.0 / sqrt((double)deg_out) : 0.0;
}

/* Coefficient of the i-th in-edge (u, v) of v inside S_v: the edge's stored weight alpha_uv for the
 * weighted sum with per-edge weights (Table 1), else the source-side coefficient c_u. */
static double in_edge_coef(const oracle_t *o, int v, int i) {
    if (o->weighted) return (double)o->in[v].w[i];
    return coef_src(o, o->out[o->in[v].a[i]].n);
}

/* Sink-side normalisation applied to S_v at compute time (Table 1: mean, weighted sum). */
static double norm_sink(const oracle_t *o, int deg_in) {
    if (o->agg == AGG_SUM || o->agg == AGG_WSUM_EDGE || MONOTONIC(o->agg)) return 1.0;
    if (deg_in <= 0) return 0.0;
    return o->agg == AGG_MEAN ? 1.0 / (double)deg_in : 1.0 / sqrt((double)deg_in);
}

/* h^l_v = sigma(Update^l(h^{l-1}_v, x^l_v)) for one vertex (Eq. 2), x = scale * S_v. */
static void layer_row(const layer_t *ly, const double *hprev, const double *Srow, double scale,
                      double *out) {
    int K = ly->d_in, J = ly->d_out;
    if (ly->kind == KIND_SAGE) {
        for (int j = 0; j < J; ++j) out[j] = ly->ba[j];
        for (int k = 0; k < K; ++k) {
            double h = hprev[k], x = scale * Srow[k];
            const double *wa = ly->Wa + (size_t)k * J, *wb = ly->Wb + (size_t)k * J;
            for (int j = 0; j < J; ++j) out[j] += h * wa[j] + x * wb[j];
        }
    } else if (ly->kind == KIND_GRAPHCONV) {
        for (int j = 0; j < J; ++j) out[j] = ly->ba[j];
        for (int k = 0; k < K; ++k) {
            double x = scale * Srow[k];
            const double *wa = ly->Wa + (size_t)k * J;
            for (int j = 0; j < J; ++j) out[j] += x * wa[j];
        }
    } else { /* GIN: two-layer MLP on (1 + eps) h_v + x_v */
        int Hd = ly->d_hid;
        double *z = (double *)malloc(sizeof(double) * (size_t)Hd);
        for (int j = 0; j < Hd; ++j) z[j] = ly->ba[j];
        for (int k = 0; k < K; ++k) {
            double t = (1.0 + ly->eps) * hprev[k] + scale * Srow[k];
            const double *wa = ly->Wa + (size_t)k * Hd;
            for (int j = 0; j < Hd; ++j) z[j] += t * wa[j];
        }
        for (int j = 0; j < J; ++j) out[j] = ly->bb[j];
        for (int k = 0; k < Hd; ++k) {
            double t = z[k] > 0.0 ? z[k] : 0.0;
            const double *wb = ly->Wb + (size_t)k * J;
            for (int j = 0; j < J; ++j) out[j] += t * wb[j];
        }
        free(z);
    }
    if (ly->act == ACT_RELU)
        for (int j = 0; j < J; ++j) out[j] = out[j] > 0.0 ? out[j] : 0.0;
}

/* x^l_v before normalisation: S_v = sum over in-neighbours of c_u h^{l-1}_u (Eq. 1, Table 1). */
static void aggregate_row(const oracle_t *o, int v, const double *Hprev, int K, double *Srow) {
    for (int k = 0; k < K; ++k) Srow[k] = 0.0;
    const ivec *in = &o->in[v];
    if (MONOTONIC(o->agg)) { /* element-wise maximum (minimum) over the in-neighbours; none: zeros */
        int is_min = o->agg == AGG_MIN;
        for (int i = 0; i < in->n; ++i) {
            const double *h = Hprev + (size_t)in->a[i] * K;
            for (int k = 0; k < K; ++k)
                if (i == 0 || (is_min ? h[k] < Srow[k] : h[k] > Srow[k])) Srow[k] = h[k];
        }
        return;
    }
    for (int i = 0; i < in->n; ++i) {
        int u = in->a[i];
        double c = in_edge_coef(o, v, i);
        const double *h = Hprev + (size_t)u * K;
        for (int k = 0; k < K; ++k) Srow[k] += c * h[k];
    }
}

/* ------------------------------------------------------------------------------------------ */
typedef struct { int id; float w; } idw_t;
static int cmp_idw(const void *a, const void *b) {
    int x = ((const idw_t *)a)->id, y = ((const idw_t *)b)->id;
    return (x > y) - (x < y);
}
static void sort_list(ivec *r) {   /* ascending ids, weights (if any) moving with them */
    if (!r->w) { qsort(r->a, (size_t)r->n, sizeof(int), cmp_int); return; }
    idw_t *t = (idw_t *)malloc(sizeof(idw_t) * (size_t)(r->n + 1));
    for (int i = 0; i < r->n; ++i) { t[i].id = r->a[i]; t[i].w = r->w[i]; }
    qsort(t, (size_t)r->n, sizeof(idw_t), cmp_idw);
    for (int i = 0; i < r->n; ++i) { r->a[i] = t[i].id; r->w[i] = t[i].w; }
    free(t);
}

/* weight: one stored weight per edge (required for the weighted sum with per-edge weights), or NULL */
oracle_t *orc_create_weighted(int N, int64_t E, const int32_t *src, const int32_t *dst, const float *weight,
                              const float *feat, int L, const int *dims, int agg) {
    oracle_t *o = (oracle_t *)calloc(1, sizeof(oracle_t));
    o->N = N; o->L = L; o->agg = agg;
    o->weighted = agg == AGG_WSUM_EDGE;
    o->d = (int *)malloc(sizeof(int) * (size_t)(L + 1));
    memcpy(o->d, dims, sizeof(int) * (size_t)(L + 1));
    o->layer = (layer_t *)calloc((size_t)L + 1, sizeof(layer_t));
    o->out = (ivec *)calloc((size_t)N, sizeof(ivec));
    o->in = (ivec *)calloc((size_t)N, sizeof(ivec));
    for (int64_t e = 0; e < E; ++e) { o->out[src[e]].cap++; o->in[dst[e]].cap++; }
    for (int v = 0; v < N; ++v) {
        if (o->out[v].cap) o->out[v].a = (int *)malloc(sizeof(int) * (size_t)o->out[v].cap);
        if (o->in[v].cap) o->in[v].a = (int *)malloc(sizeof(int) * (size_t)o->in[v].cap);
        if (o->weighted && o->out[v].cap) o->out[v].w = (float *)malloc(sizeof(float) * (size_t)o->out[v].cap);
        if (o->weighted && o->in[v].cap) o->in[v].w = (float *)malloc(sizeof(float) * (size_t)o->in[v].cap);
    }
    for (int64_t e = 0; e < E; ++e) {
        ivec *r = &o->out[src[e]];
        ivec *c = &o->in[dst[e]];
        if (o->weighted) { r->w[r->n] = weight ? weight[e] : 1.0f; c->w[c->n] = weight ? weight[e] : 1.0f; }
        r->a[r->n++] = dst[e];
        c->a[c->n++] = src[e];
    }
#pragma omp parallel for schedule(dynamic, 1024)
    for (int v = 0; v < N; ++v) {
        sort_list(&o->out[v]);
        sort_list(&o->in[v]);
    }
    o->H = (double **)calloc((size_t)L + 1, sizeof(double *));
    o->S = (double **)calloc((size_t)L + 1, sizeof(double *));
    o->FH = (double **)calloc((size_t)L + 1, sizeof(double *));
    o->FS = (double **)calloc((size_t)L + 1, sizeof(double *));
    o->Den = (double **)calloc((size_t)L + 1, sizeof(double *));
    o->A = (int **)calloc((size_t)L + 1, sizeof(int *));
    o->nA = (int *)calloc((size_t)L + 1, sizeof(int));
    o->active_edges = (long *)calloc((size_t)L + 1, sizeof(long));
    o->mark = (unsigned char *)calloc((size_t)N, 1);
    for (int l = 0; l <= L; ++l) {
        o->H[l] = (double *)calloc((size_t)N * (size_t)dims[l], sizeof(double));
        if (l > 0) o->S[l] = (double *)calloc((size_t)N * (size_t)dims[l - 1], sizeof(double));
        if (l > 0) o->Den[l] = (double *)calloc((size_t)N, sizeof(double));
    }
    for (size_t i = 0; i < (size_t)N * (size_t)dims[0]; ++i) o->H[0][i] = (double)feat[i];
    return o;
}

oracle_t *orc_create(int N, int64_t E, const int32_t *src, const int32_t *dst, const float *feat,
                     int L, const int *dims, int agg) {
    return orc_create_weighted(N, E, src, dst, NULL, feat, L, dims, agg);
}

static double *widen(const float *x, size_t n) {
    if (!x) return NULL;
    double *r = (double *)malloc(sizeof(double) * n);
    for (size_t i = 0; i < n; ++i) r[i] = (double)x[i];
    return r;
}

/* l is 1-based.  Matrices are input-major (fan_in x fan_out, row-major). */
void orc_set_layer(oracle_t *o, int l, int kind, int d_hid, int act, double eps,
                   const float *Wa, const float *Wb, const float *ba, const float *bb) {
    layer_t *ly = &o->layer[l];
    ly->kind = kind; ly->d_in = o->d[l - 1]; ly->d_out = o->d[l]; ly->d_hid = d_hid;
    ly->act = act; ly->eps = eps;
    size_t K = (size_t)ly->d_in, J = (size_t)ly->d_out, Hd = (size_t)d_hid;
    if (kind == KIND_GIN) {
        ly->Wa = widen(Wa, K * Hd); ly->ba = widen(ba, Hd);
        ly->Wb = widen(Wb, Hd * J); ly->bb = widen(bb, J);
    } else if (kind == KIND_GAT) {   /* Wa = W (d_in x d_hid), ba = source half of a, bb = sink half of a (Eq. 3) */
        ly->Wa = widen(Wa, K * Hd); ly->ba = widen(ba, Hd); ly->bb = widen(bb, Hd);
    } else {
        ly->Wa = widen(Wa, K * J); ly->ba = widen(ba, J);
        ly->Wb = kind == KIND_SAGE ? widen(Wb, K * J) : NULL;
    }
}

void orc_destroy(oracle_t *o) {
    if (!o) return;
    for (int v = 0; v < o->N; ++v) { free(o->out[v].a); free(o->in[v].a); free(o->out[v].w); free(o->in[v].w); }
    for (int l = 0; l <= o->L; ++l) {
        free(o->H[l]); free(o->S[l]); free(o->FH[l]); free(o->FS[l]); free(o->A[l]); free(o->Den[l]);
        free(o->layer[l].Wa); free(o->layer[l].Wb); free(o->layer[l].ba); free(o->layer[l].bb);
    }
    free(o->out); free(o->in); free(o->H); free(o->S); free(o->FH); free(o->FS); free(o->A); free(o->Den);
    free(o->nA); free(o->layer); free(o->d); free(o->mark); free(o->active_edges); free(o);
}

/* One whole layer for every vertex (Eq. 1-2): S = aggregate, H = sigma(Update). */
/* ------------------------------------------------------------------------------------------ */
/* Attention layers (Sec. 3.4.1, Eq. 3): h^{l+1}_v = sum_{u in In(v)} alpha_uv h^l_u,
 * alpha_uv = softmax over In(v) of z_uv, z_uv = a . (W h_u || W h_v).  No in-neighbours: zeros. */
/* z = a . (W h_u || W h_v) as Eq. 3 prints it when eps (the slope for negative arguments) is 1; the
 * architecture Eq. 3 cites passes that number through a leaky rectifier, which is eps < 1 */
static double gat_logit(const layer_t *ly, double s_u, double t_v) {
    double z = s_u + t_v;
    return z < 0.0 ? ly->eps * z : z;
}

static double gat_logit_part(const layer_t *ly, const double *a_half, const double *h) {
    double s = 0.0;   /* a_half . (W h), W h = Wa^T h with Wa input-major */
    for (int j = 0; j < ly->d_hid; ++j) {
        double wh = 0.0;
        for (int k = 0; k < ly->d_in; ++k) wh += ly->Wa[(size_t)k * ly->d_hid + j] * h[k];
        s += a_half[j] * wh;
    }
    return s;
}

/* the definition for one vertex, with the usual shift by the largest logit; sv / tv: the two halves of
 * the logit for every vertex if the caller has them (whole-graph passes), else NULL */
static void gat_row_definition(const oracle_t *o, int l, int v, const double *Hprev, const double *sv,
                               const double *tv_all, double *out) {
    const layer_t *ly = &o->layer[l];
    int K = o->d[l - 1];
    const ivec *in = &o->in[v];
    for (int k = 0; k < K; ++k) out[k] = 0.0;
    if (in->n == 0) return;
    double tv = tv_all ? tv_all[v] : gat_logit_part(ly, ly->bb, Hprev + (size_t)v * K);
    double *z = (double *)malloc(sizeof(double) * (size_t)in->n), zmax = -1e300, den = 0.0;
    for (int i = 0; i < in->n; ++i) {
        z[i] = gat_logit(ly, sv ? sv[in->a[i]] : gat_logit_part(ly, ly->ba, Hprev + (size_t)in->a[i] * K), tv);
        if (z[i] > zmax) zmax = z[i];
    }
    for (int i = 0; i < in->n; ++i) den += exp(z[i] - zmax);
    for (int i = 0; i < in->n; ++i) {
        double alpha = exp(z[i] - zmax) / den;
        const double *h = Hprev + (size_t)in->a[i] * K;
        for (int k = 0; k < K; ++k) out[k] += alpha * h[k];
    }
    free(z);
    if (ly->act == ACT_RELU) for (int k = 0; k < K; ++k) out[k] = out[k] > 0.0 ? out[k] : 0.0;
}

/* numerator and denominator sums of Eq. 3 as the incremental route caches them (no shift) */
static void gat_sums(const oracle_t *o, int l, int v, const double *Hprev, const double *sv,
                     const double *tv_all, double *num, double *den) {
    const layer_t *ly = &o->layer[l];
    int K = o->d[l - 1];
    const ivec *in = &o->in[v];
    for (int k = 0; k < K; ++k) num[k] = 0.0;
    *den = 0.0;
    double tv = tv_all ? tv_all[v] : gat_logit_part(ly, ly->bb, Hprev + (size_t)v * K);
    for (int i = 0; i < in->n; ++i) {
        const double *h = Hprev + (size_t)in->a[i] * K;
        double e = exp(gat_logit(ly, sv ? sv[in->a[i]] : gat_logit_part(ly, ly->ba, h), tv));
        for (int k = 0; k < K; ++k) num[k] += e * h[k];
        *den += e;
    }
}

static void gat_output(const layer_t *ly, int K, int deg_in, const double *num, double den, double *out) {
    for (int k = 0; k < K; ++k) {
        double x = deg_in > 0 ? num[k] / den : 0.0;
        out[k] = (ly->act == ACT_RELU && x < 0.0) ? 0.0 : x;
    }
}

static void full_layer(const oracle_t *o, int l, const double *Hprev, double *S, double *H) {
    int K = o->d[l - 1], J = o->d[l];
    if (o->layer[l].kind == KIND_GAT) {
        double *sv = (double *)malloc(sizeof(double) * (size_t)o->N), *tv = (double *)malloc(sizeof(double) * (size_t)o->N);
#pragma omp parallel for schedule(static)
        for (int v = 0; v < o->N; ++v) {
            sv[v] = gat_logit_part(&o->layer[l], o->layer[l].ba, Hprev + (size_t)v * K);
            tv[v] = gat_logit_part(&o->layer[l], o->layer[l].bb, Hprev + (size_t)v * K);
        }
#pragma omp parallel for schedule(dynamic, 256)
        for (int v = 0; v < o->N; ++v) {
            double den;
            gat_sums(o, l, v, Hprev, sv, tv, S + (size_t)v * K, &den);
            if (S == o->S[l]) o->Den[l][v] = den;          /* the cached state (bootstrap), not the buffers of orc_full */
            gat_row_definition(o, l, v, Hprev, sv, tv, H + (size_t)v * J);
        }
        free(sv); free(tv);
        return;
    }
#pragma omp parallel for schedule(dynamic, 256)
    for (int v = 0; v < o->N; ++v) {
        aggregate_row(o, v, Hprev, K, S + (size_t)v * K);
        layer_row(&o->layer[l], Hprev + (size_t)v * K, S + (size_t)v * K,
                  norm_sink(o, o->in[v].n), H + (size_t)v * J);
    }
}

/* O-full: layer-wise inference over the whole current graph into separate buffers
 * (Sec. 1.1 layer-wise inference; Sec. 3.1 bootstrap embeddings H^l_{T0}). */
void orc_full(oracle_t *o) {
    for (int l = 1; l <= o->L; ++l) {
        if (!o->FH[l]) o->FH[l] = (double *)malloc(sizeof(double) * (size_t)o->N * (size_t)o->d[l]);
        if (!o->FS[l]) o->FS[l] = (double *)malloc(sizeof(double) * (size_t)o->N * (size_t)o->d[l - 1]);
        full_layer(o, l, l == 1 ? o->H[0] : o->FH[l - 1], o->FS[l], o->FH[l]);
    }
}

/* Bootstrap: the cached state becomes the full inference on the current graph (Sec. 3.1). */
void orc_bootstrap(oracle_t *o) {
    for (int l = 1; l <= o->L; ++l) full_layer(o, l, o->H[l - 1], o->S[l], o->H[l]);
}

/* ------------------------------------------------------------------------------------------ */
/* Batch normalisation shared by the two update routes (Sec. 3.1 batching; Sec. 3.3 Apply). */
typedef struct { int u, v, seq, op; } eop_t;
typedef struct { int v, seq, row; } fop_t;

static int cmp_eop(const void *a, const void *b) {
    const eop_t *x = (const eop_t *)a, *y = (const eop_t *)b;
    if (x->u != y->u) return x->u < y->u ? -1 : 1;
    if (x->v != y->v) return x->v < y->v ? -1 : 1;
    return (x->seq > y->seq) - (x->seq < y->seq);
}
static int cmp_fop(const void *a, const void *b) {
    const fop_t *x = (const fop_t *)a, *y = (const fop_t *)b;
    if (x->v != y->v) return x->v < y->v ? -1 : 1;
    return (x->seq > y->seq) - (x->seq < y->seq);
}
static int cmp_pair(const void *a, const void *b) {
    const pair_t *x = (const pair_t *)a, *y = (const pair_t *)b;
    if (x->u != y->u) return x->u < y->u ? -1 : 1;
    return (x->v > y->v) - (x->v < y->v);
}

typedef struct {
    pair_t *add, *del; /* net added / deleted edges, sorted by (u, v) */
    int n_add, n_del;
    int *F, *Frow;     /* vertices with a feature update (ascending) and the winning payload row */
    int nF;
} delta_t;

/* last explicit edge operation on (u, v) in the sorted table, or NULL */
static const eop_t *eop_last(const eop_t *eo, int ne, int u, int v) {
    int lo = 0, hi = ne;   /* first entry with (u', v') > (u, v) */
    while (lo < hi) {
        int mid = (lo + hi) / 2;
        if (eo[mid].u < u || (eo[mid].u == u && eo[mid].v <= v)) lo = mid + 1; else hi = mid;
    }
    if (lo == 0 || eo[lo - 1].u != u || eo[lo - 1].v != v) return NULL;
    return &eo[lo - 1];
}

/* Net effect of applying the operations one after the other:
 *   - an edge operation is the final word on its pair if no later edge operation names the pair
 *     and neither endpoint is deleted later; it then adds / deletes the edge or is a counted no-op;
 *     every other edge operation is counted as superseded;
 *   - a vertex deletion removes every edge of E_old at that vertex whose pair has no final word;
 *   - the last of {feature replacement, deletion} of a vertex fixes its row (deletion: zeros). */
static int normalise(oracle_t *o, const update_t *ups, int64_t n, int64_t n_rows, delta_t *dl) {
    memset(dl, 0, sizeof(*dl));
    for (int64_t i = 0; i < n; ++i) {
        if (ups[i].op < 0 || ups[i].op > 3) return -1;
        if (ups[i].u < 0 || ups[i].u >= o->N) return -2;
        if (ups[i].op == OP_DEL_VERTEX) continue;
        if (ups[i].op == OP_SET_FEATURE) { if (ups[i].v < 0 || ups[i].v >= n_rows) return -1; }
        else if (ups[i].v < 0 || ups[i].v >= o->N) return -2;
    }
    eop_t *eo = (eop_t *)malloc(sizeof(eop_t) * (size_t)(n + 1));
    fop_t *fo = (fop_t *)malloc(sizeof(fop_t) * (size_t)(n + 1));
    int *gone = (int *)malloc(sizeof(int) * (size_t)(n + 1));   /* deleted vertices, one entry per deletion */
    int ne = 0, nf = 0, ng = 0;
    int *vdel = NULL;   /* position of the last deletion of each vertex, -1 if none */
    for (int64_t i = 0; i < n; ++i) {
        if (ups[i].op == OP_DEL_VERTEX) {
            if (!vdel) { vdel = (int *)malloc(sizeof(int) * (size_t)o->N); for (int v = 0; v < o->N; ++v) vdel[v] = -1; }
            vdel[ups[i].u] = (int)i;
            gone[ng++] = ups[i].u;
            fo[nf].v = ups[i].u; fo[nf].seq = (int)i; fo[nf].row = -1; nf++;
        } else if (ups[i].op == OP_SET_FEATURE) {
            fo[nf].v = ups[i].u; fo[nf].seq = (int)i; fo[nf].row = ups[i].v; nf++;
        } else { eo[ne].u = ups[i].u; eo[ne].v = ups[i].v; eo[ne].seq = (int)i; eo[ne].op = ups[i].op; ne++; }
    }
    qsort(eo, (size_t)ne, sizeof(eop_t), cmp_eop);
    qsort(fo, (size_t)nf, sizeof(fop_t), cmp_fop);
    size_t del_cap = (size_t)ne + 1;
    for (int i = 0; i < ng; ++i) del_cap += (size_t)o->out[gone[i]].n + (size_t)o->in[gone[i]].n;
    dl->add = (pair_t *)malloc(sizeof(pair_t) * (size_t)(ne + 1));
    dl->del = (pair_t *)malloc(sizeof(pair_t) * del_cap);
    o->noop_add = o->noop_del = o->superseded = 0;
#define FINAL_WORD(e) (!vdel || ((e)->seq > vdel[(e)->u] && (e)->seq > vdel[(e)->v]))
    for (int i = 0; i < ne; ++i) {
        if (i + 1 < ne && eo[i + 1].u == eo[i].u && eo[i + 1].v == eo[i].v) { o->superseded++; continue; }
        if (!FINAL_WORD(&eo[i])) { o->superseded++; continue; }
        int at = ivec_find(&o->out[eo[i].u], eo[i].v), present = at >= 0;
        if (eo[i].op == OP_ADD_EDGE) {   /* an edge that exists keeps the weight it has */
            if (present) o->noop_add++;
            else {
                dl->add[dl->n_add].u = eo[i].u; dl->add[dl->n_add].v = eo[i].v;
                dl->add[dl->n_add].w = o->op_w ? o->op_w[eo[i].seq] : 1.0f;
                dl->n_add++;
            }
        } else {
            if (!present) o->noop_del++;
            else {
                dl->del[dl->n_del].u = eo[i].u; dl->del[dl->n_del].v = eo[i].v;
                dl->del[dl->n_del].w = o->weighted ? o->out[eo[i].u].w[at] : 1.0f;
                dl->n_del++;
            }
        }
    }
    if (ng) {
        for (int i = 0; i < ng; ++i) {
            int w = gone[i];
            for (int side = 0; side < 2; ++side) {
                const ivec *r = side ? &o->in[w] : &o->out[w];
                for (int j = 0; j < r->n; ++j) {
                    int u = side ? r->a[j] : w, v = side ? w : r->a[j];
                    const eop_t *e = eop_last(eo, ne, u, v);
                    if (e && FINAL_WORD(e)) continue;   /* a later operation on the pair decided */
                    dl->del[dl->n_del].u = u; dl->del[dl->n_del].v = v;
                    dl->del[dl->n_del].w = o->weighted ? r->w[j] : 1.0f;
                    dl->n_del++;
                }
            }
        }
        /* a pair is met once per deleted endpoint and per list it is in: keep one copy */
        qsort(dl->del, (size_t)dl->n_del, sizeof(pair_t), cmp_pair);
        int k = 0;
        for (int i = 0; i < dl->n_del; ++i)
            if (k == 0 || dl->del[k - 1].u != dl->del[i].u || dl->del[k - 1].v != dl->del[i].v) dl->del[k++] = dl->del[i];
        dl->n_del = k;
    }
#undef FINAL_WORD
    dl->F = (int *)malloc(sizeof(int) * (size_t)(nf + 1));
    dl->Frow = (int *)malloc(sizeof(int) * (size_t)(nf + 1));
    for (int i = 0; i < nf; ++i) {
        if (i + 1 < nf && fo[i + 1].v == fo[i].v) continue;
        dl->F[dl->nF] = fo[i].v; dl->Frow[dl->nF] = fo[i].row; dl->nF++;
    }
    o->n_added = dl->n_add; o->n_deleted = dl->n_del;
    free(eo); free(fo); free(gone); free(vdel);
    return 0;
}

static void delta_free(delta_t *dl) { free(dl->add); free(dl->del); free(dl->F); free(dl->Frow); }

static void set_list(oracle_t *o, int l, const int *ids, int n) {
    free(o->A[l]);
    o->A[l] = (int *)malloc(sizeof(int) * (size_t)(n + 1));
    memcpy(o->A[l], ids, sizeof(int) * (size_t)n);
    o->nA[l] = n;
}

/* sorted list of the marked vertices among cand[0..nc); clears the marks */
static int collect_marked(oracle_t *o, int *cand, int nc, int *out) {
    int n = 0;
    for (int i = 0; i < nc; ++i) if (o->mark[cand[i]]) { o->mark[cand[i]] = 0; out[n++] = cand[i]; }
    qsort(out, (size_t)n, sizeof(int), cmp_int);
    return n;
}

/* A_l = sinks(dE) U Out_new(C_{l-1}) U (self term ? A_{l-1} : {}) -- the hop-l vertices of the
 * propagation tree (Sec. 3.2: sink of an edge change is touched at every hop, out-neighbours of
 * changed vertices at the next hop; Sec. 3.3: BFS from the roots).  Returns the list, ascending. */
static int *next_affected(oracle_t *o, const delta_t *dl, const int *Cprev, int nCprev,
                          const int *Aprev, int nAprev, int self_term, int *n_out, long *walked) {
    size_t bound = (size_t)dl->n_add + (size_t)dl->n_del + (size_t)nAprev + 1;
    for (int i = 0; i < nCprev; ++i) bound += (size_t)o->out[Cprev[i]].n;
    int *cand = (int *)malloc(sizeof(int) * bound), nc = 0;
    long w = 0;
    for (int i = 0; i < dl->n_add; ++i) { cand[nc++] = dl->add[i].v; o->mark[dl->add[i].v] = 1; }
    for (int i = 0; i < dl->n_del; ++i) { cand[nc++] = dl->del[i].v; o->mark[dl->del[i].v] = 1; }
    for (int i = 0; i < nCprev; ++i) {
        const ivec *r = &o->out[Cprev[i]];
        w += r->n;
        for (int j = 0; j < r->n; ++j) { cand[nc++] = r->a[j]; o->mark[r->a[j]] = 1; }
    }
    if (self_term) for (int i = 0; i < nAprev; ++i) { cand[nc++] = Aprev[i]; o->mark[Aprev[i]] = 1; }
    int *out = (int *)malloc(sizeof(int) * (size_t)(nc + 1));
    *n_out = collect_marked(o, cand, nc, out);
    free(cand);
    if (walked) *walked = w;
    return out;
}

/* C_l = A_l U (source-side coefficient depends on degree ? sources(dE) : {}) */
static int *changed_senders(oracle_t *o, const delta_t *dl, const int *A, int nA, int *n_out) {
    int cap = nA + dl->n_add + dl->n_del + 1;
    int *cand = (int *)malloc(sizeof(int) * (size_t)cap), nc = 0;
    for (int i = 0; i < nA; ++i) { cand[nc++] = A[i]; o->mark[A[i]] = 1; }
    if (o->agg == AGG_WSUM_GCN) {
        for (int i = 0; i < dl->n_add; ++i) { cand[nc++] = dl->add[i].u; o->mark[dl->add[i].u] = 1; }
        for (int i = 0; i < dl->n_del; ++i) { cand[nc++] = dl->del[i].u; o->mark[dl->del[i].u] = 1; }
    }
    int *out = (int *)malloc(sizeof(int) * (size_t)(nc + 1));
    *n_out = collect_marked(o, cand, nc, out);
    free(cand);
    return out;
}

/* Apply: mutate topology and features (Sec. 3.3, first step of the lifecycle). */
static void apply_topology(oracle_t *o, const delta_t *dl) {
    for (int i = 0; i < dl->n_add; ++i) {
        ivec_insert(&o->out[dl->add[i].u], dl->add[i].v, o->weighted, dl->add[i].w);
        ivec_insert(&o->in[dl->add[i].v], dl->add[i].u, o->weighted, dl->add[i].w);
    }
    for (int i = 0; i < dl->n_del; ++i) {
        ivec_erase(&o->out[dl->del[i].u], dl->del[i].v);
        ivec_erase(&o->in[dl->del[i].v], dl->del[i].u);
    }
}

static int find_sorted(const int *a, int n, int x) {
    int lo = 0, hi = n;
    while (lo < hi) { int mid = (lo + hi) >> 1; if (a[mid] < x) lo = mid + 1; else hi = mid; }
    return (lo < n && a[lo] == x) ? lo : -1;
}

/* Per distinct source of a net edge change: how many of its out-edges were added / deleted, and
 * its source-side coefficient before the batch. */
typedef struct { int u, n_add, n_del; double c_old; } srcinfo_t;

static int cmp_srcinfo(const void *a, const void *b) {
    int x = ((const srcinfo_t *)a)->u, y = ((const srcinfo_t *)b)->u;
    return (x > y) - (x < y);
}

/* call after Apply: deg_out_old(u) = deg_out_new(u) - added + deleted */
static srcinfo_t *source_table(const oracle_t *o, const delta_t *dl, int *n_out) {
    int n = dl->n_add + dl->n_del, m = 0;
    srcinfo_t *raw = (srcinfo_t *)calloc((size_t)n + 1, sizeof(srcinfo_t));
    for (int i = 0; i < dl->n_add; ++i) { raw[i].u = dl->add[i].u; raw[i].n_add = 1; }
    for (int i = 0; i < dl->n_del; ++i) { raw[dl->n_add + i].u = dl->del[i].u; raw[dl->n_add + i].n_del = 1; }
    qsort(raw, (size_t)n, sizeof(srcinfo_t), cmp_srcinfo);
    for (int i = 0; i < n; ++i) {
        if (m > 0 && raw[m - 1].u == raw[i].u) { raw[m - 1].n_add += raw[i].n_add; raw[m - 1].n_del += raw[i].n_del; }
        else raw[m++] = raw[i];
    }
    for (int i = 0; i < m; ++i)
        raw[i].c_old = coef_src(o, o->out[raw[i].u].n - raw[i].n_add + raw[i].n_del);
    *n_out = m;
    return raw;
}

static const srcinfo_t *source_find(const srcinfo_t *t, int n, int u) {
    srcinfo_t key; key.u = u;
    return (const srcinfo_t *)bsearch(&key, t, (size_t)n, sizeof(srcinfo_t), cmp_srcinfo);
}

/* ------------------------------------------------------------------------------------------ */
/* Monotonic aggregation (Sec. 3.4.2), max (min is its mirror image: read "exceeds" as "is below"
 * and so on), for GraphConv and SAGE layers.  A message
 * <old, new> from a changed in-neighbour, <-, new> along an added edge or <old, -> along a deleted
 * one leads, per element, to one of three actions at the sink:
 *   - new exceeds the cached maximum: the cache is raised to it (incremental);
 *   - old was the cached maximum and new is smaller (or the edge is gone): the maximum is no longer
 *     known, the sink recomputes it over all current in-neighbours;
 *   - otherwise nothing happens.
 * A sink whose cached row ends up unchanged is not affected and sends nothing on (the pruning of
 * Sec. 6.3); with a self term a vertex is also affected when its own previous-layer row changed.  "Changed" is decided on the values rounded to single precision, the precision of the
 * embeddings this oracle is compared with. */
static int differs_f32(const double *a, const double *b, int n) {
    for (int k = 0; k < n; ++k) if ((float)a[k] != (float)b[k]) return 1;
    return 0;
}

static int apply_incremental_max(oracle_t *o, const delta_t *dl, const float *feat_rows) {
    int L = o->L, N = o->N, self_term = o->layer[1].kind != KIND_GRAPHCONV;
    int d0 = o->d[0];
    int is_min = o->agg == AGG_MIN;
#define BEATS(a, b) (is_min ? (a) < (b) : (a) > (b))   /* a improves on b */
    /* in-degree before the batch: a sink that had no in-neighbour caches zeros, not a maximum */
    int *din_old = (int *)malloc(sizeof(int) * (size_t)N);
    for (int v = 0; v < N; ++v) din_old[v] = o->in[v].n;
    for (int i = 0; i < dl->n_add; ++i) din_old[dl->add[i].v]--;
    for (int i = 0; i < dl->n_del; ++i) din_old[dl->del[i].v]++;

    int nA = dl->nF;
    int *A = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
    memcpy(A, dl->F, sizeof(int) * (size_t)nA);
    double *oldA = (double *)malloc(sizeof(double) * ((size_t)nA * (size_t)d0 + 1));
    for (int i = 0; i < nA; ++i) {
        double *row = o->H[0] + (size_t)A[i] * d0;
        memcpy(oldA + (size_t)i * d0, row, sizeof(double) * (size_t)d0);
        const float *src = dl->Frow[i] >= 0 ? feat_rows + (size_t)dl->Frow[i] * d0 : NULL;
        for (int k = 0; k < d0; ++k) row[k] = src ? (double)src[k] : 0.0;
    }
    set_list(o, 0, A, nA);

    int *snap_of = (int *)malloc(sizeof(int) * (size_t)N);   /* vertex -> its saved row, or -1 */
    for (int v = 0; v < N; ++v) snap_of[v] = -1;
    unsigned char *need = (unsigned char *)calloc((size_t)N, 1);

    for (int l = 1; l <= L; ++l) {
        int K = o->d[l - 1], J = o->d[l];
        const double *Hp = o->H[l - 1];
        double *S = o->S[l];
        /* senders: rows of A_{l-1} that really changed */
        int nC = 0;
        int *C = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
        int *Cold = (int *)malloc(sizeof(int) * (size_t)(nA + 1));   /* index of the sender's old row */
        for (int i = 0; i < nA; ++i)
            if (differs_f32(Hp + (size_t)A[i] * K, oldA + (size_t)i * K, K)) { C[nC] = A[i]; Cold[nC] = i; nC++; }

        int cap = 1024, nT = 0;              /* touched sinks and their rows before this hop */
        int *T = (int *)malloc(sizeof(int) * (size_t)cap);
        double *snap = (double *)malloc(sizeof(double) * (size_t)cap * (size_t)K);
        long walked = 0;
#define TOUCH(v)                                                                                   \
        do {                                                                                       \
            if (snap_of[v] < 0) {                                                                  \
                if (nT == cap) { cap *= 2; T = (int *)realloc(T, sizeof(int) * (size_t)cap);       \
                                 snap = (double *)realloc(snap, sizeof(double) * (size_t)cap * (size_t)K); } \
                memcpy(snap + (size_t)nT * K, S + (size_t)(v) * K, sizeof(double) * (size_t)K);    \
                snap_of[v] = nT; T[nT++] = (v);                                                    \
            }                                                                                      \
        } while (0)
        /* <old, new> along the surviving out-edges of the senders */
        for (int i = 0; i < nC; ++i) {
            int u = C[i];
            const double *hnew = Hp + (size_t)u * K, *hold = oldA + (size_t)Cold[i] * K;
            const ivec *r = &o->out[u];
            walked += r->n;
            for (int j = 0; j < r->n; ++j) {
                int v = r->a[j];
                pair_t p = { u, v, 0.f };
                if (dl->n_add && bsearch(&p, dl->add, (size_t)dl->n_add, sizeof(pair_t), cmp_pair)) continue;
                double *Sv = S + (size_t)v * K;
                for (int k = 0; k < K; ++k) {
                    if (BEATS(hnew[k], Sv[k])) { TOUCH(v); Sv[k] = hnew[k]; }
                    else if (hold[k] == Sv[k] && BEATS(hold[k], hnew[k])) need[v] = 1;
                }
            }
        }
        /* <-, new> along added edges */
        for (int i = 0; i < dl->n_add; ++i) {
            int u = dl->add[i].u, v = dl->add[i].v;
            if (din_old[v] == 0) { need[v] = 1; continue; }
            const double *hnew = Hp + (size_t)u * K;
            double *Sv = S + (size_t)v * K;
            for (int k = 0; k < K; ++k) if (BEATS(hnew[k], Sv[k])) { TOUCH(v); Sv[k] = hnew[k]; }
        }
        /* <old, -> along deleted edges */
        for (int i = 0; i < dl->n_del; ++i) {
            int u = dl->del[i].u, v = dl->del[i].v;
            int ia = find_sorted(A, nA, u);
            const double *hold = ia >= 0 ? oldA + (size_t)ia * K : Hp + (size_t)u * K;
            const double *Sv = S + (size_t)v * K;
            if (o->in[v].n == 0) need[v] = 1;
            for (int k = 0; k < K && !need[v]; ++k) if (hold[k] == Sv[k]) need[v] = 1;
        }
        /* recomputation of the sinks whose maximum is no longer known */
        for (int v = 0; v < N; ++v) {
            if (!need[v]) continue;
            need[v] = 0;
            TOUCH(v);
            aggregate_row(o, v, Hp, K, S + (size_t)v * K);
        }
#undef TOUCH
        o->active_edges[l] = walked + dl->n_add + dl->n_del;
        /* affected = cached row changed */
        int nAn = 0;
        int *An = (int *)malloc(sizeof(int) * (size_t)(nT + 1));
        for (int t = 0; t < nT; ++t) {
            int v = T[t];
            if (differs_f32(S + (size_t)v * K, snap + (size_t)t * K, K)) An[nAn++] = v;
            snap_of[v] = -1;
        }
        /* with a self term a vertex whose own h^{l-1} changed recomputes h^l as well */
        if (self_term) {
            for (int t = 0; t < nAn; ++t) o->mark[An[t]] = 1;
            An = (int *)realloc(An, sizeof(int) * (size_t)(nAn + nC + 1));
            int base = nAn;
            for (int i = 0; i < nC; ++i) if (!o->mark[C[i]]) An[nAn++] = C[i];
            for (int t = 0; t < base; ++t) o->mark[An[t]] = 0;
        }
        qsort(An, (size_t)nAn, sizeof(int), cmp_int);
        free(T); free(snap); free(C); free(Cold);

        double *oldAn = (double *)malloc(sizeof(double) * ((size_t)nAn * (size_t)J + 1));
#pragma omp parallel for schedule(dynamic, 64)
        for (int i = 0; i < nAn; ++i) {
            int v = An[i];
            double *row = o->H[l] + (size_t)v * J;
            memcpy(oldAn + (size_t)i * J, row, sizeof(double) * (size_t)J);
            layer_row(&o->layer[l], Hp + (size_t)v * K, S + (size_t)v * K, 1.0, row);
        }
        set_list(o, l, An, nAn);
        free(A); free(oldA);
        A = An; nA = nAn; oldA = oldAn;
    }
#undef BEATS
    free(A); free(oldA); free(din_old); free(snap_of); free(need);
    return 0;
}

/* Hybrid-incremental propagation through attention layers (Sec. 3.4.1).  Every vertex caches the
 * numerator sum_u exp(z_uv) h_u and the denominator sum_u exp(z_uv) of its output.  A vertex that
 * was in the tree at hop l-1 (its own h^{l-1} changed, so every z_uv it is the sink of changed) is in
 * the tree at hop l too and recomputes both sums over all of its in-neighbours; any other hop-l vertex
 * takes <numerator, denominator> messages: exp(z_new) h_new - exp(z_old) h_old from a changed
 * in-neighbour, the whole new term along an added edge, minus the whole old term along a deleted one. */
static int apply_incremental_gat(oracle_t *o, const delta_t *dl, const float *feat_rows) {
    int L = o->L, d0 = o->d[0];
    int nA = dl->nF;
    int *A = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
    memcpy(A, dl->F, sizeof(int) * (size_t)nA);
    double *oldA = (double *)malloc(sizeof(double) * ((size_t)nA * (size_t)d0 + 1));
    for (int i = 0; i < nA; ++i) {
        double *row = o->H[0] + (size_t)A[i] * d0;
        memcpy(oldA + (size_t)i * d0, row, sizeof(double) * (size_t)d0);
        const float *src = dl->Frow[i] >= 0 ? feat_rows + (size_t)dl->Frow[i] * d0 : NULL;
        for (int k = 0; k < d0; ++k) row[k] = src ? (double)src[k] : 0.0;
    }
    set_list(o, 0, A, nA);
    unsigned char *recomputes = (unsigned char *)calloc((size_t)o->N, 1);

    for (int l = 1; l <= L; ++l) {
        const layer_t *ly = &o->layer[l];
        int K = o->d[l - 1];
        const double *Hp = o->H[l - 1];
        double *S = o->S[l], *Den = o->Den[l];
        int nAn; long walked;
        int *An = next_affected(o, dl, A, nA, A, nA, 1, &nAn, &walked);
        o->active_edges[l] = walked + dl->n_add + dl->n_del;
        for (int i = 0; i < nA; ++i) recomputes[A[i]] = 1;

        for (int i = 0; i < nA; ++i) {      /* changed in-neighbour, surviving edge */
            int u = A[i];
            const double *hnew = Hp + (size_t)u * K, *hold = oldA + (size_t)i * K;
            double s_new = gat_logit_part(ly, ly->ba, hnew), s_old = gat_logit_part(ly, ly->ba, hold);
            const ivec *r = &o->out[u];
            for (int j = 0; j < r->n; ++j) {
                int v = r->a[j];
                if (recomputes[v]) continue;
                pair_t p = { u, v, 0.f };
                if (dl->n_add && bsearch(&p, dl->add, (size_t)dl->n_add, sizeof(pair_t), cmp_pair)) continue;
                double tv = gat_logit_part(ly, ly->bb, Hp + (size_t)v * K);
                double e_new = exp(gat_logit(ly, s_new, tv)), e_old = exp(gat_logit(ly, s_old, tv));
                double *Sv = S + (size_t)v * K;
                for (int k = 0; k < K; ++k) Sv[k] += e_new * hnew[k] - e_old * hold[k];
                Den[v] += e_new - e_old;
            }
        }
        for (int i = 0; i < dl->n_add; ++i) {   /* added edge: the new term arrives */
            int u = dl->add[i].u, v = dl->add[i].v;
            if (recomputes[v]) continue;
            const double *hnew = Hp + (size_t)u * K;
            double e = exp(gat_logit(ly, gat_logit_part(ly, ly->ba, hnew), gat_logit_part(ly, ly->bb, Hp + (size_t)v * K)));
            double *Sv = S + (size_t)v * K;
            for (int k = 0; k < K; ++k) Sv[k] += e * hnew[k];
            Den[v] += e;
        }
        for (int i = 0; i < dl->n_del; ++i) {   /* deleted edge: the old term leaves */
            int u = dl->del[i].u, v = dl->del[i].v;
            if (recomputes[v]) continue;
            int ia = find_sorted(A, nA, u);
            const double *hold = ia >= 0 ? oldA + (size_t)ia * K : Hp + (size_t)u * K;
            double e = exp(gat_logit(ly, gat_logit_part(ly, ly->ba, hold), gat_logit_part(ly, ly->bb, Hp + (size_t)v * K)));
            double *Sv = S + (size_t)v * K;
            for (int k = 0; k < K; ++k) Sv[k] -= e * hold[k];
            Den[v] -= e;
        }
#pragma omp parallel for schedule(dynamic, 64)
        for (int i = 0; i < nA; ++i) {      /* in the tree one hop earlier: recompute */
            int v = A[i];
            gat_sums(o, l, v, Hp, NULL, NULL, S + (size_t)v * K, &Den[v]);
            recomputes[v] = 0;
        }
        double *oldAn = (double *)malloc(sizeof(double) * ((size_t)nAn * (size_t)K + 1));
        for (int i = 0; i < nAn; ++i) {
            int v = An[i];
            double *row = o->H[l] + (size_t)v * K;
            memcpy(oldAn + (size_t)i * K, row, sizeof(double) * (size_t)K);
            if (o->in[v].n == 0) { memset(S + (size_t)v * K, 0, sizeof(double) * (size_t)K); Den[v] = 0.0; }
            gat_output(ly, K, o->in[v].n, S + (size_t)v * K, Den[v], row);
        }
        set_list(o, l, An, nAn);
        free(A); free(oldA);
        A = An; nA = nAn; oldA = oldAn;
    }
    free(A); free(oldA); free(recomputes);
    return 0;
}

/* O-inc: incremental propagation of one batch (Sec. 3.3).  Returns 0, or <0 if the batch is
 * rejected (nothing changed).
 * pull = 0: every sender walks its out-list and adds its message to each sink's inbox, one thread
 *           (the order in which the paper states Send and Aggregate, Sec. 3.3.1).
 * pull = 1: the same messages, delivered the other way round: every hop-l vertex walks its in-list
 *           and sums the messages of the senders it finds there.  Summation is order-free
 *           (Sec. 3.3.3), every sink of a message is a hop-l vertex (A_l contains Out_new(C_{l-1})),
 *           and no two vertices write the same inbox row, so the sinks run in parallel without
 *           atomics.  Only the order of the additions differs from pull = 0. */
static int apply_incremental(oracle_t *o, const update_t *ups, int64_t n, const float *feat_rows,
                             int64_t n_rows, int pull) {
    delta_t dl;
    int rc = normalise(o, ups, n, n_rows, &dl);
    if (rc) return rc;
    int L = o->L, self_term = o->layer[1].kind != KIND_GRAPHCONV;

    if (MONOTONIC(o->agg)) {
        if (o->layer[1].kind >= KIND_GIN) { delta_free(&dl); return -3; }   /* GraphConv and SAGE layers only */
        apply_topology(o, &dl);
        rc = apply_incremental_max(o, &dl, feat_rows);
        delta_free(&dl);
        return rc;
    }
    if (o->layer[1].kind == KIND_GAT) {
        apply_topology(o, &dl);
        rc = apply_incremental_gat(o, &dl, feat_rows);
        delta_free(&dl);
        return rc;
    }
    apply_topology(o, &dl);
    /* old source coefficients of the endpoints whose out-degree changed */
    int nsrc; srcinfo_t *srcs = source_table(o, &dl, &nsrc);

    /* hop 0: feature replacements; keep the old rows for the messages (Sec. 3.3.3, first case) */
    int d0 = o->d[0];
    int nA = dl.nF;
    int *A = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
    memcpy(A, dl.F, sizeof(int) * (size_t)nA);
    double *oldA = (double *)malloc(sizeof(double) * ((size_t)nA * (size_t)d0 + 1));
    for (int i = 0; i < nA; ++i) {
        double *row = o->H[0] + (size_t)A[i] * d0;
        memcpy(oldA + (size_t)i * d0, row, sizeof(double) * (size_t)d0);
        const float *src = dl.Frow[i] >= 0 ? feat_rows + (size_t)dl.Frow[i] * d0 : NULL;   /* deleted vertex: zeros */
        for (int k = 0; k < d0; ++k) row[k] = src ? (double)src[k] : 0.0;
    }
    set_list(o, 0, A, nA);
    int nC; int *C = changed_senders(o, &dl, A, nA, &nC);
    int *sender_pos = NULL;   /* pull form: vertex -> index of its message, or -1 */
    if (pull) {
        sender_pos = (int *)malloc(sizeof(int) * (size_t)o->N);
        for (int v = 0; v < o->N; ++v) sender_pos[v] = -1;
    }

    for (int l = 1; l <= L; ++l) { /* one BSP superstep per hop (Sec. 3.3.1) */
        int K = o->d[l - 1], J = o->d[l];
        const double *Hp = o->H[l - 1];
        double *S = o->S[l];
        double *m = (double *)malloc(sizeof(double) * (size_t)K * (size_t)(pull ? nC + 1 : 1));
        int nAn; long walked;
        int *An = next_affected(o, &dl, C, nC, A, nA, self_term, &nAn, &walked);
        o->active_edges[l] = walked + dl.n_add + dl.n_del;

        /* Prepare + Send + Aggregate: surviving edges of changed senders carry
         * c_new h_new - c_old h_old (Sec. 3.3.3 first case; weighted form: "other linear
         * aggregators"); messages are summed into the sink's inbox in any order. */
        for (int i = 0; i < nC; ++i) {
            int u = C[i];
            int ia = find_sorted(A, nA, u);
            const double *hnew = Hp + (size_t)u * K;
            const double *hold = ia >= 0 ? oldA + (size_t)ia * K : hnew;
            double cnew = coef_src(o, o->out[u].n), cold = cnew;
            int has_add = 0;
            const srcinfo_t *si = source_find(srcs, nsrc, u);
            if (si) { cold = si->c_old; has_add = si->n_add > 0; }
            double *mu = pull ? m + (size_t)i * K : m;
            for (int k = 0; k < K; ++k) mu[k] = cnew * hnew[k] - cold * hold[k];
            if (pull) { sender_pos[u] = i; continue; }
            const ivec *r = &o->out[u];
            for (int j = 0; j < r->n; ++j) {
                int v = r->a[j];
                if (has_add) { pair_t p = { u, v, 0.f }; if (bsearch(&p, dl.add, (size_t)dl.n_add, sizeof(pair_t), cmp_pair)) continue; }
                double *Sv = S + (size_t)v * K;
                double a = o->weighted ? (double)r->w[j] : 1.0;   /* the edge's weight scales the message (Sec. 3.3.3) */
                for (int k = 0; k < K; ++k) Sv[k] += a * m[k];
            }
        }
        if (pull) {
#pragma omp parallel for schedule(dynamic, 64)
            for (int i = 0; i < nAn; ++i) {
                int v = An[i];
                double *Sv = S + (size_t)v * K;
                const ivec *r = &o->in[v];
                for (int j = 0; j < r->n; ++j) {
                    int u = r->a[j], p = sender_pos[u];
                    if (p < 0) continue;
                    /* an edge added by this batch carries no delta message */
                    if (dl.n_add) { pair_t e = { u, v, 0.f }; if (bsearch(&e, dl.add, (size_t)dl.n_add, sizeof(pair_t), cmp_pair)) continue; }
                    const double *mu = m + (size_t)p * K;
                    double a = o->weighted ? (double)r->w[j] : 1.0;
                    for (int k = 0; k < K; ++k) Sv[k] += a * mu[k];
                }
            }
            for (int i = 0; i < nC; ++i) sender_pos[C[i]] = -1;
        }
        /* added edge: the old contribution is taken as 0, so the whole new term arrives */
        for (int i = 0; i < dl.n_add; ++i) {
            int u = dl.add[i].u;
            double cnew = coef_src(o, o->out[u].n) * (o->weighted ? (double)dl.add[i].w : 1.0);
            const double *hnew = Hp + (size_t)u * K;
            double *Sv = S + (size_t)dl.add[i].v * K;
            for (int k = 0; k < K; ++k) Sv[k] += cnew * hnew[k];
        }
        /* deleted edge: the new contribution is taken as 0, so the whole old term leaves */
        for (int i = 0; i < dl.n_del; ++i) {
            int u = dl.del[i].u;
            int ia = find_sorted(A, nA, u);
            const double *hold = ia >= 0 ? oldA + (size_t)ia * K : Hp + (size_t)u * K;
            double cold = source_find(srcs, nsrc, u)->c_old * (o->weighted ? (double)dl.del[i].w : 1.0);
            double *Sv = S + (size_t)dl.del[i].v * K;
            for (int k = 0; k < K; ++k) Sv[k] -= cold * hold[k];
        }
        free(m);

        /* Compute: re-apply Update and the activation to the hop-l vertices, keeping old rows */
        double *oldAn = (double *)malloc(sizeof(double) * ((size_t)nAn * (size_t)J + 1));
#pragma omp parallel for schedule(dynamic, 64)
        for (int i = 0; i < nAn; ++i) {
            int v = An[i];
            double *row = o->H[l] + (size_t)v * J;
            memcpy(oldAn + (size_t)i * J, row, sizeof(double) * (size_t)J);
            layer_row(&o->layer[l], Hp + (size_t)v * K, S + (size_t)v * K, norm_sink(o, o->in[v].n), row);
        }
        set_list(o, l, An, nAn);
        free(A); free(oldA); free(C);
        A = An; nA = nAn; oldA = oldAn;
        C = changed_senders(o, &dl, A, nA, &nC);
    }
    free(A); free(oldA); free(C); free(srcs); free(sender_pos);
    delta_free(&dl);
    return 0;
}

int orc_apply_incremental(oracle_t *o, const update_t *ups, int64_t n, const float *feat_rows,
                          int64_t n_rows) {
    return apply_incremental(o, ups, n, feat_rows, n_rows, 0);
}

/* The incremental algorithm with Send + Aggregate in pull form on all host cores (see apply_incremental). */
int orc_apply_incremental_pull(oracle_t *o, const update_t *ups, int64_t n, const float *feat_rows,
                               int64_t n_rows) {
    return apply_incremental(o, ups, n, feat_rows, n_rows, 1);
}

/* O-rc: layer-wise recompute scoped to the affected sets (Sec. 3.2): every affected vertex pulls
 * all of its current in-neighbours; rows outside A_l are left untouched. */
int orc_apply_scoped(oracle_t *o, const update_t *ups, int64_t n, const float *feat_rows,
                     int64_t n_rows) {
    delta_t dl;
    int rc = normalise(o, ups, n, n_rows, &dl);
    if (rc) return rc;
    int L = o->L, self_term = o->layer[1].kind != KIND_GRAPHCONV;
    apply_topology(o, &dl);
    int d0 = o->d[0];
    int nA = dl.nF;
    int *A = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
    memcpy(A, dl.F, sizeof(int) * (size_t)nA);
    for (int i = 0; i < nA; ++i) {
        double *row = o->H[0] + (size_t)A[i] * d0;
        const float *src = dl.Frow[i] >= 0 ? feat_rows + (size_t)dl.Frow[i] * d0 : NULL;   /* deleted vertex: zeros */
        for (int k = 0; k < d0; ++k) row[k] = src ? (double)src[k] : 0.0;
    }
    set_list(o, 0, A, nA);
    int nC; int *C = changed_senders(o, &dl, A, nA, &nC);
    for (int l = 1; l <= L; ++l) {
        int K = o->d[l - 1], J = o->d[l];
        int nAn; long walked;
        int *An = next_affected(o, &dl, C, nC, A, nA, self_term, &nAn, &walked);
        o->active_edges[l] = walked + dl.n_add + dl.n_del;
#pragma omp parallel for schedule(dynamic, 64)
        for (int i = 0; i < nAn; ++i) {
            int v = An[i];
            if (o->layer[l].kind == KIND_GAT) {
                gat_sums(o, l, v, o->H[l - 1], NULL, NULL, o->S[l] + (size_t)v * K, &o->Den[l][v]);
                gat_row_definition(o, l, v, o->H[l - 1], NULL, NULL, o->H[l] + (size_t)v * J);
                continue;
            }
            aggregate_row(o, v, o->H[l - 1], K, o->S[l] + (size_t)v * K);
            layer_row(&o->layer[l], o->H[l - 1] + (size_t)v * K, o->S[l] + (size_t)v * K,
                      norm_sink(o, o->in[v].n), o->H[l] + (size_t)v * J);
        }
        set_list(o, l, An, nAn);
        free(A); free(C);
        A = An; nA = nAn;
        C = changed_senders(o, &dl, A, nA, &nC);
    }
    free(A); free(C);
    delta_free(&dl);
    return 0;
}

/* Graph state and affected sets only: Apply (Sec. 3.3) and the hops of the propagation tree, with
 * no embedding arithmetic.  The cached H / S are NOT maintained by this call; it exists so that a
 * test can follow the structure of a large graph batch by batch and check single rows against
 * the definition with orc_row_from_prev. */
int orc_apply_structure(oracle_t *o, const update_t *ups, int64_t n, int64_t n_rows) {
    delta_t dl;
    int rc = normalise(o, ups, n, n_rows, &dl);
    if (rc) return rc;
    int L = o->L, self_term = o->layer[1].kind != KIND_GRAPHCONV;
    apply_topology(o, &dl);
    int nA = dl.nF;
    int *A = (int *)malloc(sizeof(int) * (size_t)(nA + 1));
    memcpy(A, dl.F, sizeof(int) * (size_t)nA);
    set_list(o, 0, A, nA);
    int nC; int *C = changed_senders(o, &dl, A, nA, &nC);
    for (int l = 1; l <= L; ++l) {
        int nAn; long walked;
        int *An = next_affected(o, &dl, C, nC, A, nA, self_term, &nAn, &walked);
        o->active_edges[l] = walked + dl.n_add + dl.n_del;
        set_list(o, l, An, nAn);
        free(A); free(C);
        A = An; nA = nAn;
        C = changed_senders(o, &dl, A, nA, &nC);
    }
    free(A); free(C);
    delta_free(&dl);
    return 0;
}

/* One row of one layer from a caller-supplied previous-layer matrix (fp32, leading dimension
 * ld) over the oracle's current graph: h^l_v by Eq. 1-2.  Lets a test check any single row of a
 * large state against the definition without recomputing the whole graph. */
void orc_row_from_prev(const oracle_t *o, int l, int v, const float *Hprev, int64_t ld,
                       double *S_out, double *h_out) {
    int K = o->d[l - 1];
    const ivec *in = &o->in[v];
    if (o->layer[l].kind == KIND_GAT) {   /* Eq. 3 over the widened rows of v and its in-neighbours; S_out: numerator sum */
        const layer_t *ly = &o->layer[l];
        double *rows = (double *)malloc(sizeof(double) * (size_t)K * (size_t)(in->n + 1));
        double *z = (double *)malloc(sizeof(double) * (size_t)(in->n + 1));
        for (int k = 0; k < K; ++k) { rows[k] = (double)Hprev[(size_t)v * (size_t)ld + k]; S_out[k] = 0.0; h_out[k] = 0.0; }
        double tv = gat_logit_part(ly, ly->bb, rows), zmax = -1e300, den = 0.0;
        for (int i = 0; i < in->n; ++i) {
            double *r = rows + (size_t)(i + 1) * K;
            for (int k = 0; k < K; ++k) r[k] = (double)Hprev[(size_t)in->a[i] * (size_t)ld + k];
            z[i] = gat_logit(ly, gat_logit_part(ly, ly->ba, r), tv);
            if (z[i] > zmax) zmax = z[i];
        }
        for (int i = 0; i < in->n; ++i) den += exp(z[i] - zmax);
        for (int i = 0; i < in->n; ++i) {
            const double *r = rows + (size_t)(i + 1) * K;
            for (int k = 0; k < K; ++k) { S_out[k] += exp(z[i]) * r[k]; h_out[k] += exp(z[i] - zmax) / den * r[k]; }
        }
        if (ly->act == ACT_RELU) for (int k = 0; k < K; ++k) h_out[k] = h_out[k] > 0.0 ? h_out[k] : 0.0;
        free(rows); free(z);
        return;
    }
    double *hp = (double *)malloc(sizeof(double) * (size_t)K);
    for (int k = 0; k < K; ++k) { S_out[k] = 0.0; hp[k] = (double)Hprev[(size_t)v * (size_t)ld + k]; }
    for (int i = 0; i < in->n; ++i) {
        int u = in->a[i];
        double c = in_edge_coef(o, v, i);
        const float *h = Hprev + (size_t)u * (size_t)ld;
        for (int k = 0; k < K; ++k) S_out[k] += c * (double)h[k];
    }
    layer_row(&o->layer[l], hp, S_out, norm_sink(o, in->n), h_out);
    free(hp);
}

/* The same for many rows at once (ids[0..n)), one row per thread at a time: S_out is n x d[l-1],
 * h_out n x d[l]. */
void orc_rows_from_prev(const oracle_t *o, int l, const int32_t *ids, int64_t n, const float *Hprev,
                        int64_t ld, double *S_out, double *h_out) {
    int K = o->d[l - 1], J = o->d[l];
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t i = 0; i < n; ++i)
        orc_row_from_prev(o, l, ids[i], Hprev, ld, S_out + (size_t)i * K, h_out + (size_t)i * J);
}

/* ------------------------------------------------------------------------------------------ */
/* threads the parallel loops (full inference, the compute step) run on */
int orc_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
double *orc_H(oracle_t *o, int l) { return o->H[l]; }
double *orc_S(oracle_t *o, int l) { return o->S[l]; }
double *orc_Den(oracle_t *o, int l) { return o->Den[l]; }
double *orc_full_H(oracle_t *o, int l) { return l == 0 ? o->H[0] : o->FH[l]; }
double *orc_full_S(oracle_t *o, int l) { return o->FS[l]; }
const int *orc_affected(oracle_t *o, int l, int *n) { *n = o->nA[l]; return o->A[l]; }
long orc_active_edges(oracle_t *o, int l) { return o->active_edges[l]; }
void orc_counts(oracle_t *o, long *out5) {
    out5[0] = o->n_added; out5[1] = o->n_deleted; out5[2] = o->noop_add; out5[3] = o->noop_del;
    out5[4] = o->superseded;
}
int64_t orc_num_edges(oracle_t *o) {
    int64_t e = 0;
    for (int v = 0; v < o->N; ++v) e += o->out[v].n;
    return e;
}
void orc_degrees(oracle_t *o, int32_t *deg_out, int32_t *deg_in) {
    for (int v = 0; v < o->N; ++v) { deg_out[v] = o->out[v].n; deg_in[v] = o->in[v].n; }
}
void orc_set_batch_weights(oracle_t *o, const float *op_w) { o->op_w = op_w; }

/* the stored weight of every edge, in the order of orc_export_csr's col */
void orc_export_weights(oracle_t *o, float *w) {
    int64_t p = 0;
    for (int v = 0; v < o->N; ++v)
        for (int j = 0; j < o->out[v].n; ++j) w[p++] = o->weighted ? o->out[v].w[j] : 1.0f;
}

/* canonical CSR of the out-lists: rowptr[N+1], col sorted within each row */
void orc_export_csr(oracle_t *o, int64_t *rowptr, int32_t *col) {
    int64_t p = 0;
    for (int v = 0; v < o->N; ++v) {
        rowptr[v] = p;
        for (int j = 0; j < o->out[v].n; ++j) col[p++] = o->out[v].a[j];
    }
    rowptr[o->N] = p;
}
