/*
 * CPU oracle for HAG aggregation -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Plain, slow, single-threaded C.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library never does and
 * shares no code with it.
 *
 * What each function follows in the paper (arxiv 1906.03707):
 *   o1_direct_forward   Algorithm 1 line 4 with the GCN row of Table 1:
 *                       a_v = sum over u in N(v) of h_u   (mode 1, mean: divided by |N(v)|;
 *                       mode 2: the argument of GCN's Update, (a_v + h_v) / (|N(v)| + 1))
 *   o2_direct_backward  equivalence clause (2) of Section 3.2 ("the same
 *                       gradients"): gx_u = sum over v with u in N(v) of s_v g_v
 *   o4_hag_forward      Algorithm 2 lines 3-8, evaluated over a given HAG
 *   o4_hag_backward     the adjoint of Algorithm 2 over the transposed HAG
 *   o3b_greedy          Algorithm 3, set-Aggregate branch, with the pair-count
 *                       heap the complexity appendix sketches
 *   o3c_greedy          the same algorithm without a count per pair (memory O(|E|)):
 *                       per-node upper bounds confirmed by recounts from the definition
 *   o_count_pair / o_max_pair_recount   the Redundancy function of Algorithm 3
 *                       evaluated from its definition
 *   o6_max_forward(_rows) / o6_max_backward    the element-wise max Aggregate of the GraphSAGE-P
 *                       row of Table 1, a_v = max over u in N(v) of z_u, straight
 *                       from the definition, and its gradient
 *   o7_hag_max_forward / o7_hag_max_backward   Algorithm 2 with max as the (associative,
 *                       commutative: Section 3.1, set Aggregate) operator, and its
 *                       gradient over the transposed HAG
 *
 * All floating point is fp64.  Graph layout: CSR of in-neighbours, row v lists
 * the sources u of v, int64 row pointers, int32 sorted duplicate-free columns.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

/* ------------------------------------------------------------------------- */
/* O1: direct forward.  rows == NULL: all n rows, out is n x d.  Otherwise out
 * is n_rows x d, row i holding the result for node rows[i].  abs_out (may be
 * NULL) receives sum |x_u| (mean: divided by |N(v)|), the tolerance scale.   */
void o1_direct_forward(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t d,
                       const double *x, int mean, const int64_t *rows, int64_t n_rows,
                       double *out, double *abs_out)
{
    int64_t count = rows ? n_rows : n;
    for (int64_t i = 0; i < count; ++i) {
        int64_t v = rows ? rows[i] : i;
        double *o = out + i * d;
        double *ao = abs_out ? abs_out + i * d : NULL;
        for (int64_t k = 0; k < d; ++k) o[k] = 0.0;
        if (ao) for (int64_t k = 0; k < d; ++k) ao[k] = 0.0;
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            const double *xu = x + (int64_t)col[e] * d;
            for (int64_t k = 0; k < d; ++k) o[k] += xu[k];
            if (ao) for (int64_t k = 0; k < d; ++k) ao[k] += fabs(xu[k]);
        }
        int64_t deg = row_ptr[v + 1] - row_ptr[v];
        if (mean == 1 && deg > 0) {
            for (int64_t k = 0; k < d; ++k) o[k] /= (double)deg;
            if (ao) for (int64_t k = 0; k < d; ++k) ao[k] /= (double)deg;
        }
        if (mean == 2) {                 /* Table 1, GCN: (a_v + h_v) / (|N(v)| + 1) */
            const double *xv = x + v * d;
            for (int64_t k = 0; k < d; ++k) o[k] = (o[k] + xv[k]) / (double)(deg + 1);
            if (ao) for (int64_t k = 0; k < d; ++k) ao[k] = (ao[k] + fabs(xv[k])) / (double)(deg + 1);
        }
    }
}

/* O2: direct backward.  slot == NULL: gx is n x d and every source row is
 * produced.  Otherwise slot[u] is -1 (skip) or the row of gx that receives
 * node u's gradient (gx then has as many rows as there are slots).          */
void o2_direct_backward(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t d,
                        const double *g, int mean, const int64_t *slot, int64_t n_slots,
                        double *gx, double *abs_gx)
{
    int64_t out_rows = slot ? n_slots : n;
    memset(gx, 0, sizeof(double) * (size_t)(out_rows * d));
    if (abs_gx) memset(abs_gx, 0, sizeof(double) * (size_t)(out_rows * d));
    for (int64_t v = 0; v < n; ++v) {
        int64_t deg = row_ptr[v + 1] - row_ptr[v];
        double s = (mean == 1 && deg > 0) ? 1.0 / (double)deg : 1.0;
        if (mean == 2) s = 1.0 / (double)(deg + 1);
        const double *gv = g + v * d;
        if (mean == 2) {                 /* the h_v term of (a_v + h_v) / (|N(v)| + 1) sends s_v g_v back to v itself */
            int64_t r = slot ? slot[v] : v;
            if (r >= 0) {
                double *o = gx + r * d;
                for (int64_t k = 0; k < d; ++k) o[k] += s * gv[k];
                if (abs_gx) { double *ao = abs_gx + r * d; for (int64_t k = 0; k < d; ++k) ao[k] += fabs(s * gv[k]); }
            }
        }
        for (int64_t e = row_ptr[v]; e < row_ptr[v + 1]; ++e) {
            int64_t u = col[e];
            int64_t r = slot ? slot[u] : u;
            if (r < 0) continue;
            double *o = gx + r * d;
            for (int64_t k = 0; k < d; ++k) o[k] += s * gv[k];
            if (abs_gx) {
                double *ao = abs_gx + r * d;
                for (int64_t k = 0; k < d; ++k) ao[k] += fabs(s * gv[k]);
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* O4: Algorithm 2 over a HAG in canonical layout.
 *   ids 0..n-1 graph nodes, n..n+num_agg-1 aggregation nodes in an order in
 *   which every aggregation node comes after both of its inputs;
 *   agg_in[2j], agg_in[2j+1]: the two inputs of aggregation node n+j;
 *   res_ptr/res_idx: the remaining in-neighbours of every graph node;
 *   in_degree[v] = |N(v)| in the input graph (mean divides by it).
 * scratch: (n + num_agg) x d doubles, the a-hat buffer of Algorithm 2.        */
void o4_hag_forward(int64_t n, int64_t num_agg, const int32_t *agg_in,
                    const int64_t *res_ptr, const int32_t *res_idx, const int32_t *in_degree,
                    int64_t d, const double *x, int mean, double *scratch, double *out)
{
    double *ahat = scratch;
    memcpy(ahat, x, sizeof(double) * (size_t)(n * d));                 /* lines 3-4 */
    for (int64_t j = 0; j < num_agg; ++j) {                            /* lines 5-6 */
        const double *p = ahat + (int64_t)agg_in[2 * j] * d;
        const double *q = ahat + (int64_t)agg_in[2 * j + 1] * d;
        double *w = ahat + (n + j) * d;
        for (int64_t k = 0; k < d; ++k) w[k] = p[k] + q[k];
    }
    for (int64_t v = 0; v < n; ++v) {                                  /* lines 7-8 */
        double *o = out + v * d;
        for (int64_t k = 0; k < d; ++k) o[k] = 0.0;
        for (int64_t e = res_ptr[v]; e < res_ptr[v + 1]; ++e) {
            const double *a = ahat + (int64_t)res_idx[e] * d;
            for (int64_t k = 0; k < d; ++k) o[k] += a[k];
        }
        if (mean && in_degree[v] > 0)
            for (int64_t k = 0; k < d; ++k) o[k] /= (double)in_degree[v];
    }
}

/* Adjoint of the above over the transposed HAG: t_ptr has n+num_agg+1
 * entries, row s lists the destinations of source s; a destination < n is the
 * OUTPUT row of that graph node, a destination >= n an aggregation node.
 * Aggregation nodes are visited in reverse canonical order, then the graph
 * nodes as sources.  scratch: num_agg x d doubles.                           */
void o4_hag_backward(int64_t n, int64_t num_agg, const int64_t *t_ptr, const int32_t *t_idx,
                     const int32_t *in_degree, int64_t d, const double *g, int mean,
                     double *scratch, double *gx)
{
    double *ghat = scratch;
    for (int64_t s = n + num_agg - 1; s >= 0; --s) {
        double *o = (s >= n) ? ghat + (s - n) * d : gx + s * d;
        for (int64_t k = 0; k < d; ++k) o[k] = 0.0;
        for (int64_t e = t_ptr[s]; e < t_ptr[s + 1]; ++e) {
            int64_t dst = t_idx[e];
            if (dst < n) {
                double sc = (mean && in_degree[dst] > 0) ? 1.0 / (double)in_degree[dst] : 1.0;
                const double *gv = g + dst * d;
                for (int64_t k = 0; k < d; ++k) o[k] += sc * gv[k];
            } else {
                const double *gh = ghat + (dst - n) * d;
                for (int64_t k = 0; k < d; ++k) o[k] += gh[k];
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* O6: element-wise max aggregation (Table 1, GraphSAGE-P) from the definition.
 * An empty neighbourhood gives a zero row (the reading used for sum as well).  */
void o6_max_forward(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t d,
                    const double *z, double *out)
{
    for (int64_t v = 0; v < n; ++v) {
        double *o = out + v * d;
        int64_t b = row_ptr[v], e = row_ptr[v + 1];
        if (e == b) { for (int64_t k = 0; k < d; ++k) o[k] = 0.0; continue; }
        const double *z0 = z + (int64_t)col[b] * d;
        for (int64_t k = 0; k < d; ++k) o[k] = z0[k];
        for (int64_t i = b + 1; i < e; ++i) {
            const double *zu = z + (int64_t)col[i] * d;
            for (int64_t k = 0; k < d; ++k) if (zu[k] > o[k]) o[k] = zu[k];
        }
    }
}

/* The same for a subset of the nodes: out is n_rows x d, row i holding a_v for v = rows[i]. */
void o6_max_forward_rows(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t d,
                         const double *z, const int64_t *rows, int64_t n_rows, double *out)
{
    (void)n;
    for (int64_t r = 0; r < n_rows; ++r) {
        int64_t v = rows[r];
        double *o = out + r * d;
        int64_t b = row_ptr[v], e = row_ptr[v + 1];
        if (e == b) { for (int64_t k = 0; k < d; ++k) o[k] = 0.0; continue; }
        const double *z0 = z + (int64_t)col[b] * d;
        for (int64_t k = 0; k < d; ++k) o[k] = z0[k];
        for (int64_t i = b + 1; i < e; ++i) {
            const double *zu = z + (int64_t)col[i] * d;
            for (int64_t k = 0; k < d; ++k) if (zu[k] > o[k]) o[k] = zu[k];
        }
    }
}

/* Gradient of the above for L = sum_v <g_v, a_v>: component k of g_v goes to the
 * in-neighbours u of v that attain the maximum, z_u[k] == a_v[k].  Reading (the
 * paper does not say what happens on ties): every such u receives it.  a is
 * the forward result.  abs_gz receives the same sums over |g|.               */
void o6_max_backward(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t d,
                     const double *z, const double *a, const double *g, double *gz, double *abs_gz)
{
    memset(gz, 0, sizeof(double) * (size_t)(n * d));
    memset(abs_gz, 0, sizeof(double) * (size_t)(n * d));
    for (int64_t v = 0; v < n; ++v) {
        const double *av = a + v * d, *gv = g + v * d;
        for (int64_t i = row_ptr[v]; i < row_ptr[v + 1]; ++i) {
            int64_t u = col[i];
            const double *zu = z + u * d;
            for (int64_t k = 0; k < d; ++k)
                if (zu[k] == av[k]) { gz[u * d + k] += gv[k]; abs_gz[u * d + k] += fabs(gv[k]); }
        }
    }
}

/* O7: Algorithm 2 with max.  Layout as for o4_hag_forward.  ahat: (n + num_agg) x d
 * doubles; on return rows n.. hold the maxima of the aggregation nodes (the
 * backward pass needs them).                                                  */
void o7_hag_max_forward(int64_t n, int64_t num_agg, const int32_t *agg_in,
                        const int64_t *res_ptr, const int32_t *res_idx,
                        int64_t d, const double *z, double *ahat, double *out)
{
    memcpy(ahat, z, sizeof(double) * (size_t)(n * d));                 /* lines 3-4 */
    for (int64_t j = 0; j < num_agg; ++j) {                            /* lines 5-6 */
        const double *p = ahat + (int64_t)agg_in[2 * j] * d;
        const double *q = ahat + (int64_t)agg_in[2 * j + 1] * d;
        double *w = ahat + (n + j) * d;
        for (int64_t k = 0; k < d; ++k) w[k] = p[k] > q[k] ? p[k] : q[k];
    }
    for (int64_t v = 0; v < n; ++v) {                                  /* lines 7-8 */
        double *o = out + v * d;
        int64_t b = res_ptr[v], e = res_ptr[v + 1];
        if (e == b) { for (int64_t k = 0; k < d; ++k) o[k] = 0.0; continue; }
        const double *a0 = ahat + (int64_t)res_idx[b] * d;
        for (int64_t k = 0; k < d; ++k) o[k] = a0[k];
        for (int64_t i = b + 1; i < e; ++i) {
            const double *a = ahat + (int64_t)res_idx[i] * d;
            for (int64_t k = 0; k < d; ++k) if (a[k] > o[k]) o[k] = a[k];
        }
    }
}

/* Gradient over the transposed HAG (layout as for o4_hag_backward): a source s
 * (graph node or aggregation node) receives component k from a destination t
 * when its value equals the destination's maximum.  Values: ahat for sources and
 * aggregation-node destinations, the forward output a for graph-node
 * destinations.  ghat: num_agg x d doubles.                                  */
void o7_hag_max_backward(int64_t n, int64_t num_agg, const int64_t *t_ptr, const int32_t *t_idx,
                         int64_t d, const double *ahat, const double *a, const double *g,
                         double *ghat, double *gz)
{
    for (int64_t s = n + num_agg - 1; s >= 0; --s) {
        double *o = (s >= n) ? ghat + (s - n) * d : gz + s * d;
        const double *val = ahat + s * d;
        for (int64_t k = 0; k < d; ++k) o[k] = 0.0;
        for (int64_t e = t_ptr[s]; e < t_ptr[s + 1]; ++e) {
            int64_t t = t_idx[e];
            const double *tv = (t < n) ? a + t * d : ahat + t * d;
            const double *tg = (t < n) ? g + t * d : ghat + (t - n) * d;
            for (int64_t k = 0; k < d; ++k) if (val[k] == tv[k]) o[k] += tg[k];
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Redundancy(v1, v2) from its definition: the number of graph-node rows of the
 * current edge set that contain both.  cur_ptr/cur_len/cur_idx: row u occupies
 * cur_idx[cur_ptr[u] .. cur_ptr[u]+cur_len[u]), sorted.                       */
static int row_has(const int32_t *row, int32_t len, int32_t key)
{
    int32_t lo = 0, hi = len;
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if (row[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo < len && row[lo] == key;
}

int64_t o_count_pair(int64_t n, const int64_t *cur_ptr, const int32_t *cur_len, const int32_t *cur_idx,
                     int32_t v1, int32_t v2)
{
    int64_t r = 0;
    for (int64_t u = 0; u < n; ++u) {
        const int32_t *row = cur_idx + cur_ptr[u];
        if (row_has(row, cur_len[u], v1) && row_has(row, cur_len[u], v2)) ++r;
    }
    return r;
}

/* Full recount for one node a: over every row that holds a, count every other
 * member; returns the largest count, *best_partner = the smallest id attaining
 * it.  counts: zeroed scratch of n_ids int32, left zeroed on return.          */
int64_t o_max_pair_recount(int64_t n, const int64_t *cur_ptr, const int32_t *cur_len, const int32_t *cur_idx,
                           int64_t n_ids, int32_t a, int32_t *counts, int32_t *best_partner)
{
    int64_t best = 0;
    int32_t arg = -1;
    for (int64_t u = 0; u < n; ++u) {
        const int32_t *row = cur_idx + cur_ptr[u];
        if (!row_has(row, cur_len[u], a)) continue;
        for (int32_t i = 0; i < cur_len[u]; ++i) if (row[i] != a) counts[row[i]]++;
    }
    for (int64_t y = 0; y < n_ids; ++y) {
        if (counts[y] > best) { best = counts[y]; arg = (int32_t)y; }
    }
    for (int64_t u = 0; u < n; ++u) {
        const int32_t *row = cur_idx + cur_ptr[u];
        if (!row_has(row, cur_len[u], a)) continue;
        for (int32_t i = 0; i < cur_len[u]; ++i) counts[row[i]] = 0;
    }
    *best_partner = arg;
    return best;
}

/* ------------------------------------------------------------------------- */
/* O3b: Algorithm 3 (set Aggregate) with an explicit map pair -> redundancy and
 * a max-heap over (redundancy, pair), as the complexity appendix describes.
 * The heap is lazy: an entry is valid only while the map still shows its
 * count; counts of existing pairs only ever fall and a new pair gets its
 * count once, so every live (pair, count >= 2) has exactly one valid entry.
 * Tie-break: highest redundancy, then the smallest v1, then the smallest v2
 * (v1 < v2, aggregation nodes numbered n, n+1, ... in creation order).       */

typedef struct { uint64_t *keys; int32_t *vals; uint64_t mask; uint64_t used; } pairmap;
#define PM_EMPTY UINT64_MAX

static uint64_t pm_hash(uint64_t k) {
    k ^= k >> 33; k *= 0xff51afd7ed558ccdULL; k ^= k >> 33; k *= 0xc4ceb9fe1a85ec53ULL; k ^= k >> 33;
    return k;
}
static int pm_init(pairmap *m, uint64_t cap_pow2) {
    m->keys = (uint64_t *)malloc(sizeof(uint64_t) * cap_pow2);
    m->vals = (int32_t *)malloc(sizeof(int32_t) * cap_pow2);
    if (!m->keys || !m->vals) return -1;
    memset(m->keys, 0xff, sizeof(uint64_t) * cap_pow2);
    m->mask = cap_pow2 - 1; m->used = 0;
    return 0;
}
static void pm_free(pairmap *m) { free(m->keys); free(m->vals); }
static int32_t *pm_slot(pairmap *m, uint64_t key);
static int pm_grow(pairmap *m) {
    pairmap bigger;
    if (pm_init(&bigger, (m->mask + 1) * 2)) return -1;
    for (uint64_t i = 0; i <= m->mask; ++i)
        if (m->keys[i] != PM_EMPTY) *pm_slot(&bigger, m->keys[i]) = m->vals[i];
    pm_free(m);
    *m = bigger;
    return 0;
}
/* pointer to the count of `key`, inserted with 0 if absent (NULL: out of memory) */
static int32_t *pm_slot(pairmap *m, uint64_t key) {
    if ((m->used + 1) * 10 > (m->mask + 1) * 6) { if (pm_grow(m)) return NULL; }
    uint64_t i = pm_hash(key) & m->mask;
    while (m->keys[i] != PM_EMPTY && m->keys[i] != key) i = (i + 1) & m->mask;
    if (m->keys[i] == PM_EMPTY) { m->keys[i] = key; m->vals[i] = 0; m->used++; }
    return &m->vals[i];
}
static uint64_t pair_key(int32_t a, int32_t b) {
    if (a > b) { int32_t t = a; a = b; b = t; }
    return ((uint64_t)(uint32_t)a << 32) | (uint32_t)b;
}

typedef struct { int32_t cnt, a, b; } hent;
/* 1 if x must come out of the heap before y */
static int h_before(const hent *x, const hent *y) {
    if (x->cnt != y->cnt) return x->cnt > y->cnt;
    if (x->a != y->a) return x->a < y->a;
    return x->b < y->b;
}
typedef struct { hent *e; int64_t n, cap; } heap;
static int h_push(heap *h, hent v) {
    if (h->n == h->cap) {
        int64_t nc = h->cap ? h->cap * 2 : 1024;
        hent *ne = (hent *)realloc(h->e, sizeof(hent) * (size_t)nc);
        if (!ne) return -1;
        h->e = ne; h->cap = nc;
    }
    int64_t i = h->n++;
    while (i > 0) {
        int64_t p = (i - 1) / 2;
        if (!h_before(&v, &h->e[p])) break;
        h->e[i] = h->e[p]; i = p;
    }
    h->e[i] = v;
    return 0;
}
static hent h_pop(heap *h) {
    hent top = h->e[0];
    hent last = h->e[--h->n];
    int64_t i = 0;
    for (;;) {
        int64_t l = 2 * i + 1, r = l + 1, c;
        if (l >= h->n) break;
        c = (r < h->n && h_before(&h->e[r], &h->e[l])) ? r : l;
        if (!h_before(&h->e[c], &last)) break;
        h->e[i] = h->e[c]; i = c;
    }
    if (h->n > 0) h->e[i] = last;
    return top;
}

typedef struct { int32_t *v; int32_t len; } ilist;

/* Returns the number of aggregation nodes created (<= capacity), or a negative
 * number when memory runs out.
 *   trace_v1/v2/r: capacity entries each, the merged pair (creation ids,
 *                  v1 < v2) and its redundancy, in creation order;
 *   cur_len[n], cur_idx[E]: on return row u's remaining in-neighbours (creation
 *                  ids, ascending) are cur_idx[row_ptr[u] .. row_ptr[u]+cur_len[u]).
 *   min_redundancy: 2 is Algorithm 3 as printed; larger values stop the loop earlier (an
 *                  option of the library, not of the paper);
 *   final_max_redundancy: the largest redundancy left when the loop stopped.  */
int64_t o3b_greedy(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t capacity, int32_t min_redundancy,
                   int32_t *trace_v1, int32_t *trace_v2, int32_t *trace_r,
                   int32_t *cur_len, int32_t *cur_idx, int32_t *final_max_redundancy)
{
    int64_t E = row_ptr[n];
    int64_t n_ids = n + capacity;
    int64_t num_agg = 0, rc = 0;
    pairmap map; heap hp = {0, 0, 0};
    ilist *out = (ilist *)calloc((size_t)n_ids, sizeof(ilist));
    int32_t *out_store = (int32_t *)malloc(sizeof(int32_t) * (size_t)(E > 0 ? E : 1));
    int32_t *delta = (int32_t *)calloc((size_t)n_ids, sizeof(int32_t));
    int32_t *touched = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_ids);
    int32_t *users = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    uint64_t cap0 = 1024;
    *final_max_redundancy = 0;
    if (!out || !out_store || !delta || !touched || !users || pm_init(&map, cap0)) return -1;

    memcpy(cur_idx, col, sizeof(int32_t) * (size_t)E);
    for (int64_t u = 0; u < n; ++u) cur_len[u] = (int32_t)(row_ptr[u + 1] - row_ptr[u]);

    /* out(s): the graph nodes whose row holds s (ascending because u ascends) */
    {
        int64_t *fill = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));
        if (!fill) return -1;
        for (int64_t e = 0; e < E; ++e) fill[col[e] + 1]++;
        for (int64_t s = 0; s < n; ++s) fill[s + 1] += fill[s];
        for (int64_t s = 0; s < n; ++s) { out[s].v = out_store + fill[s]; out[s].len = 0; }
        for (int64_t u = 0; u < n; ++u)
            for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) { ilist *l = &out[col[e]]; l->v[l->len++] = (int32_t)u; }
        free(fill);
    }

    /* initial redundancy of every pair that shares at least one row */
    for (int64_t u = 0; u < n; ++u) {
        const int32_t *row = col + row_ptr[u];
        int32_t len = cur_len[u];
        for (int32_t i = 0; i < len; ++i)
            for (int32_t j = i + 1; j < len; ++j) {
                int32_t *c = pm_slot(&map, pair_key(row[i], row[j]));
                if (!c) { rc = -1; goto done; }
                (*c)++;
            }
    }
    for (uint64_t i = 0; i <= map.mask; ++i)
        if (map.keys[i] != PM_EMPTY && map.vals[i] >= 2) {
            hent h = { map.vals[i], (int32_t)(map.keys[i] >> 32), (int32_t)(map.keys[i] & 0xffffffffu) };
            if (h_push(&hp, h)) { rc = -1; goto done; }
        }

    while (num_agg < capacity) {
        /* argmax of Redundancy over all pairs */
        hent top; int found = 0;
        while (hp.n > 0) {
            top = h_pop(&hp);
            int32_t *c = pm_slot(&map, pair_key(top.a, top.b));
            if (!c) { rc = -1; goto done; }
            if (*c == top.cnt) { found = 1; break; }
        }
        if (!found || top.cnt < min_redundancy) {              /* "if Redundancy > 1" when min_redundancy is 2 */
            if (found) h_push(&hp, top);                       /* keep it for the final maximum below */
            break;
        }
        int32_t v1 = top.a, v2 = top.b, w = (int32_t)(n + num_agg);

        /* R = { u : (v1,u) and (v2,u) are edges } */
        int32_t nu = 0;
        {
            ilist *A = &out[v1], *B = &out[v2];
            int32_t i = 0, j = 0;
            while (i < A->len && j < B->len) {
                if (A->v[i] < B->v[j]) ++i; else if (A->v[i] > B->v[j]) ++j;
                else { users[nu++] = A->v[i]; ++i; ++j; }
            }
        }
        if (nu != top.cnt) { rc = -2; goto done; }              /* map and rows disagree */
        trace_v1[num_agg] = v1; trace_v2[num_agg] = v2; trace_r[num_agg] = nu;

        /* how often every other member y shares a row of R with the pair */
        int32_t nt = 0;
        for (int32_t k = 0; k < nu; ++k) {
            int32_t u = users[k];
            int32_t *row = cur_idx + row_ptr[u];
            for (int32_t i = 0; i < cur_len[u]; ++i) {
                int32_t y = row[i];
                if (y == v1 || y == v2) continue;
                if (delta[y]++ == 0) touched[nt++] = y;
            }
        }
        for (int32_t t = 0; t < nt; ++t) {
            int32_t y = touched[t], dl = delta[y];
            delta[y] = 0;
            int32_t ends[2] = { v1, v2 };
            for (int q = 0; q < 2; ++q) {
                int32_t *c = pm_slot(&map, pair_key(ends[q], y));
                if (!c) { rc = -1; goto done; }
                *c -= dl;
                if (*c >= 2) {
                    hent h = { *c, ends[q] < y ? ends[q] : y, ends[q] < y ? y : ends[q] };
                    if (h_push(&hp, h)) { rc = -1; goto done; }
                }
            }
            int32_t *c = pm_slot(&map, pair_key(y, w));
            if (!c) { rc = -1; goto done; }
            *c = dl;
            if (dl >= 2) { hent h = { dl, y, w }; if (h_push(&hp, h)) { rc = -1; goto done; } }
        }
        { int32_t *c = pm_slot(&map, pair_key(v1, v2)); if (!c) { rc = -1; goto done; } *c -= nu; }

        /* E-hat <- E-hat - (v1,u) - (v2,u) + (w,u) for u in R; + (v1,w) + (v2,w) */
        for (int32_t k = 0; k < nu; ++k) {
            int32_t u = users[k];
            int32_t *row = cur_idx + row_ptr[u];
            int32_t len = cur_len[u], o = 0;
            for (int32_t i = 0; i < len; ++i) if (row[i] != v1 && row[i] != v2) row[o++] = row[i];
            row[o++] = w;                                       /* w exceeds every older id */
            cur_len[u] = o;
        }
        {
            int32_t ends[2] = { v1, v2 };
            for (int q = 0; q < 2; ++q) {
                ilist *L = &out[ends[q]];
                int32_t o = 0, k = 0;
                for (int32_t i = 0; i < L->len; ++i) {
                    while (k < nu && users[k] < L->v[i]) ++k;
                    if (k < nu && users[k] == L->v[i]) continue;
                    L->v[o++] = L->v[i];
                }
                L->len = o;
            }
            out[w].v = (int32_t *)malloc(sizeof(int32_t) * (size_t)nu);
            if (!out[w].v) { rc = -1; goto done; }
            memcpy(out[w].v, users, sizeof(int32_t) * (size_t)nu);
            out[w].len = nu;
        }
        ++num_agg;
    }
    /* what is left: the best still-valid entry, if any */
    while (hp.n > 0) {
        hent top = h_pop(&hp);
        int32_t *c = pm_slot(&map, pair_key(top.a, top.b));
        if (c && *c == top.cnt) { *final_max_redundancy = top.cnt; break; }
    }
    if (*final_max_redundancy == 0 && map.used > 0) {
        for (uint64_t i = 0; i <= map.mask; ++i)
            if (map.keys[i] != PM_EMPTY && map.vals[i] > *final_max_redundancy) *final_max_redundancy = map.vals[i];
    }
done:
    for (int64_t s = n; s < n_ids; ++s) free(out[s].v);
    free(out); free(out_store); free(delta); free(touched); free(users); free(hp.e); pm_free(&map);
    return rc < 0 ? rc : num_agg;
}

/* ------------------------------------------------------------------------- */
/* O3c: Algorithm 3 (set Aggregate) without a count per pair, for graphs whose
 * pair map does not fit in memory.  Exact, by this argument:
 *   - a merge of (v1, v2) only removes v1 and v2 from the rows that held both and
 *     adds the new node w there, so the redundancy of every existing pair can only
 *     fall, and a new pair (w, y) is held by a subset of the merged pair's rows;
 *   - hence bound[x] >= max over b of Redundancy(x, b) stays valid if it is set
 *     once to a true value (or to |out(x)| at the start, or to the merged pair's
 *     redundancy for a new node) and never raised;
 *   - the node x with the largest bound (ties: smallest id) is recounted from the
 *     definition; if its true maximum equals its bound, no pair anywhere has a
 *     larger redundancy, x is the smaller member of the lexicographically smallest
 *     pair attaining it (a smaller member would carry the same bound and a smaller
 *     id), and its partner is the smallest id attaining the count.  Otherwise the
 *     bound is lowered to the true maximum and the search goes on.
 * Same outputs as o3b_greedy.                                                 */
typedef struct { int32_t key, id; } lent;
static int l_before(const lent *x, const lent *y) {
    if (x->key != y->key) return x->key > y->key;
    return x->id < y->id;
}
typedef struct { lent *e; int64_t n, cap; } lheap;
static int l_push(lheap *h, lent v) {
    if (h->n == h->cap) {
        int64_t nc = h->cap ? h->cap * 2 : 1024;
        lent *ne = (lent *)realloc(h->e, sizeof(lent) * (size_t)nc);
        if (!ne) return -1;
        h->e = ne; h->cap = nc;
    }
    int64_t i = h->n++;
    while (i > 0) {
        int64_t p = (i - 1) / 2;
        if (!l_before(&v, &h->e[p])) break;
        h->e[i] = h->e[p]; i = p;
    }
    h->e[i] = v;
    return 0;
}
static lent l_pop(lheap *h) {
    lent top = h->e[0];
    lent last = h->e[--h->n];
    int64_t i = 0;
    for (;;) {
        int64_t l = 2 * i + 1, r = l + 1, c;
        if (l >= h->n) break;
        c = (r < h->n && l_before(&h->e[r], &h->e[l])) ? r : l;
        if (!l_before(&h->e[c], &last)) break;
        h->e[i] = h->e[c]; i = c;
    }
    if (h->n > 0) h->e[i] = last;
    return top;
}

int64_t o3c_greedy(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t capacity, int32_t min_redundancy,
                   int32_t *trace_v1, int32_t *trace_v2, int32_t *trace_r,
                   int32_t *cur_len, int32_t *cur_idx, int32_t *final_max_redundancy)
{
    int64_t E = row_ptr[n];
    int64_t n_ids = n + capacity;
    int64_t num_agg = 0, rc = 0;
    lheap hp = {0, 0, 0};
    ilist *out = (ilist *)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(ilist));
    int32_t *out_store = (int32_t *)malloc(sizeof(int32_t) * (size_t)(E > 0 ? E : 1));
    int32_t *bound = (int32_t *)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(int32_t));
    int32_t *count = (int32_t *)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(int32_t));
    int32_t *touched = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_ids > 0 ? n_ids : 1));
    int32_t *users = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    *final_max_redundancy = 0;
    if (!out || !out_store || !bound || !count || !touched || !users) return -1;

    memcpy(cur_idx, col, sizeof(int32_t) * (size_t)E);
    for (int64_t u = 0; u < n; ++u) cur_len[u] = (int32_t)(row_ptr[u + 1] - row_ptr[u]);
    {
        int64_t *fill = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));
        if (!fill) return -1;
        for (int64_t e = 0; e < E; ++e) fill[col[e] + 1]++;
        for (int64_t s = 0; s < n; ++s) fill[s + 1] += fill[s];
        for (int64_t s = 0; s < n; ++s) { out[s].v = out_store + fill[s]; out[s].len = 0; }
        for (int64_t u = 0; u < n; ++u)
            for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) { ilist *l = &out[col[e]]; l->v[l->len++] = (int32_t)u; }
        free(fill);
    }
    /* a pair cannot be held by more rows than hold either member */
    for (int64_t s = 0; s < n; ++s) {
        bound[s] = out[s].len;
        if (bound[s] >= 2) { lent v = { bound[s], (int32_t)s }; if (l_push(&hp, v)) { rc = -1; goto done; } }
    }
    for (;;) {
        /* the node with the largest bound whose recount confirms the bound */
        int32_t x = -1, best = 0, arg = -1;
        while (hp.n > 0) {
            lent top = l_pop(&hp);
            if (top.key != bound[top.id]) continue;             /* an older, higher bound of this node */
            int32_t cand = top.id, nt = 0;
            for (int32_t k = 0; k < out[cand].len; ++k) {       /* Redundancy(cand, y) for every y, from the definition */
                int32_t u = out[cand].v[k];
                const int32_t *row = cur_idx + row_ptr[u];
                for (int32_t i = 0; i < cur_len[u]; ++i) {
                    int32_t y = row[i];
                    if (y == cand) continue;
                    if (count[y]++ == 0) touched[nt++] = y;
                }
            }
            int32_t b = 0, a = -1;
            for (int32_t t = 0; t < nt; ++t) {
                int32_t y = touched[t], c = count[y];
                count[y] = 0;
                if (c > b || (c == b && y < a)) { b = c; a = y; }
            }
            if (b < top.key) {                                   /* stale: tighten and look again */
                bound[cand] = b;
                if (b >= 2) { lent v = { b, cand }; if (l_push(&hp, v)) { rc = -1; goto done; } }
                continue;
            }
            x = cand; best = b; arg = a;
            break;
        }
        if (x < 0) {                                             /* no pair is shared by two rows any more */
            int any = 0;
            for (int64_t u = 0; u < n && !any; ++u) any = cur_len[u] >= 2;
            *final_max_redundancy = any ? 1 : 0;
            break;
        }
        if (best < min_redundancy || num_agg >= capacity) {      /* "if Redundancy > 1" when min_redundancy is 2 */
            *final_max_redundancy = best;
            break;
        }
        if (arg <= x) { rc = -3; goto done; }                    /* would contradict the argument above */
        int32_t v1 = x, v2 = arg, w = (int32_t)(n + num_agg);
        int32_t nu = 0;
        {
            ilist *A = &out[v1], *B = &out[v2];
            int32_t i = 0, j = 0;
            while (i < A->len && j < B->len) {
                if (A->v[i] < B->v[j]) ++i; else if (A->v[i] > B->v[j]) ++j;
                else { users[nu++] = A->v[i]; ++i; ++j; }
            }
        }
        if (nu != best) { rc = -2; goto done; }
        trace_v1[num_agg] = v1; trace_v2[num_agg] = v2; trace_r[num_agg] = nu;
        for (int32_t k = 0; k < nu; ++k) {                       /* E-hat <- E-hat - (v1,u) - (v2,u) + (w,u) */
            int32_t u = users[k];
            int32_t *row = cur_idx + row_ptr[u];
            int32_t len = cur_len[u], o = 0;
            for (int32_t i = 0; i < len; ++i) if (row[i] != v1 && row[i] != v2) row[o++] = row[i];
            row[o++] = w;
            cur_len[u] = o;
        }
        {
            int32_t ends[2] = { v1, v2 };
            for (int q = 0; q < 2; ++q) {
                ilist *L = &out[ends[q]];
                int32_t o = 0, k = 0;
                for (int32_t i = 0; i < L->len; ++i) {
                    while (k < nu && users[k] < L->v[i]) ++k;
                    if (k < nu && users[k] == L->v[i]) continue;
                    L->v[o++] = L->v[i];
                }
                L->len = o;
            }
            out[w].v = (int32_t *)malloc(sizeof(int32_t) * (size_t)nu);
            if (!out[w].v) { rc = -1; goto done; }
            memcpy(out[w].v, users, sizeof(int32_t) * (size_t)nu);
            out[w].len = nu;
        }
        bound[w] = nu;                                           /* a pair with w is held by a subset of the nu rewritten rows */
        { lent v = { nu, w }; if (nu >= 2 && l_push(&hp, v)) { rc = -1; goto done; } }
        { lent v = { bound[v1], v1 }; if (l_push(&hp, v)) { rc = -1; goto done; } }   /* v1 left the heap when it was popped */
        ++num_agg;
    }
done:
    for (int64_t s = n; s < n_ids; ++s) free(out[s].v);
    free(out); free(out_store); free(bound); free(count); free(touched); free(users); free(hp.e);
    return rc < 0 ? rc : num_agg;
}

/* ------------------------------------------------------------------------- */
/* Replay of a recorded run of Algorithm 3 from the Redundancy definition, at any
 * size.  Independent of how the trace was found: no bounds, no heap, no pair map.
 *
 * State: the current rows (the edge set E-hat of Algorithm 3, graph-node rows
 * only, sorted) and, per node s, a candidate list cand(s) of rows that MAY hold s.
 * The rows are the authority; cand(s) only narrows which rows are looked at.  It is
 * a superset of the holders of s at all times: a graph node enters rows only in
 * the input graph (cand = its out-neighbours there), an aggregation node w only at
 * its creation (cand = the rows rewritten then), and entries are never added to
 * a row otherwise.
 *
 * Before merge i (recorded v1 < v2, redundancy r):
 *   - Redundancy(v1, v2) = number of rows that contain both, counted by testing
 *     every row of cand(v1); it must equal r, and r must be >= min_redundancy;
 *   - if i is one of check_steps: Redundancy of EVERY pair is recounted (for each
 *     node a, over the rows that hold a, one count per larger member b) and the
 *     recorded pair must be the largest, ties to the smallest v1 and then the
 *     smallest v2 (aggregation nodes numbered n, n+1, ... in creation order).
 * Then the rewrite of the algorithm's inner loop is applied: each such row loses v1
 * and v2 and gains w = n + i.
 * A check step equal to k (after the last merge) recounts every pair once more
 * and reports the largest redundancy that is left.
 *
 * report[0] = -1 when everything held, else the step that failed;
 * report[1] = what failed (1 bad pair ids, 2 redundancy differs, 3 below the stop
 *             value, 4 another pair is larger or earlier, 5 out of memory);
 * report[2] = largest redundancy left after the last merge (-1 if k was not a check step);
 * report[3] = full recounts done; report[4] = pair-count updates they made;
 * report[5], report[6], report[7] = on code 2: recount; on code 4: the arg-max pair and its redundancy.
 * cur_len / cur_idx receive the final rows laid over row_ptr.                     */
static int32_t row_pos(const int32_t *row, int32_t len, int32_t key)
{
    int32_t lo = 0, hi = len;
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if (row[mid] < key) lo = mid + 1; else hi = mid;
    }
    return (lo < len && row[lo] == key) ? lo : -1;
}

static void recount_all_pairs(int64_t n, int64_t n_ids, const int64_t *row_ptr, const int32_t *cur_len,
                              const int32_t *cur_idx, int32_t *const *cand, const int32_t *cand_len,
                              int32_t *count, int32_t *touched, int64_t *best_out, int32_t *a_out, int32_t *b_out,
                              int64_t *updates)
{
    int64_t best = 0;
    int32_t ba = -1, bb = -1;
    (void)n;
    for (int64_t a = 0; a < n_ids; ++a) {
        int32_t nt = 0;
        for (int32_t q = 0; q < cand_len[a]; ++q) {
            int32_t u = cand[a][q];
            const int32_t *row = cur_idx + row_ptr[u];
            int32_t p = row_pos(row, cur_len[u], (int32_t)a);
            if (p < 0) continue;
            for (int32_t i = p + 1; i < cur_len[u]; ++i) {      /* members b > a of a row that holds a */
                int32_t b = row[i];
                if (count[b]++ == 0) touched[nt++] = b;
            }
            *updates += cur_len[u] - p - 1;
        }
        int64_t loc = 0;
        int32_t lb = -1;
        for (int32_t t = 0; t < nt; ++t) {
            int32_t b = touched[t], c = count[b];
            count[b] = 0;
            if (c > loc || (c == loc && b < lb)) { loc = c; lb = b; }
        }
        if (loc > best) { best = loc; ba = (int32_t)a; bb = lb; }   /* strictly larger only: the smallest a wins ties */
    }
    *best_out = best; *a_out = ba; *b_out = bb;
}

int64_t o_replay_trace(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t k,
                       const int32_t *t1, const int32_t *t2, const int32_t *tr, int32_t min_redundancy,
                       int64_t n_checks, const int64_t *check_steps,
                       int32_t *cur_len, int32_t *cur_idx, int64_t *report)
{
    int64_t E = row_ptr[n], n_ids = n + k, rc = 0, next_check = 0;
    int64_t extra = 0;
    for (int64_t i = 0; i < k; ++i) extra += tr[i] > 0 ? tr[i] : 0;
    int32_t **cand = (int32_t **)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(int32_t *));
    int32_t *cand_len = (int32_t *)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(int32_t));
    int32_t *store = (int32_t *)malloc(sizeof(int32_t) * (size_t)(E + extra + 1));
    int32_t *count = (int32_t *)calloc((size_t)(n_ids > 0 ? n_ids : 1), sizeof(int32_t));
    int32_t *touched = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_ids > 0 ? n_ids : 1));
    for (int j = 0; j < 8; ++j) report[j] = -1;
    report[3] = 0; report[4] = 0;
    if (!cand || !cand_len || !store || !count || !touched) { report[0] = 0; report[1] = 5; rc = -1; goto done; }
    memcpy(cur_idx, col, sizeof(int32_t) * (size_t)E);
    for (int64_t u = 0; u < n; ++u) cur_len[u] = (int32_t)(row_ptr[u + 1] - row_ptr[u]);
    {
        int64_t *fill = (int64_t *)calloc((size_t)n + 1, sizeof(int64_t));
        if (!fill) { report[0] = 0; report[1] = 5; rc = -1; goto done; }
        for (int64_t e = 0; e < E; ++e) fill[col[e] + 1]++;
        for (int64_t s = 0; s < n; ++s) fill[s + 1] += fill[s];
        for (int64_t s = 0; s < n; ++s) cand[s] = store + fill[s];
        for (int64_t u = 0; u < n; ++u)
            for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) { int32_t s = col[e]; cand[s][cand_len[s]++] = (int32_t)u; }
        free(fill);
    }
    int32_t *free_store = store + E;
    for (int64_t i = 0; i <= k; ++i) {
        int check = 0;
        while (next_check < n_checks && check_steps[next_check] < i) ++next_check;
        if (next_check < n_checks && check_steps[next_check] == i) check = 1;
        if (check) {
            int64_t best; int32_t a, b;
            recount_all_pairs(n, n + i, row_ptr, cur_len, cur_idx, cand, cand_len, count, touched, &best, &a, &b, &report[4]);
            report[3]++;
            if (i == k) { report[2] = best; break; }
            if (best != tr[i] || a != t1[i] || b != t2[i]) {
                report[0] = i; report[1] = 4; report[5] = a; report[6] = b; report[7] = best; rc = -1; goto done;
            }
        }
        if (i == k) break;
        int32_t v1 = t1[i], v2 = t2[i], r = tr[i], w = (int32_t)(n + i);
        if (!(0 <= v1 && v1 < v2 && v2 < w)) { report[0] = i; report[1] = 1; rc = -1; goto done; }
        if (r < min_redundancy) { report[0] = i; report[1] = 3; rc = -1; goto done; }
        /* Redundancy(v1, v2): rows holding both; every row that holds v1 is in cand(v1) */
        int32_t nu = 0;
        int32_t *users = free_store;
        for (int32_t q = 0; q < cand_len[v1]; ++q) {
            int32_t u = cand[v1][q];
            const int32_t *row = cur_idx + row_ptr[u];
            if (row_pos(row, cur_len[u], v1) >= 0 && row_pos(row, cur_len[u], v2) >= 0) {
                if (nu < r) users[nu] = u;
                ++nu;
            }
        }
        if (nu != r) { report[0] = i; report[1] = 2; report[5] = nu; rc = -1; goto done; }
        for (int32_t q = 0; q < nu; ++q) {                       /* E-hat <- E-hat - (v1,u) - (v2,u) + (w,u) */
            int32_t u = users[q];
            int32_t *row = cur_idx + row_ptr[u];
            int32_t len = cur_len[u], o = 0;
            for (int32_t j = 0; j < len; ++j) if (row[j] != v1 && row[j] != v2) row[o++] = row[j];
            row[o++] = w;                                        /* w is the largest id so far: the row stays sorted */
            cur_len[u] = o;
        }
        cand[w] = users; cand_len[w] = nu;
        free_store += nu;
    }
done:
    free(cand); free(cand_len); free(store); free(count); free(touched);
    return rc;
}

/* Theorem 2's condition on rows in creation-id space: expanding every aggregation
 * node of row u into its two inputs (t1, t2) until only graph nodes remain must
 * give N(u) of the input graph, every source exactly once.  Returns -1 when all
 * rows pass, else the first row that does not.                                 */
static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int64_t o_cover_check(int64_t n, const int64_t *row_ptr, const int32_t *col, int64_t k,
                      const int32_t *t1, const int32_t *t2, const int32_t *cur_len, const int32_t *cur_idx)
{
    int64_t max_deg = 0, bad = -1;
    (void)k;
    for (int64_t u = 0; u < n; ++u) if (row_ptr[u + 1] - row_ptr[u] > max_deg) max_deg = row_ptr[u + 1] - row_ptr[u];
    int32_t *leaves = (int32_t *)malloc(sizeof(int32_t) * (size_t)(max_deg + 1));
    int32_t *stack = (int32_t *)malloc(sizeof(int32_t) * (size_t)(max_deg + 2));
    if (!leaves || !stack) { free(leaves); free(stack); return -2; }
    for (int64_t u = 0; u < n && bad < 0; ++u) {
        int64_t deg = row_ptr[u + 1] - row_ptr[u], nl = 0, ns = 0;
        if (cur_len[u] > deg) { bad = u; break; }
        for (int32_t i = 0; i < cur_len[u]; ++i) stack[ns++] = cur_idx[row_ptr[u] + i];
        while (ns > 0 && bad < 0) {
            int32_t s = stack[--ns];
            if (s < n) { leaves[nl++] = s; }
            else { stack[ns++] = t1[s - n]; stack[ns++] = t2[s - n]; }
            if (nl + ns > deg) bad = u;              /* more sources than N(u) has: stop before the buffers overflow */
        }
        if (bad >= 0) break;
        if (nl != deg) { bad = u; break; }
        qsort(leaves, (size_t)nl, sizeof(int32_t), cmp_i32);
        for (int64_t j = 0; j < nl; ++j) if (leaves[j] != col[row_ptr[u] + j]) { bad = u; break; }
    }
    free(leaves); free(stack);
    return bad;
}
