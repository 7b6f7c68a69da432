/*
 * hag.h -- C ABI of the B200 HAG aggregation library.
 *
 * Sum / mean neighbourhood aggregation of a GNN layer, forward and backward,
 * evaluated over a Hierarchically Aggregated computation Graph (HAG) as defined
 * in "Redundancy-Free Computation Graphs for Graph Neural Networks"
 * (arxiv 1906.03707).  The three operations the paper implements
 * (Section 5.1: graph_to_hag, hag_aggregate, hag_aggregate_grad) map to
 * hag_build, hag_aggregate_fwd and hag_aggregate_bwd; csr_aggregate_* evaluate
 * the plain GNN-graph (the special case V_A = {} of Section 3.1) with the same
 * kernels, as the comparison path.  Beyond that core: hag_max_* / csr_max_* (the
 * element-wise max Aggregate of Table 1's GraphSAGE-P row over the same HAG) and
 * hag_graph_pool_* (the mean-pooling read-out of Section 5.1 over the graphs of
 * a batch).
 *
 * Conventions
 *   ids        graph nodes 0..N-1; aggregation nodes N..N+|V_A|-1, sorted by level
 *              (level = longest path from a graph node; every aggregation node
 *              comes after both of its inputs).
 *   graphs     CSR of IN-neighbours on the HOST: row v lists the sources u that v
 *              aggregates (the edge (u,v) of Section 3.1), int64 row_ptr[N+1],
 *              int32 col_idx[E], every row strictly ascending (no duplicates).
 *              Self-loops are ordinary edges.
 *   features   x, out, grad_out, grad_x are DEVICE pointers to N x D row-major
 *              contiguous matrices of the given dtype, 16-byte aligned, with
 *              D * sizeof(dtype) a multiple of 16.
 *   workspace  DEVICE pointer to hag_workspace_bytes() bytes, 16-byte aligned; holds
 *              the fp32 rows of the aggregation nodes (a-hat of Algorithm 2, or their
 *              gradients) and the partial sums of split long rows.  It carries
 *              nothing between calls and may be shared by all layers and by
 *              forward and backward (Algorithm 2's caption).
 *   streams    cuda_stream is a cudaStream_t passed as void* (NULL = default
 *              stream).  Calls only enqueue work; they never synchronise.
 *   errors     every function returns a hag_status; nothing throws, aborts or
 *              traps.  Argument checks are synchronous.  A failing kernel surfaces
 *              at the caller's next synchronisation, as usual for CUDA.
 *   threads    a handle may be used from one thread at a time, and its aggregate calls
 *              must be ordered on the device (one stream, or events between
 *              streams): the handle owns small scheduling counters that the
 *              kernels of consecutive calls take turns on.
 *   results    no floating-point atomics anywhere: the same inputs give the same
 *              bits on every run.
 */
#ifndef HAG_B200_H
#define HAG_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hag hag_t; /* opaque: owns the structure arrays on host and device */

typedef enum {
    HAG_OK = 0,
    HAG_ERR_NULL = 1,        /* a required pointer is NULL                                  */
    HAG_ERR_ARG = 2,         /* a scalar argument is out of range                           */
    HAG_ERR_GRAPH = 3,       /* malformed CSR (unsorted / duplicate / out-of-range columns) */
    HAG_ERR_OOM_HOST = 4,
    HAG_ERR_OOM_DEVICE = 5,
    HAG_ERR_CUDA = 6,        /* a CUDA runtime call failed (incl. no device)                */
    HAG_ERR_DTYPE = 7,
    HAG_ERR_ALIGN = 8,       /* pointer or row size not 16-byte aligned                     */
    HAG_ERR_WORKSPACE = 9,   /* workspace missing although the HAG has aggregation nodes    */
    HAG_ERR_TIMEOUT = 10,    /* a bounded device-side wait gave up (see hag_device_status)  */
    HAG_ERR_NOT_ON_DEVICE = 11,/* hag_to_device has not been called                         */
    HAG_ERR_TOO_LARGE = 12     /* the problem needs more than the built-in scratch array holds */
} hag_status;

/* HAG_SUM: a_v = sum of h_u over N(v) (GCN's Aggregate, Table 1).  HAG_MEAN: that sum / |N(v)|.
 * HAG_GCN: the argument of GCN's Update in Table 1, (a_v + h_v) / (|N(v)| + 1), i.e. the sum with the
 * node's own row added and the normalisation fused into the gather's epilogue (the weight matrix and the
 * non-linearity stay with the caller).  Its gradient is gx_u = sum over v with u in N(v) of
 * g_v / (|N(v)| + 1), plus g_u / (|N(u)| + 1). */
typedef enum { HAG_SUM = 0, HAG_MEAN = 1, HAG_GCN = 2 } hag_reduce;
typedef enum { HAG_F32 = 0, HAG_BF16 = 1 } hag_dtype;

/* Counters of one built HAG.  "aggregations" are binary aggregations as counted
 * by the cost function of Section 4.1: sum over nodes of (in-edges - 1). */
typedef struct hag_info {
    int32_t n;                      /* |V|                                                    */
    int32_t capacity;               /* the limit that was asked for                           */
    int32_t num_agg;                /* |V_A| (<= capacity: the search stops at redundancy 1)   */
    int32_t num_levels;             /* depth of the hierarchy                                 */
    int64_t e;                      /* |E| of the input graph (directed)                      */
    int64_t e_hat;                  /* |E-hat| = 2 |V_A| + residual edges                     */
    int64_t aggregations_gnn;       /* sum_v max(|N(v)| - 1, 0)                               */
    int64_t aggregations_hag;       /* the same sum over V and V_A of the HAG                 */
    int64_t aggregations_hag_closed;/* |E-hat| - |V| - |V_A| (equal when no row is empty)     */
    int64_t saved;                  /* sum_i (r_i - 1) = f of the Theorem 4 proof             */
    int32_t first_redundancy;       /* r of the first merge (0 if none)                       */
    int32_t last_redundancy;        /* r of the last merge                                    */
    int32_t max_in_degree;          /* longest row of the input graph                         */
    int32_t max_res_degree;         /* longest residual row                                   */
    int32_t max_out_degree;         /* longest row of the transposed HAG                      */
    int32_t device;                 /* CUDA device holding the arrays, -1 if host only        */
    double build_seconds;           /* host time spent in the search and layout               */
} hag_info;

/* Borrowed HOST views of the canonical arrays; valid until hag_destroy. */
typedef struct hag_arrays {
    int32_t n, num_agg, num_levels;
    const int64_t *level_ptr;  /* [num_levels+1] level l (1-based) = ids n+level_ptr[l-1] .. n+level_ptr[l]-1 */
    const int32_t *agg_in;     /* [2*num_agg] inputs (lo < hi) of aggregation node n+j                 */
    const int64_t *res_ptr;    /* [n+1]                                                                */
    const int32_t *res_idx;    /* residual in-neighbours of every graph node, ascending                */
    const int64_t *t_ptr;      /* [n+num_agg+1] transposed HAG, by source                              */
    const int32_t *t_idx;      /* destinations ascending; d < n: output row d; d >= n: aggregation node */
    const int32_t *in_degree;  /* [n] |N(v)| of the input graph                                        */
    const int32_t *trace;      /* [3*num_agg] merges in creation order: v1 < v2 (creation ids), r      */
    const int64_t *csr_t_ptr;  /* [n+1] transposed input graph                                          */
    const int32_t *csr_t_idx;
    /* Deep levels evaluated in one launch each way (see hag_build): */
    int32_t fwd_cut;           /* levels 1..fwd_cut run level by level; deeper nodes from their expansion  */
    int32_t bwd_cut;           /* same for the backward pass                                              */
    const int64_t *ftail_ptr;  /* [num_agg - level_ptr[fwd_cut] + 1]                                       */
    const int32_t *ftail_idx;  /* per deep node: the ids of level <= fwd_cut whose sum it is, ascending    */
    const int64_t *btail_ptr;  /* [num_agg - level_ptr[bwd_cut] + 1]                                       */
    const int32_t *btail_idx;  /* per deep node: the graph nodes whose output uses it, ascending           */
} hag_arrays;

/* Algorithm 3, set-Aggregate branch (the paper's graph_to_hag): starting from the
 * GNN-graph, repeatedly merge the pair of nodes (graph or aggregation nodes) that
 * the most graph nodes aggregate together into a new aggregation node, until
 * `capacity` nodes exist or no pair is shared by more than one node.  Ties go to
 * the lexicographically smallest pair (v1 < v2; aggregation nodes numbered N, N+1,
 * ... as created).  Then lays the result out for the device (levels, level-sorted
 * ids, input pairs, residual CSR, transposed HAG, transposed input graph).
 * Deep levels are usually tiny, and a launch per level would cost more than the
 * rows it moves.  So the layout also picks a cut c: levels 1..c are evaluated
 * level by level (Algorithm 2 lines 5-6), and every deeper node directly as the
 * sum over its cover restricted to ids of level <= c (Section 3.1: aggr(v) is the
 * aggregate over cover(v)), all in one launch.  c minimises
 *   32768 * (launches) + sum over deep nodes of (expanded inputs - 1),
 * ties to the larger c; c = num_levels means no expansion.  The backward pass
 * has its own cut: nodes deeper than it gather straight from the graph-node
 * outputs that use them (transitively), 131072 per launch, cost term (expanded
 * users - direct users).
 * Host only; the input arrays are read during the call and not kept.
 * Errors: HAG_ERR_NULL; HAG_ERR_ARG (n < 0, capacity < 0, n + capacity or |E| >=
 * 2^31); HAG_ERR_GRAPH; HAG_ERR_OOM_HOST.  On error *out is NULL. */
hag_status hag_build(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t capacity, hag_t **out);

/* hag_build with a different stop value (an extension: the paper stops at redundancy 1).
 * Merging a pair shared by r rows removes r - 2 row reads but adds one row write and, later,
 * re-reads of the new row: it saves aggregations for every r >= 2 (the paper's cost function) but
 * bytes only from r >= 4 on.  The search stops as soon as the best redundancy is below
 * min_redundancy (>= 2; 2 reproduces hag_build exactly) or `capacity` nodes exist.
 * HAG_ERR_ARG if min_redundancy < 2; otherwise as hag_build. */
hag_status hag_build_ex(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t capacity,
                        int32_t min_redundancy, hag_t **out);

/* Host threads hag_build may use for recounting pair redundancies (process-wide).
 * 0 = as many as the host has, at most 16 (the default); 1 = single-threaded;
 * a negative value only queries.  Returns the previous setting.  The merge
 * sequence, and so every array of the result, does not depend on it. */
int32_t hag_build_threads(int32_t threads);

/* The HAG the same graph would get with a smaller capacity (the capacity study of
 * Section 5.4 without repeating the search): Algorithm 3 adds one node per
 * iteration, so its result for capacity c is its first c merges.  Replays the
 * first min(capacity, |V_A|) merges recorded in `src` and lays the result out;
 * *out equals hag_build(graph, capacity) bit for bit.  `src` is unchanged and the
 * new handle is independent of it (host only until hag_to_device).
 * HAG_ERR_ARG if capacity < 0, or if capacity exceeds the recorded merges while
 * `src` stopped only because it hit its own capacity. */
hag_status hag_truncate(const hag_t *src, int32_t capacity, hag_t **out);

/* The HAG of a graph from a merge trace recorded earlier (hag_export's `trace`: 3 int32 per merge, v1 < v2 in
 * creation ids, redundancy), without running the search again: a 30-second build becomes a replay of a second or
 * two (the paper computes a HAG once per graph and reuses it: Section 5.1).  Every merge is checked as it is
 * replayed: ids in range and ordered, recorded redundancy >= 2 and equal to the number of rows that hold both nodes
 * at that point, so the result is always a correct HAG of THIS graph (Theorem 2's cover condition holds by
 * construction); it equals hag_build's bit for bit when the trace came from hag_build on the same graph, which is
 * not checked (whether each merge was the arg-max is the search's business).  The handle's capacity is num_merges.
 * Errors: as hag_build for the graph; NULL (trace missing); ARG (num_merges < 0, or a merge that does not replay). */
hag_status hag_import(int32_t n, const int64_t *row_ptr, const int32_t *col_idx, int32_t num_merges, const int32_t *trace,
                      hag_t **out);

/* Replaces the cuts that hag_build chose (see there) and rebuilds the expansion lists of the
 * deep levels.  Every cut 0 <= c <= num_levels evaluates the same HAG to the same values up to
 * the order of additions (Section 3.1, Eq. 1: a node is the Aggregate over its cover); the
 * choice only trades launches or dependent steps against longer input lists.  -1 for either
 * argument keeps the library's own choice for that pass.  Host only, before hag_to_device.
 * Errors: NULL; ARG (a cut outside -1..num_levels, or the handle is already on a device);
 * OOM_HOST. */
hag_status hag_set_cuts(hag_t *h, int32_t fwd_cut, int32_t bwd_cut);

/* Frees host and device arrays.  NULL is allowed. */
hag_status hag_destroy(hag_t *h);

/* Counters of Section 4.1 / Section 5.3 for this HAG. */
hag_status hag_get_info(const hag_t *h, hag_info *out);

/* Borrowed host pointers to the canonical arrays (for checking and export). */
hag_status hag_export(const hag_t *h, hag_arrays *out);

/* Copies the structure arrays to CUDA device `device` (idempotent for the same
 * device; HAG_ERR_ARG if already on another one).  Synchronous.  Allocates with
 * cudaMalloc; HAG_ERR_OOM_DEVICE / HAG_ERR_CUDA on failure. */
hag_status hag_to_device(hag_t *h, int device);

/* Bytes of workspace hag_aggregate_* need for feature width D: fp32 rows (whatever
 * the dtype) for the |V_A| aggregation nodes, plus one partial row per segment of the
 * rows that are summed by several warps.  Rows are split at one of three granularities,
 * by the size of the launch or pass: more than 64 entries into segments of 32, more than
 * 256 into 128, more than 1024 into 512; the table with the most segments decides.
 * 0 on bad arguments or when
 * neither exists.  csr_workspace_bytes: the same for csr_aggregate_* (segments of
 * the input graph's long rows only; 0 for graphs without such rows). */
size_t hag_workspace_bytes(const hag_t *h, int32_t D);
size_t csr_workspace_bytes(const hag_t *h, int32_t D);

/* Algorithm 2 (the paper's hag_aggregate), one layer:
 *   a-hat_w = a-hat_in0(w) + a-hat_in1(w)  for aggregation nodes, level by level;
 *   out_v   = sum over the residual in-neighbours of v of a-hat  (x_u for graph nodes),
 *   times 1/|N(v)| for HAG_MEAN (|N(v)| = in-degree in the input graph; an empty
 *   neighbourhood gives a zero row).
 * x and out are N x D of `dtype`, must not overlap; accumulation is fp32.
 * Enqueues 1 + (number of level launches) kernels on the stream (hag_set_schedule 1: one kernel).
 * Errors: NULL, ARG (D <= 0), DTYPE, ALIGN, WORKSPACE, NOT_ON_DEVICE, CUDA. */
hag_status hag_aggregate_fwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                             const void *x, void *out, void *workspace, void *cuda_stream);

/* Gradient of the above (the paper's hag_aggregate_grad; Section 3.2 requires the
 * same gradients as the GNN-graph): grad_x = A^T (s * grad_out), s_v = 1 or
 * 1/|N(v)|, computed without atomics by gathering over the transposed HAG --
 * aggregation nodes from the last level to the first, then the input rows. */
hag_status hag_aggregate_bwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                             const void *grad_out, void *grad_x, void *workspace, void *cuda_stream);

/* The GNN-graph itself (Algorithm 1 line 4; V_A = {} in Section 3.1): the same
 * gather kernel over the input CSR held by the handle, and over its transpose for
 * the gradient.  workspace: csr_workspace_bytes() bytes (may be NULL when that is 0). */
hag_status csr_aggregate_fwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                             const void *x, void *out, void *workspace, void *cuda_stream);
hag_status csr_aggregate_bwd(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                             const void *grad_out, void *grad_x, void *workspace, void *cuda_stream);

/* Host-buffer variants for callers that keep features in host memory: x_host and
 * out_host are HOST pointers to N x D matrices (pinned memory makes the copies
 * asynchronous).  The call copies the input to device staging buffers owned by
 * the handle (grown on demand with cudaMalloc), runs the aggregation on
 * cuda_stream and copies the result back on cuda_stream; it returns after
 * enqueuing, so the caller synchronises the stream before reading out_host.
 * The copy-in runs on a stream of the handle's own, into one of two buffers, so
 * that the copy-in of a call overlaps the aggregation and the copy-out of the
 * call before it (both directions of the host link are busy at once).  For that
 * reason x_host must hold its data when the call is made (it is read without
 * waiting for earlier work in cuda_stream) and must stay unchanged until the
 * stream has been synchronised; consecutive calls on one handle must use the same
 * cuda_stream or be separated by a synchronisation.  `backward` != 0 runs
 * hag_aggregate_bwd instead of hag_aggregate_fwd; `use_hag` == 0 runs the
 * csr_aggregate_* path. */
hag_status hag_aggregate_host(hag_t *h, int backward, int use_hag, hag_reduce reduce, hag_dtype dtype, int32_t D,
                              const void *in_host, void *out_host, void *cuda_stream);

/* Per-launch timing for measurement (no counterpart in the paper; it reports
 * kernel time only).  While enabled, every kernel an aggregate call enqueues is
 * bracketed by a pair of CUDA events on the caller's stream (created on first use
 * with cudaEventCreate and kept by the handle).  hag_profile_read synchronises
 * on the events of the LAST call and returns how many launches it made; for the
 * first `max` of them it fills ms[i] (device time), kind[i] (0 = level pair-sum,
 * 1 = gather over aggregation nodes: one level of the backward pass, or the
 * expanded deep levels of either pass, 2 = gather over the graph nodes, 3 = a whole
 * pass in one launch), rows[i]
 * (rows written) and edges[i] (source rows read).  A gather over a table with
 * split long rows is still one launch: segments and rows share it.
 * Arrays may be NULL.  Returns -1 on error. */
hag_status hag_profile_enable(hag_t *h, int enable);
int32_t hag_profile_read(hag_t *h, int32_t max, float *ms, int32_t *kind, int64_t *rows, int64_t *edges);

/* Graph read-out for graph classification (Section 5.1: after the GNN layers "a
 * mean-pooling layer" gathers graph-level activations).  A batch of graphs is laid
 * out as in workload shapes of that kind: graph i owns the consecutive node rows
 * seg_ptr[i] .. seg_ptr[i+1]-1 of x.
 *   forward : out_i = sum of the rows of graph i, times 1/(number of rows) for
 *             HAG_MEAN; a graph without rows gives a zero row.  HAG_SUM and HAG_MEAN only.
 *   backward: grad_x_v = s_i * grad_out_i for every row v of graph i (s_i = 1 or
 *             1/rows); rows of grad_x before seg_ptr[0] and from seg_ptr[n_graphs]
 *             to n_rows are set to zero.
 * seg_ptr: DEVICE pointer to n_graphs + 1 non-decreasing int32 row offsets (not
 * checked: it lives on the device).  x / grad_x: n_rows x D, out / grad_out:
 * n_graphs x D of `dtype`, DEVICE pointers, 16-byte aligned, D * sizeof(dtype) a
 * multiple of 16; accumulation is fp32 on two levels (a row of the sum passes
 * through at most about rows/64 + 12 roundings).  One kernel each, on the current
 * device, no handle, no workspace, no allocation.  One warp reads the rows of one
 * graph, so the launch suits batches of many small graphs.
 * A matrix that has no rows (out / grad_out when n_graphs = 0, grad_x when n_rows = 0)
 * may be NULL; x is not read when n_graphs = 0.
 * Errors: NULL, ARG (D <= 0, n_graphs < 0, n_rows < 0, reduce), DTYPE, ALIGN, CUDA. */
hag_status hag_graph_pool_fwd(const int32_t *seg_ptr, int32_t n_graphs, hag_reduce reduce, hag_dtype dtype,
                              int32_t D, const void *x, void *out, void *cuda_stream);
hag_status hag_graph_pool_bwd(const int32_t *seg_ptr, int32_t n_graphs, int32_t n_rows, hag_reduce reduce,
                              hag_dtype dtype, int32_t D, const void *grad_out, void *grad_x, void *cuda_stream);

/* Element-wise max aggregation over the same HAG (Table 1, GraphSAGE-P:
 * a_v = max over u in N(v) of z_u, z = the activations the model feeds to the
 * pooling).  Max is associative and commutative, i.e. a set Aggregate in the sense
 * of Section 3.1, so Algorithm 2 applies with max in place of the sum and the HAG
 * built by hag_build is reused as it is.
 *   hag_max_fwd : a-hat_w = max(a-hat_in0, a-hat_in1) for aggregation nodes, then
 *                 out_v = max over the residual in-neighbours of v; an empty
 *                 neighbourhood gives a zero row.  Exact (no rounding): the result
 *                 equals the direct evaluation bit for bit, for both dtypes.
 *                 `workspace`: hag_max_workspace_bytes(h, D) bytes (|V_A| x D fp32);
 *                 after the call it holds the maxima of the aggregation nodes,
 *                 which hag_max_bwd needs: keep it until then.
 *   hag_max_bwd : gradient for L = sum_v <grad_out_v, out_v>: component k of
 *                 grad_out_v goes to the in-neighbours u with z_u[k] == out_v[k];
 *                 on a tie every such u receives it (the paper does not say; ties
 *                 have probability zero for continuous activations).  Computed as
 *                 a gather over the transposed HAG, no atomics, fixed summation
 *                 order.  Takes z and out of the forward call, `fwd_workspace` as
 *                 hag_max_fwd left it (read only), and a second buffer `workspace`
 *                 of the same size for the gradients of the aggregation nodes.
 *   csr_max_fwd / csr_max_bwd : the same on the plain GNN-graph (no workspace).
 * z, out, grad_out, grad_z: N x D of `dtype`, DEVICE pointers, 16-byte aligned, must not
 * overlap one another; values must not be NaN.  Rows are not split: a row of a
 * thousand entries is walked by one warp.
 * Errors: NULL, ARG (D <= 0, overlapping buffers), DTYPE, ALIGN, WORKSPACE,
 * NOT_ON_DEVICE, CUDA. */
size_t hag_max_workspace_bytes(const hag_t *h, int32_t D);
hag_status hag_max_fwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, void *out, void *workspace,
                       void *cuda_stream);
hag_status hag_max_bwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, const void *out,
                       const void *fwd_workspace, const void *grad_out, void *grad_z, void *workspace,
                       void *cuda_stream);
hag_status csr_max_fwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, void *out, void *cuda_stream);
hag_status csr_max_bwd(const hag_t *h, hag_dtype dtype, int32_t D, const void *z, const void *out,
                       const void *grad_out, void *grad_z, void *cuda_stream);

/* hag_aggregate_fwd for callers that must not allocate device memory (the paper
 * has no counterpart: its operators take their buffers from the framework).
 *
 * Some hosts cannot hand this library a workspace and cannot let it call
 * cudaMalloc either: a serving process whose device memory is one arena sized at
 * start-up and owned by another component, or a latency-bound loop in which the
 * device-wide synchronisation that cudaMalloc/cudaFree imply would stall every
 * other stream.  For them the rows of the aggregation nodes live in an array that
 * is part of the library image itself: HAG_STATIC_SCRATCH_BYTES of device memory,
 * reserved on every GPU that loads the library until the process exits.
 *
 * Same arguments, results and errors as hag_aggregate_fwd, without `workspace`.
 * Bit-identical output to hag_aggregate_fwd.  Additionally:
 *   - HAG_ERR_TOO_LARGE when hag_workspace_bytes(h, D) (aggregation-node rows plus
 *     the partial rows of split long rows) exceeds
 *     HAG_STATIC_SCRATCH_BYTES (nothing is launched);
 *   - the call itself allocates nothing: no cudaMalloc, cudaFree, event or stream
 *     creation, and no host heap use;
 *   - the first call on each device looks up the array's device address (a
 *     one-off query, made with that device current).  Make that first call
 *     during start-up, before any stream capture begins;
 *   - there is ONE array per device, shared by every handle and every call, and
 *     it still holds the previous call's rows.  The forward pass writes every
 *     aggregation-node row before it reads it, so nothing needs clearing; but
 *     two calls that can run at the same time on one device (different streams,
 *     or different threads) race on the array and corrupt each other's result.
 *     Keep such calls on one stream or order them with events. */
#define HAG_STATIC_SCRATCH_BYTES (16u << 20)
hag_status hag_aggregate_fwd_static(const hag_t *h, hag_reduce reduce, hag_dtype dtype, int32_t D,
                                    const void *x, void *out, void *cuda_stream);

/* How a pass is scheduled on the device (no counterpart in the paper, which does not describe its kernels).
 *   0 (default)  a launch per level: pair-sum kernels for the levels up to the cut, one gather for the expanded
 *                deeper nodes, one gather for the graph nodes (hag_last_launch_count says how many).
 *   1            ONE launch per pass.  Algorithm 2 only asks that every aggregation node comes after its
 *                inputs and the graph nodes last.  The pass is a list of rows in that order -- one phase per
 *                level evaluated pair by pair (rows of two entries), one for the expanded deeper nodes, the
 *                graph-node rows last; a row too long for one warp is cut into chunk rows of a phase of their
 *                own and becomes the short sum of their partial rows -- which resident warps take in list
 *                order.  A row sums its entries from the layer input at once and waits, before it reads rows
 *                of an earlier phase, until that phase's count of finished rows is complete.
 *                The wait cannot deadlock (what it waits for was handed out earlier, to a running warp) and
 *                is bounded anyway: after about a second of polling the warp records the failure and goes
 *                on, the launch ends, and hag_device_status reports HAG_ERR_TIMEOUT (results of that call
 *                are then undefined).  The plain-CSR calls use the same kernel (phases: chunk rows, rows).
 *                Measured on B200 this form is level with the default on the two largest fp32 shapes and
 *                slower on small graphs and deep hierarchies (resident warps hide less latency than the
 *                hardware's block scheduling does on launches of 10^5 rows), which is why it is not the default.
 *   2            TWO launches per pass: the rows of the aggregation nodes (every phase of the list of form 1 before
 *                the graph nodes) in one launch of that kernel, then the graph nodes by the row kernels of form
 *                0.  For hierarchies of many small levels, where form 0 spends most of a pass launching and
 *                draining kernels of a few thousand rows; the same bounded waits and the same report apply.
 *                The plain-CSR calls are not affected (they have no aggregation nodes).
 * Passes whose hierarchy has more than 56 phases always run level by level.
 * Errors: NULL; ARG (a value other than 0, 1 or 2). */
hag_status hag_set_schedule(hag_t *h, int32_t schedule);

/* HAG_OK, or HAG_ERR_TIMEOUT if a bounded device-side wait of an earlier call on this handle gave up
 * (reading clears it).  Does not synchronise: call it after synchronising the stream of the calls
 * in question.  Reads one word of pinned host memory that the kernels can write.
 * Errors: NULL, NOT_ON_DEVICE. */
hag_status hag_device_status(hag_t *h);

/* Exercises the give-up path of that wait on purpose, safely: a launch of ONE thread block over a
 * two-phase list of four rows whose first phase nobody ever finishes, with a poll limit of a few
 * milliseconds.  The kernel must record the failure and end.  Synchronises the stream and returns what
 * hag_device_status then says: HAG_ERR_TIMEOUT means the mechanism works, HAG_OK that it does not.
 * Allocates a few hundred bytes with cudaMalloc for the call.  Errors: NULL, NOT_ON_DEVICE, OOM_DEVICE, CUDA. */
hag_status hag_selftest_wait_limit(hag_t *h, void *cuda_stream);

/* Borrowed HOST view of the row list of one pass (pass: 0 forward over the HAG, 1 backward over the HAG,
 * 2 forward over the input graph, 3 backward over it), for inspection and checking.  rows: 4 int32 per row
 * {b, e, row, phases}: the row sums the entries ids[b .. e) into output row `row` (row < 0: padding; row < n: a
 * graph node; n <= row < n + |V_A|: an aggregation node; from n + |V_A| on: a chunk row, the fp32 partial sum of a
 * piece of a long row, which a later short row adds up); phases = (phase that must be complete before the row
 * reads, plus one; 0 = none) | (the row's own phase) << 8.  n_rows = 0: the pass has no list (it runs level by level). */
typedef struct hag_pass_view {
    int64_t n_rows, n_phases, n_chunk_rows, n_ids;
    const int32_t *rows;        /* [4 * n_rows]  */
    const int32_t *phase_size;  /* [n_phases] rows per phase, padding included */
    const int32_t *ids;         /* [n_ids]       */
} hag_pass_view;
hag_status hag_export_pass(const hag_t *h, int32_t pass, hag_pass_view *out);

/* The order in which the kernels that walk several rows per warp take the rows of one list (feature rows of 256 bytes
 * or less: every group of lanes walks a row of its own, in lock step with the warp's other groups, so rows of like
 * length belong side by side).  list: 0 residual rows (Algorithm 2 lines 7-8), 1 transposed HAG, 2 input graph
 * (Algorithm 1 line 4), 3 its transpose, 4 / 5 the expansion lists of the forward / backward cut.  order[i] is the
 * row taking the place of row first_row + i: a permutation that sorts the rows by length (longest first) within
 * windows of 2048 rows, the windows never crossing from the graph nodes into a level or from one level into the next,
 * so every launch's rows map onto themselves.  Aggregation nodes are numbered in the order of the search, not of the
 * graph; a level or an expansion list of 8192 of their rows or more is therefore first put in the order of the rows'
 * first entries (rows that read the same neighbourhood side by side: what one brings into the L2 the next find
 * there; the one-row-per-warp kernel uses the order for these launches too), then cut into the windows.
 * count = 0 (order NULL): the rows are taken as they are (pairs of neighbouring rows already lose less than 8 % of
 * the lock-step rounds, and no segment qualifies for the order of first entries).  No value depends on the order: each row is
 * summed by one group in the row's own order of entries.  The array lives as long as the handle; hag_set_cuts
 * rebuilds lists 4 and 5.  Errors: NULL, ARG (list outside 0..5). */
hag_status hag_export_row_order(const hag_t *h, int32_t list, int32_t *first_row, int64_t *count, const int32_t **order);

/* Device-side check of the uploaded structure: small kernels read every index array on the device and test each
 * pointer (first one 0, none stepping back, last one the list's length) and each id (inside the range of rows its
 * list may name: graph nodes and aggregation nodes for the HAG's lists, graph nodes for the input graph, the levels
 * up to the cut for the forward expansion, a permutation's own range for the row orders).  The aggregation kernels
 * trust these arrays (hag_build validated the graph on the host before anything was derived from it), so this is
 * the call that notices an upload or a device memory that went wrong, without a gather kernel ever being handed a
 * bad index.  *failed_lists (may be NULL): bit 0 input pairs, 1 residual rows, 2 transposed HAG, 3 input graph, 4 its
 * transpose, 5 / 6 forward / backward expansion, 7 row orders.  Allocates one word, synchronises the stream.
 * Returns HAG_OK, or HAG_ERR_GRAPH if any bit is set.  Errors: NULL, NOT_ON_DEVICE, OOM_DEVICE, CUDA. */
hag_status hag_device_validate(hag_t *h, uint32_t *failed_lists, void *cuda_stream);

/* Test hook: the two predicates of hag_device_validate evaluated on the host: bit 0 = id lies in [lo, hi), bit 1 =
 * pointer number i of a list of `rows` rows is acceptable (cur == first if i == 0, else cur >= prev; cur == last if
 * i == rows). */
int32_t hag_test_range_predicates(int32_t id, int32_t lo, int32_t hi, int64_t i, int64_t rows, int32_t prev, int32_t cur,
                                  int32_t first, int32_t last);

/* Test hook (process-wide): makes one of the library's next allocation attempts fail as if memory had run out,
 * so that callers can exercise their handling of HAG_ERR_OOM_HOST / HAG_ERR_OOM_DEVICE.  kind 0: host memory
 * (the checked points are the start of the search, of the layout and of every array upload), 1: device memory
 * (every array upload of hag_to_device).  countdown 0 fails the next attempt, 1 the one after it, ...; a
 * negative value switches the hook off.  The failing call frees what it had built and returns the status;
 * nothing is left half-made, and no GPU work is involved.  Errors: ARG (kind). */
hag_status hag_test_fail_allocation(int32_t kind, int32_t countdown);

/* Number of kernels the last aggregate call on this handle enqueued. */
int32_t hag_last_launch_count(const hag_t *h);

const char *hag_status_str(hag_status s);

#ifdef __cplusplus
}
#endif
#endif /* HAG_B200_H */
