/* ripple.h -- C ABI of the B200-native incremental GNN inference library.
 *
 * The library keeps, resident on one GPU, a dynamic directed graph, the vertex features H^0 and
 * the cached per-layer embeddings H^1..H^L of an L-layer GNN -- with a linear aggregator, or,
 * hybrid-incrementally, with max / min or attention layers (Sec. 3.4) -- and brings them up to
 * date after each batch of updates by incremental propagation: only the vertices of the L-hop
 * propagation tree of the batch are touched, and the result equals full layer-wise inference on
 * the updated graph (RIPPLE++, Sec. 3.1 and Sec. 3.3).  ripple_part.h holds the calls of the
 * partitioned execution over several GPUs (Sec. 4).
 *
 * Conventions
 *   - Edge (u, v): u is the source, v the sink; v aggregates over its in-neighbours (Eq. 1).
 *   - The vertex ids are {0..N-1}, N a capacity given at creation that ripple_reserve_vertices
 *     can raise.  The graph is simple and directed; a self-loop is an ordinary edge.
 *   - All matrices are fp32, row-major.  Device matrices returned by the library have a leading
 *     dimension `ld` >= width (a multiple of 4 floats); columns beyond the width hold zeros.
 *   - Pointers marked HOST must be dereferenceable by the CPU, DEVICE by the GPU the context
 *     lives on; pointers marked HOST|DEVICE are accompanied by a `ripple_mem` flag.
 *   - The caller owns every buffer it passes in; the library copies what it keeps.  Pointers
 *     handed out by the library are borrowed and stay valid until the next ripple_apply_batch,
 *     ripple_recompute_full, ripple_reserve_vertices or ripple_destroy on the same context.
 *   - Every call returns a ripple_status; nothing aborts or traps.  After a non-zero status,
 *     ripple_last_error() describes it.  A batch that is rejected leaves graph, features and
 *     embeddings exactly as they were.
 *   - A context is not thread-safe; all of its work runs on the stream given at creation and
 *     each call returns after that stream has finished the call's work.
 */
#ifndef RIPPLE_H
#define RIPPLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RIPPLE_MAX_LAYERS 8

typedef struct ripple_ctx ripple_ctx;

typedef enum {
    RIPPLE_OK = 0,
    RIPPLE_ERR_INVALID_ARG = 1,  /* null pointer, bad enum, bad dimension, unknown op code       */
    RIPPLE_ERR_VERTEX_RANGE = 2, /* a vertex id outside [0, N) or a payload row outside range    */
    RIPPLE_ERR_CAPACITY = 3,     /* batch larger than max_batch, or overflow edge pool exhausted  */
    RIPPLE_ERR_OOM = 4,          /* device allocation failed                                     */
    RIPPLE_ERR_CUDA = 5,         /* a CUDA runtime call failed                                   */
    RIPPLE_ERR_TIMEOUT = 6       /* a bounded device-side wait gave up; destroy the context      */
} ripple_status;

typedef enum { RIPPLE_MEM_HOST = 0, RIPPLE_MEM_DEVICE = 1 } ripple_mem;

/* Aggregators of Table 1.  WSUM_GCN is the weighted sum with alpha_uv = 1/sqrt(deg_out(u) deg_in(v))
 * taken from the current graph and recomputed whenever a degree changes.
 * MAX, MIN (Sec. 3.4.2, monotonic aggregation): element-wise maximum / minimum over the in-neighbours,
 * zeros for a vertex without in-neighbours; GRAPHCONV and SAGE layers.  Its batches run hybrid-incrementally:
 * a message carries the sender's old and new row, a sink raises its cached maximum, recomputes it
 * over all in-neighbours, or ignores the message; a sink whose cached maximum did not change is
 * not affected and propagates nothing (ripple_get_affected then lists exactly the vertices whose
 * cached maximum changed -- for SAGE also those whose own previous-layer row changed;
 * ripple_stats.senders those whose embedding changed).
 * WSUM_EDGE: the weighted sum of Table 1 with a stored weight alpha_uv per edge (the GC-W workload of
 * Sec. 6.1.1): x_v = sum over in-neighbours u of alpha_uv h_u, no normalisation.  Weights are static:
 * an edge takes its weight when it is created (ripple_graph.weight, or the per-operation weights of
 * ripple_apply_batch_weighted) and keeps it for as long as it exists at batch boundaries -- adding an
 * edge that exists is a counted no-op whatever weight comes with it.  Messages along an edge are scaled
 * by its weight (Sec. 3.3.3, "other linear aggregators"). */
typedef enum {
    RIPPLE_AGG_SUM = 0, RIPPLE_AGG_MEAN = 1, RIPPLE_AGG_WSUM_GCN = 2, RIPPLE_AGG_MAX = 3, RIPPLE_AGG_MIN = 4,
    RIPPLE_AGG_WSUM_EDGE = 5
} ripple_agg;

/* Update functions (Eq. 2) of the model families of Sec. 6.1.1, x_v = normalised aggregate:
 *   SAGE       h = act(Wa^T h_v + Wb^T x_v + ba)                         (self term)
 *   GRAPHCONV  h = act(Wa^T x_v + ba)                                    (no self term)
 *   GIN        h = act(Wb^T relu(Wa^T ((1 + eps) h_v + x_v) + ba) + bb)  (self term)
 * and the attention layer of Sec. 3.4.1 (Eq. 3), which takes the hybrid-incremental path:
 *   GAT        h = act(sum over in-neighbours u of alpha_uv h_u),  alpha_uv = softmax over In(v) of z_uv,
 *              z_uv = rect(ba . (Wa^T h_u) + bb . (Wa^T h_v)),  rect(z) = z for z >= 0 and eps * z below
 *              (eps = 1: the linear logit Eq. 3 prints; eps < 1: the leaky rectifier of the architecture it
 *              cites).  ba, bb are the source and sink halves of Eq. 3's vector a.  d_out = d_in; a vertex
 *              without in-neighbours outputs zeros; agg must be RIPPLE_AGG_SUM (it is not read).
 *              A vertex whose own row changed at hop l-1 is a hop-l vertex and gathers its sums anew there;
 *              every other hop-l vertex is updated by <numerator, denominator> messages.
 *              ripple_get_aggregate: width d_in + 1, columns 0..d_in-1 the numerator sum_u exp(z_uv) h_u,
 *              column d_in the denominator sum_u exp(z_uv). */
typedef enum { RIPPLE_LAYER_SAGE = 0, RIPPLE_LAYER_GRAPHCONV = 1, RIPPLE_LAYER_GIN = 2, RIPPLE_LAYER_GAT = 3 } ripple_layer_kind;

typedef enum { RIPPLE_ACT_IDENTITY = 0, RIPPLE_ACT_RELU = 1 } ripple_act;

/* The update types of Sec. 3.1.  Vertex ids live in [0, num_vertices) for the life of the context:
 * num_vertices is a capacity.
 *   - Vertex deletion (Sec. 3.2): DEL_VERTEX removes, at its position in the batch, every edge
 *     that has u as an endpoint and replaces u's feature row by zeros; propagation starts from u
 *     as root (the sinks of the removed edges and u itself are affected).  The id stays valid.
 *   - Vertex addition arrives, as in Sec. 4.1, as the edge addition that first names an unused
 *     id (plus a SET_FEATURE for its row); an unused id is an isolated vertex with a zero row. */
typedef enum {
    RIPPLE_OP_ADD_EDGE = 0, RIPPLE_OP_DEL_EDGE = 1, RIPPLE_OP_SET_FEATURE = 2, RIPPLE_OP_DEL_VERTEX = 3
} ripple_op;

/* One update.  ADD_EDGE / DEL_EDGE: edge (u, v).  SET_FEATURE: vertex u takes row `v` of the
 * batch's feature payload.  DEL_VERTEX: vertex u (v is ignored). */
typedef struct {
    int32_t op;
    int32_t u;
    int32_t v;
} ripple_update;

/* Initial graph in coordinate form: num_edges distinct pairs (src[i], dst[i]), any order.
 * src / dst / weight: HOST|DEVICE per `mem`.  Duplicate pairs are not allowed (not checked).
 * weight: one fp32 weight per edge, read for RIPPLE_AGG_WSUM_EDGE only (NULL there: all ones). */
typedef struct {
    int64_t num_vertices;
    int64_t num_edges;
    const int32_t* src;
    const int32_t* dst;
    int32_t mem; /* ripple_mem */
    const float* weight;
} ripple_graph;

/* One layer.  Matrices are input-major: Wa[k * cols + j] multiplies input k into output j.
 *   SAGE:      Wa = W_self (d_in x d_out), Wb = W_neigh (d_in x d_out), ba (d_out)
 *   GRAPHCONV: Wa (d_in x d_out), ba (d_out)
 *   GIN:       Wa (d_in x d_hidden), ba (d_hidden), Wb (d_hidden x d_out), bb (d_out)
 *   GAT:       Wa = W (d_in x d_hidden), ba = a_src (d_hidden), bb = a_dst (d_hidden), all required; eps = slope
 * All HOST pointers; biases may be NULL (zero).  d_in of layer l must equal d_out of layer l-1. */
typedef struct {
    int32_t kind; /* ripple_layer_kind */
    int32_t d_in;
    int32_t d_hidden;
    int32_t d_out;
    int32_t act; /* ripple_act */
    float eps;
    const float* Wa;
    const float* Wb;
    const float* ba;
    const float* bb;
} ripple_layer;

/* How hop l brings the cached aggregates S^l up to date.  PUSH / PULL: delta messages (Sec. 3.3.1),
 * scattered along the senders' out-edges or gathered per affected sink.  REGATHER: the aggregates
 * of the affected vertices are rebuilt from their in-lists (the scoped recomputation of Sec. 3.2,
 * for this hop only).  AUTO: PUSH, except that a hop whose senders own at least
 * regather_threshold of all edges rebuilds, and that a hop of wide messages (128 floats or more)
 * from few senders gathers per sink (chosen per hop from what the hop carried in the batch before:
 * at least 2^20 messages, eight or more per affected sink, sender rows of at most 32 MiB in all;
 * the environment variable RIPPLE_GATHER_MIN_WIDTH, read by ripple_create, replaces the 128: 0 = never). */
typedef enum {
    RIPPLE_SCATTER_AUTO = 0, RIPPLE_SCATTER_PUSH = 1, RIPPLE_SCATTER_PULL = 2, RIPPLE_SCATTER_REGATHER = 3,
    RIPPLE_SCATTER_PUSH_BULK = 4 /* PUSH with one bulk reduction of the copy engine per message (cp.reduce.async.bulk)
                                    instead of 16-byte vector reductions; measured equally fast */
} ripple_scatter_mode;
typedef enum { RIPPLE_GEMM_AUTO = 0, RIPPLE_GEMM_FP32 = 1, RIPPLE_GEMM_TF32 = 2 } ripple_gemm_mode;

/* Zero-initialise for defaults. */
typedef struct {
    double slack;         /* spare adjacency capacity per vertex as a fraction of its degree (default 0.25) */
    int64_t pool_edges;   /* overflow pool size per direction, in edges (default max(E/4, 1<<20))           */
    int64_t max_batch;    /* largest n accepted by ripple_apply_batch (default 16384)                       */
    int32_t scatter_mode; /* ripple_scatter_mode: how delta messages reach the aggregates                   */
    int32_t gemm_mode;    /* ripple_gemm_mode: arithmetic of the affected-row layer update                  */
    int32_t timing;       /* non-zero: record per-stage CUDA-event times into ripple_stats                  */
    int32_t pre_transform;/* 0: a layer not wider than its input applies its neighbour matrix to the sender
                             rows before the scatter (messages and the cached aggregate then have the
                             layer's output width; for equal widths only where nothing but that product
                             would be left per affected row: SAGE, GRAPHCONV); 1: never, aggregates
                             always hold input-width rows                                                */
    int32_t no_graphs;    /* non-zero: never replay small batches (<= 512 updates; a batch size is captured
                             the second time it is seen) as a CUDA graph                                  */
    int32_t device;       /* CUDA device ordinal, or -1 for the current device                              */
    void* stream;         /* cudaStream_t to run on (NULL: the library creates its own)                     */
    float regather_threshold; /* AUTO only: a hop rebuilds its aggregates once its messages number at least
                             this share of all edges.  0: default (0.5 for aggregate rows of 128 floats
                             or more, else 0.55, and never for hops of fewer than 4 Mi messages,
                             where pushing is as fast); < 0: never                       */
    float rebuild_budget; /* A cached aggregate row is updated by one fp32 addition per batch, and each
                             addition rounds at the magnitude the row has at that moment.  The library
                             adds these roundings up per row (as a sum of squares, in units of one
                             rounding of the row's largest entry) and gathers the row anew from its
                             in-list once the total exceeds rebuild_budget roundings of the row's
                             present largest entry: a row that keeps its size is gathered anew every
                             rebuild_budget^2 batches that touch it, a row that lost a large term (an
                             edge from a hub deleted) at once.  0: default (8); < 0: never.  Applies to
                             aggregates of input-width rows and to all aggregates of the unnormalised
                             sums (RIPPLE_AGG_SUM, RIPPLE_AGG_WSUM_EDGE).                                 */
    int32_t n_local;      /* > 0: the context is one worker of a partitioned execution (ripple_part.h): ids
                             below n_local (a multiple of 32) are its own vertices, the rest halo slots    */
} ripple_options;

typedef struct {
    int32_t num_layers;
    int64_t num_edges;                            /* after the last batch                                 */
    int64_t n_ops, n_added, n_deleted;            /* last batch: ops given, net edges added / deleted     */
    int64_t n_noop_add, n_noop_del, n_superseded; /* add-existing, delete-missing, shadowed by a later op */
    int64_t n_feature;                            /* distinct vertices with a feature update              */
    int64_t affected[RIPPLE_MAX_LAYERS + 1];      /* |A_l|, l = 0..L                                      */
    int64_t senders[RIPPLE_MAX_LAYERS + 1];       /* |C_l|: vertices whose outgoing message changed       */
    int64_t active_edges[RIPPLE_MAX_LAYERS + 1];  /* l = 1..L: edges carrying a message at hop l          */
    int32_t scatter_pull[RIPPLE_MAX_LAYERS + 1];  /* l = 1..L: 0 pushed, 1 gathered per sink, 2 rebuilt  */
    int64_t in_edges[RIPPLE_MAX_LAYERS + 1];      /* l = 1..L: in-edges of A_l (what a gather walks)      */
    int32_t message_width[RIPPLE_MAX_LAYERS + 1]; /* l = 1..L: floats per message / aggregate row (padded) */
    int64_t pool_used, pool_size;                 /* overflow pool, out-direction, in edges: handed out so far
                                                     (high-water mark of the never-used part), total size  */
    /* CUDA-event times of the last batch in milliseconds (zero unless options.timing) */
    float ms_total, ms_graph;
    float ms_frontier[RIPPLE_MAX_LAYERS + 1];
    float ms_scatter[RIPPLE_MAX_LAYERS + 1];
    float ms_update[RIPPLE_MAX_LAYERS + 1];
    float ms_scatter_kernel[RIPPLE_MAX_LAYERS + 1]; /* the push or gather kernels alone, l = 1..L           */
    float ms_regather[RIPPLE_MAX_LAYERS + 1];     /* the gather of a rebuilding hop alone, l = 1..L       */
    float ms_bootstrap;                           /* last ripple_create / ripple_recompute_full           */
    int64_t gpu_launches;                         /* kernels launched by the last call                    */
    int64_t n_expanded;                           /* last batch: edge deletions generated by vertex deletions */
    int64_t rows_rebuilt[RIPPLE_MAX_LAYERS + 1];  /* l = 1..L: aggregate rows gathered anew because their
                                                     rounding budget ran out (ripple_options.rebuild_budget) */
    int64_t pool_free, pool_lost;                 /* out-direction, in edges: room in vacated blocks (of the pool or
                                                     of the initial layout) that waits for reuse; room that cannot
                                                     be reused (tails beyond a block's power-of-two part, blocks
                                                     dropped because a free list was full)                       */
} ripple_stats;

/* Sec. 3.1 (preliminaries): the bootstrap embeddings exist before updates arrive.  Builds the
 * device graph store from `g`, copies `features` (N x d0, HOST|DEVICE per feat_mem, row-major,
 * leading dimension d0) and the L layers, runs full layer-wise inference (Eq. 1-2) to fill
 * H^1..H^L and the cached aggregates, and returns the context in *out.  On failure *out = NULL;
 * for statuses other than INVALID_ARG the text is available from ripple_last_error(NULL). */
ripple_status ripple_create(const ripple_graph* g, const float* features, int32_t feat_mem,
                            const ripple_layer* layers, int32_t L, int32_t agg,
                            const ripple_options* opt, ripple_ctx** out);

/* Sec. 3.1 (batched updates) and Sec. 3.3 (apply, then propagate hop by hop).  Applies ups[0..n)
 * in order (the last operation on a pair, and the last payload of a vertex, win; adding an
 * existing edge or deleting a missing one is counted and ignored), then propagates the changes
 * through all L layers.  ups and feat_rows (n_rows x d0, leading dimension d0) are HOST|DEVICE
 * per `mem`.  Returns after the embeddings are up to date.  n = 0 is valid.
 * A DEL_VERTEX is expanded on the device into one DEL_EDGE per incident edge; the given and the
 * generated operations together must not exceed max_batch (else CAPACITY, nothing is changed).
 * An explicit operation on an edge of u that precedes DEL_VERTEX(u) is superseded by it; one that
 * follows it acts on the emptied vertex.  Only the given operations are counted in n_superseded
 * and the no-op counters; edges removed by a vertex deletion are counted in n_deleted. */
ripple_status ripple_apply_batch(ripple_ctx* ctx, const ripple_update* ups, int64_t n,
                                 const float* feat_rows, int64_t n_rows, int32_t mem);

/* The same for a graph with stored edge weights (RIPPLE_AGG_WSUM_EDGE): edge_weights holds one fp32
 * weight per operation (HOST|DEVICE per `mem`, n entries), read only where ups[i] is an ADD_EDGE that
 * creates its edge.  NULL: every new edge gets weight 1. */
ripple_status ripple_apply_batch_weighted(ripple_ctx* ctx, const ripple_update* ups, int64_t n,
                                          const float* feat_rows, int64_t n_rows, const float* edge_weights,
                                          int32_t mem);

/* Sec. 3.1: updated predictions are available right after the batch.  *dev_ptr: DEVICE pointer
 * to H^layer (N x *ld), layer in 0..L. */
ripple_status ripple_get_embeddings(ripple_ctx* ctx, int32_t layer, const float** dev_ptr, int64_t* ld);

/* The cached un-normalised aggregate S^layer (the persistent inbox of Sec. 3.3.2):
 * S_v = sum over in-neighbours u of c_u h^{layer-1}_u, or, if *transformed is set, of
 * c_u W_n^T h^{layer-1}_u with W_n the layer's neighbour matrix (Wb for SAGE, Wa otherwise); see
 * ripple_options.pre_transform.  DEVICE, N x *ld with *width meaningful columns, layer in 1..L.
 * width and transformed may be NULL. */
ripple_status ripple_get_aggregate(ripple_ctx* ctx, int32_t layer, const float** dev_ptr, int64_t* ld,
                                   int32_t* width, int32_t* transformed);

/* Trigger-based inference (Sec. 2.2): the vertices whose H^layer the last batch recomputed --
 * hop `layer` of the propagation tree (Sec. 3.3) -- as ascending ids.  DEVICE, layer in 0..L. */
ripple_status ripple_get_affected(ripple_ctx* ctx, int32_t layer, const int32_t** dev_ids, int64_t* count);

/* Current graph in canonical CSR over out-edges: rowptr (HOST, N + 1 entries), col (HOST,
 * col_capacity >= number of edges, ascending within each row).  For parity checks. */
ripple_status ripple_export_graph(ripple_ctx* ctx, int64_t* rowptr, int32_t* col, int64_t col_capacity);

/* ripple_export_graph plus the stored weight of every edge, in the order of col (HOST, col_capacity
 * entries; all ones unless the aggregator is RIPPLE_AGG_WSUM_EDGE). */
ripple_status ripple_export_graph_weighted(ripple_ctx* ctx, int64_t* rowptr, int32_t* col, float* weight,
                                           int64_t col_capacity);

/* The same canonical CSR as ripple_export_graph, for callers that must not allocate device
 * memory.  (The paper has no counterpart: this is a property of this library, not of the method.)
 * Who needs it: a process whose framework has already claimed all device memory for its own
 * caching allocator, so that a cudaMalloc from this library would fail or force the framework to
 * give memory back; or a caller on a latency budget that cannot afford the device-wide
 * synchronisation an allocation or a free may imply.  ripple_export_graph obtains its staging
 * buffers (a device copy of the row pointers and a packed copy of the column indices) with
 * cudaMalloc on every call; this variant keeps them in fixed device arrays inside the library,
 * about 10 MB that every GPU loading the library holds until the process exits, and calls no
 * allocator at all.
 * Limits: at most 262 144 vertices and 2 097 152 edges; a larger graph is rejected with
 * RIPPLE_ERR_CAPACITY and the text says which limit was hit.
 * The first call on each device looks up the addresses of the fixed arrays (a one-time set-up
 * with that device current); make that first call before any stream capture begins.
 * All calls on a device share the arrays, which keep whatever the previous call left in them
 * (every call overwrites the part it reads, so nothing needs clearing); two calls whose GPU work
 * overlaps -- from two contexts or two threads -- race on them: serialise such calls.
 * Arguments, outputs and ordering are those of ripple_export_graph: rowptr HOST, N + 1 entries;
 * col HOST, col_capacity >= number of edges, ascending within each row. */
ripple_status ripple_export_graph_static(ripple_ctx* ctx, int64_t* rowptr, int32_t* col, int64_t col_capacity);

/* Vertex addition beyond the ids the context was created with (Sec. 3.2, Sec. 4.1: a vertex arrives with
 * the edge addition that first names it): raises the id capacity to num_vertices.  The new ids are isolated
 * vertices with zero feature rows; their embeddings are those full inference gives an isolated vertex
 * (the activation of the bias, layer by layer), everything else keeps its bits.  Every device array that
 * has a row per vertex is re-allocated and copied: pointers obtained earlier from ripple_get_embeddings,
 * ripple_get_aggregate, ripple_get_affected and ripple_get_degrees are invalid afterwards, captured launch
 * chains are dropped, and the call costs a copy of the whole state -- reserve in large steps.
 * INVALID_ARG if num_vertices is not larger than the present capacity or the context is a worker of a
 * partitioned execution; OOM leaves the context unusable (destroy it). */
ripple_status ripple_reserve_vertices(ripple_ctx* ctx, int64_t num_vertices);

/* Degree arrays of the current graph: DEVICE, N entries each. */
ripple_status ripple_get_degrees(ripple_ctx* ctx, const int32_t** deg_out, const int32_t** deg_in);

/* Full layer-wise inference (Eq. 1-2) over the current graph, overwriting all cached state: the
 * recompute-everything alternative that incremental propagation is compared against. */
ripple_status ripple_recompute_full(ripple_ctx* ctx);

/* Counters and timings of the last batch (HOST struct, filled by the call). */
ripple_status ripple_get_stats(ripple_ctx* ctx, ripple_stats* out);

/* Switches the per-stage CUDA-event timing of ripple_stats on or off.  While it is on, small
 * batches are launched kernel by kernel instead of as a captured graph. */
ripple_status ripple_set_timing(ripple_ctx* ctx, int32_t on);

/* Text of the last error on ctx (or of the last failed ripple_create if ctx is NULL). */
const char* ripple_last_error(ripple_ctx* ctx);

void ripple_destroy(ripple_ctx* ctx);

/* Diagnostic for the roofline of the push scatter (the paper has no counterpart): issues n_messages
 * rows of row_floats floats (a multiple of 4) as 16-byte vector reductions, red.global.add.v4.f32,
 * into rows of a zeroed scratch window of n_rows rows, and returns the best of three timed passes in
 * *ms_out (HOST).  pattern 0: uniformly random rows; 1: consecutive rows (the best case of the
 * reduction path); 2: random rows with a popular head (position = u^3 of the window, u uniform).
 * A window that fits L2 gives the ceiling of the on-chip reduction path, a window of the size of an
 * aggregate matrix the rate with DRAM behind it.
 * Allocates and frees its own scratch on `device` (-1: current); touches no context. */
ripple_status ripple_probe_reduction_rate(int32_t device, int64_t n_rows, int32_t row_floats,
                                          int64_t n_messages, int32_t pattern, float* ms_out);

/* Diagnostic for the roofline of the gathering kernels (bootstrap aggregation, rebuilding hops; the
 * paper has no counterpart): reads n_gathers whole rows of row_floats floats (a multiple of 4) from
 * pseudo-random places of a zeroed scratch window of n_rows rows, eight rows in flight per warp, and
 * returns the best of three timed passes in *ms_out (HOST).  Index arithmetic only, no index array: the
 * rate is what the device's memory system gives a row gather at best -- from L2 if the window fits
 * there, from L2 and DRAM otherwise.  Allocates and frees its own scratch on `device` (-1: current). */
ripple_status ripple_probe_gather_rate(int32_t device, int64_t n_rows, int32_t row_floats,
                                       int64_t n_gathers, float* ms_out);

/* Library version string. */
const char* ripple_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RIPPLE_H */
