/* Partitioned execution of the ripple library over several GPUs (Sec. 4 of the paper): one context
 * per GPU holds one vertex partition, the update stream is routed by a replicated router, and every
 * hop ends with one exchange of combined halo messages.
 *
 * How Sec. 4 maps onto this library
 *   worker (Sec. 4.2)      one ripple_ctx created with ripple_options.n_local > 0.  Its vertex ids are
 *                          LOCAL ids: [0, n_local) are the partition's own vertices (embeddings, cached
 *                          aggregates, adjacency in both directions, including the cut edges that end
 *                          or start at them), [n_local, num_vertices) are halo slots: remote endpoints
 *                          of cut edges.  A halo slot holds no embedding; its row of the per-batch
 *                          message accumulator is the halo mailbox in which the partition's messages
 *                          for that remote vertex are combined (the combiner of Sec. 4.2).
 *   remote send (Sec. 4.5) ripple_part_hop_send: after the local sends of a hop one kernel adds every
 *                          marked halo mailbox into the owner's accumulator row through a peer pointer
 *                          (16-byte vector reductions over NVLink, each combined row crosses once), marks
 *                          the vertex in the owner's frontier bitmap and clears the mailbox.  The owner
 *                          folds what arrived together with its local messages: the receiver-side
 *                          aggregation.  No kernel waits for another GPU; the caller separates
 *                          ripple_part_hop_send from ripple_part_hop_compute by a barrier over all
 *                          workers (the paper's "next hop starts only after ... messages are delivered").
 *   server (Sec. 4.3, 4.4) ripple_router: vertex-partition map, high in-degree set, routing of updates
 *                          (an edge goes to its source's worker, with a no-compute copy to the sink's
 *                          worker when that is another one), placement of new vertices by Alg. 1 or by
 *                          hashing, global-to-local id translation and halo slot assignment.  Host code;
 *                          every worker process runs its own replica on the same stream, so no server
 *                          process and no routing messages exist.
 *
 * What a partitioned context supports: the linear aggregators SUM, MEAN, WSUM_GCN and WSUM_EDGE (stored edge
 * weights: a cut edge keeps its weight at both workers) with SAGE, GRAPHCONV and GIN layers; edge additions, edge deletions and feature replacements (the router turns a vertex
 * deletion into these; a worker given one answers RIPPLE_ERR_INVALID_ARG).  Hops always take the delta
 * form (push); the rounding budget is off (a row cannot be gathered anew without its remote
 * in-neighbours' rows).  ripple_apply_batch and ripple_recompute_full are refused on such a context.
 *
 * Peer memory: ripple_part_exports_get returns the device addresses a peer needs.  Workers that share a
 * process exchange them directly; workers in different processes turn them into CUDA IPC handles with
 * ripple_part_ipc_export / ripple_part_ipc_open.  Only plain peer loads, stores and reductions are issued
 * on peer memory (no multicast, no bulk-tensor copies).
 */
#ifndef RIPPLE_PART_H
#define RIPPLE_PART_H

#include "ripple.h"

#ifdef __cplusplus
extern "C" {
#endif

#define RIPPLE_MAX_PEERS 16

/* Device addresses of one worker's state that its peers write to or read from (DEVICE pointers; for
 * l = 0..L where they exist, else NULL).  accumulator[l]: the per-batch message accumulator of hop l
 * (num_vertices x accumulator_ld[l] floats); embeddings[l]: H^l (num_vertices x embeddings_ld[l]);
 * frontier_bitmap: one bit per local id; out_degrees: int32 per local id (read during the bootstrap of
 * RIPPLE_AGG_WSUM_GCN, whose source coefficient needs a remote in-neighbour's whole out-degree). */
typedef struct {
    void* accumulator[RIPPLE_MAX_LAYERS + 1];
    int64_t accumulator_ld[RIPPLE_MAX_LAYERS + 1];
    void* embeddings[RIPPLE_MAX_LAYERS + 1];
    int64_t embeddings_ld[RIPPLE_MAX_LAYERS + 1];
    void* frontier_bitmap;
    void* out_degrees;
    int64_t num_vertices;   /* local ids of the worker: a halo slot that names a larger one is refused */
} ripple_part_exports;

/* Opaque handles of the same buffers for another process (CUDA IPC). */
typedef struct {
    unsigned char accumulator[RIPPLE_MAX_LAYERS + 1][64];
    unsigned char embeddings[RIPPLE_MAX_LAYERS + 1][64];
    unsigned char frontier_bitmap[64];
    unsigned char out_degrees[64];
    int64_t accumulator_ld[RIPPLE_MAX_LAYERS + 1];
    int64_t embeddings_ld[RIPPLE_MAX_LAYERS + 1];
    int64_t num_vertices;
    int32_t num_layers;
} ripple_part_ipc;

/* ---- worker ------------------------------------------------------------------------------------
 * A partitioned context is created by ripple_create with options.n_local > 0 (a multiple of 32): the
 * graph is given in local ids and holds every edge with a local endpoint; features are given for all
 * num_vertices rows (halo rows are ignored).  ripple_create does NOT run the bootstrap inference
 * for such a context: call ripple_part_bootstrap_layer for l = 1..L on every worker, with a barrier over
 * all workers between two layers. */

ripple_status ripple_part_exports_get(ripple_ctx* ctx, ripple_part_exports* out);

/* Registers peer `rank`'s buffers (its own rank included is allowed and ignored).  e: HOST struct of
 * DEVICE addresses valid in this process. */
ripple_status ripple_part_set_peer(ripple_ctx* ctx, int32_t rank, const ripple_part_exports* e);

/* CUDA IPC: handles of this worker's buffers for other processes / open another process's handles and
 * register them as peer `rank`.  The mappings are closed by ripple_destroy. */
ripple_status ripple_part_ipc_export(ripple_ctx* ctx, ripple_part_ipc* out);
ripple_status ripple_part_ipc_open(ripple_ctx* ctx, int32_t rank, const ripple_part_ipc* in);

/* Halo slots first .. first + count - 1 (slot h is local id n_local + h) stand for vertex remote_id[h]
 * (a LOCAL id of worker owner[h]).  HOST arrays.  Slots are assigned once and never change. */
ripple_status ripple_part_set_halos(ripple_ctx* ctx, int32_t first, int32_t count, const int32_t* owner,
                                    const int32_t* remote_id);

/* Layer-wise inference of layer l (Eq. 1-2 on the graph as it stands): fetches H^{l-1} of every assigned
 * halo slot from its owner (peer loads), then computes the cached aggregates and H^l of all local
 * vertices.  Returns when done.  Every worker must have finished layer l - 1 before any worker starts
 * layer l.  Run for l = 1..L after ripple_create, it is the bootstrap; run again for l = 1..L between
 * two batches (no phase of a batch outstanding on any worker), it recomputes every cached row from the
 * current graph and features, which also discards the rounding that incremental additions have left
 * in the cached sums (a partitioned context has no per-row rebuild of its own: the rows of a vertex's
 * remote in-neighbours are not resident). */
ripple_status ripple_part_bootstrap_layer(ripple_ctx* ctx, int32_t l);

/* One batch, in phases (Sec. 4.5).  ups / feat_rows / no_compute / edge_weights as in ripple_apply_batch_weighted
 * (HOST|DEVICE per mem), in local ids; no_compute[i] != 0 marks the copy of a cut edge that the SINK's worker
 * receives: it updates the adjacency and the degrees and sends nothing (may be NULL: none); edge_weights[i] is the
 * weight of the edge that operation i adds (RIPPLE_AGG_WSUM_EDGE only; NULL: ones).
 *   begin        Apply: normalise the batch, mutate the partition, replace features, list hop-0 senders
 *   hop_send     l = 1..L: prepare + local send + combine, then the remote send of the halo mailboxes
 *   hop_compute  l = 1..L: aggregate what arrived, update the local hop-l vertices, list the next senders
 *   end          clean up; ripple_get_stats / ripple_get_affected then describe this worker's share
 * Each call returns when its device work is done.  Between hop_send(l) and hop_compute(l) every worker
 * must have returned from hop_send(l); between hop_compute(l) and hop_send(l + 1) no barrier is needed.
 * A batch rejected by begin (status != OK) must not be followed by the other phases. */
ripple_status ripple_part_begin(ripple_ctx* ctx, const ripple_update* ups, int64_t n, const float* feat_rows,
                                int64_t n_rows, const uint8_t* no_compute, const float* edge_weights, int32_t mem);
ripple_status ripple_part_hop_send(ripple_ctx* ctx, int32_t l);
ripple_status ripple_part_hop_compute(ripple_ctx* ctx, int32_t l);
ripple_status ripple_part_end(ripple_ctx* ctx);

/* Halo rows this worker sent at hop l of the last batch (after combining), l = 1..L.  HOST array of
 * RIPPLE_MAX_LAYERS + 1 entries. */
ripple_status ripple_part_rows_sent(ripple_ctx* ctx, int64_t* out);

/* ---- router (host code; Sec. 4.3, 4.4, Alg. 1) --------------------------------------------------- */
typedef struct ripple_router ripple_router;

typedef enum { RIPPLE_ROUTE_LOCALITY = 0, RIPPLE_ROUTE_HASH = 1 } ripple_routing;

/* owner[v] in [0, P) for the vertices of the initial graph, -1 for ids that no edge has named yet (they
 * are placed when an edge addition first names them).  src / dst: the initial edges in global ids.
 * spare_local: local ids kept free per worker for vertices placed later; halo_capacity: halo slots per
 * worker.  hd_refresh: the high in-degree set (in-degree above twice the average degree) is rebuilt after
 * every hd_refresh routed updates.  All HOST. */
ripple_status ripple_router_create(int32_t n_partitions, int64_t num_vertices, const int32_t* owner,
                                   int64_t num_edges, const int32_t* src, const int32_t* dst, int32_t routing,
                                   int64_t hd_refresh, int64_t spare_local, int64_t halo_capacity,
                                   ripple_router** out);
void ripple_router_destroy(ripple_router* r);

/* Shape of worker `rank`'s initial partition: n_local (a multiple of 32, spare ids included),
 * num_vertices of its context (n_local + halo_capacity), edges it holds, halo slots in use. */
ripple_status ripple_router_partition_shape(ripple_router* r, int32_t rank, int64_t* n_local,
                                            int64_t* num_vertices, int64_t* num_edges, int64_t* halos_used);

/* The partition itself, in local ids: src_local / dst_local (num_edges entries), edge_of (num_edges entries,
 * may be NULL: the index, in the arrays given to ripple_router_create, of the edge behind each local edge --
 * for per-edge data such as stored weights), global_of (num_vertices entries: the global id behind every
 * local id, -1 for unused ones), halo_owner / halo_remote_id (halos_used entries, for ripple_part_set_halos). */
ripple_status ripple_router_partition_fill(ripple_router* r, int32_t rank, int32_t* src_local, int32_t* dst_local,
                                           int64_t* edge_of, int32_t* global_of, int32_t* halo_owner,
                                           int32_t* halo_remote_id);

/* Routes a batch given in global ids.  Afterwards, per worker, ripple_router_batch_shape gives the
 * number of operations, payload rows and halo slots assigned by this batch, and ripple_router_batch_fill
 * the operations in local ids (in batch order), their no-compute flags, for every operation the position in
 * the routed batch of the operation it comes from (op_of, may be NULL: for per-operation data such as edge
 * weights), for every payload row of the worker the index of the global payload row it is a copy of, and
 * the new halo slots (first slot index in *first_halo).  A payload row index of -1 in row_of stands for a row of zeros.
 * A vertex deletion (Sec. 4.3 routes it to the owner and says no more) is replaced, at its position in the
 * batch, by one edge deletion per incident edge -- the router keeps the edge lists for this -- each routed
 * like any edge deletion, and a feature update of the vertex with a row of zeros; the workers never see
 * a vertex deletion.  RIPPLE_ERR_INVALID_ARG (an unknown op code) and
 * RIPPLE_ERR_VERTEX_RANGE are found before anything changes.  RIPPLE_ERR_CAPACITY (a worker ran out of
 * local ids or halo slots) and RIPPLE_ERR_INVALID_ARG for a feature update of a vertex that is not placed
 * are found while routing: the batch is then partly routed and the router must be destroyed. */
ripple_status ripple_router_route(ripple_router* r, const ripple_update* ups, int64_t n);
ripple_status ripple_router_batch_shape(ripple_router* r, int32_t rank, int64_t* n_ops, int64_t* n_rows,
                                        int64_t* n_new_halos);
ripple_status ripple_router_batch_fill(ripple_router* r, int32_t rank, ripple_update* ups_local, uint8_t* no_compute,
                                       int32_t* op_of, int32_t* row_of, int32_t* first_halo, int32_t* halo_owner,
                                       int32_t* halo_remote_id);

/* Look-ups: the global id behind every local id of a worker as of now (global_of: HOST, capacity >= the
 * worker's num_vertices entries, -1 for unused ids); owner and local id of a global vertex (-1: not placed);
 * the global id behind one local id of a worker (-1: unused); whether v is in the high in-degree set;
 * vertices placed on a worker. */
ripple_status ripple_router_global_ids(ripple_router* r, int32_t rank, int32_t* global_of, int64_t capacity);
int32_t ripple_router_owner(ripple_router* r, int32_t v);
int32_t ripple_router_local_id(ripple_router* r, int32_t v);
int32_t ripple_router_global_id(ripple_router* r, int32_t rank, int32_t local_id);
int32_t ripple_router_is_high_degree(ripple_router* r, int32_t v);
int64_t ripple_router_load(ripple_router* r, int32_t rank);

#ifdef __cplusplus
}
#endif
#endif /* RIPPLE_PART_H */
