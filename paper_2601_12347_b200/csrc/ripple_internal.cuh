// Internal declarations shared by the CUDA translation units of the ripple library.
//
// Control flow: the host never learns a frontier size in the middle of a batch.  Every kernel
// reads its work size from a control block in device memory (Ctl) and runs as a grid-stride loop
// over a fixed grid, so a batch is one uninterrupted chain of launches on one stream; the control
// block is copied to pinned host memory once, at the end.
#pragma once

#include <cuda_runtime.h>

#include <stdint.h>
#include <string.h>

#include "../../include/ripple.h"
#include "../../include/ripple_part.h"

#define RP_MAXL RIPPLE_MAX_LAYERS
#define RP_TOMB (-1)
#define RP_GRAPH_MAX_BATCH 512   // batches up to this size replay a captured launch chain
#define RP_GRAPH_SLOTS 8
#define RP_GRAPH_SEEN 32    // recently seen chain keys: a chain is captured at its second appearance
#define RP_POOL_CLASSES 32          // block size classes of the adjacency store: class k holds blocks of 2^k entries
#define RP_POOL_MIN_CLASS 3         // smallest block that is kept for reuse: 8 entries
#define RP_POOL_LIST_CAP 16384      // blocks a class's free list can hold
#define RP_ATT_CHUNK 128            // attention: in-list entries per work item of a recomputation (sizes the item buffer)
#define RP_TINY_BATCH 32            // batches up to this size list their frontiers and senders in one block each
#define RP_TINY_APPLY 4             // ... and up to this size run the whole of Apply in one block (operations are resolved one after the other there)
#define RP_TINY_WORDS 16384         // ... and list a hop's frontier in one block if its bitmap has at most this many words

namespace rp {

// monotonic aggregators (Sec. 3.4.2) take the hybrid-incremental path
inline bool rp_monotonic(int agg) { return agg == RIPPLE_AGG_MAX || agg == RIPPLE_AGG_MIN; }

// ---- device-resident control block -----------------------------------------------------------
struct Ctl {
    int abort;   // set by validation / planning: the batch is rejected, mutate nothing
    int err;     // ripple_status recorded on the device
    int n_ops;   // operations given by the caller
    unsigned long long n_extra;  // edge deletions generated from vertex deletions (they follow the given ops)
    int expand_failed;           // the generated operations did not fit: none of them is used
    int n_vjobs;
    int n_rows;  // payload rows of the batch
    int n_rec;   // net edge changes of the batch (|dE+| + |dE-|)
    int n_add, n_del, n_noop_add, n_noop_del, n_superseded, n_feat;
    int n_grow[2];
    int n_shrink[2];                  // rows left with less than a quarter of their capacity in use: moved to a smaller block
    int grow_demand[2][RP_POOL_CLASSES];   // growing rows per block size class
    int grow_done;                    // blocks of k_grow_rows that have finished (the last one moves the shrinking rows)
    int plan_done;                    // blocks of k_resolve that have finished (the last one plans the row moves)
    unsigned long long pool_need[2];
    // kept across batches:
    unsigned long long pool_next[2];  // next entry of each side's adjacency array that was never handed out
    unsigned long long pool_free[2];  // entries in vacated blocks that wait in the free lists
    unsigned long long pool_lost[2];  // entries that cannot be reused: tails beyond a block's power-of-two part, overflow of a list
    int nA[RP_MAXL + 1];              // |A_l|
    int nC[RP_MAXL + 1];              // |C_l| (A_l plus sources of edge changes when coefficients depend on them)
    unsigned long long E[RP_MAXL + 1];          // out-edges of C_{l-1} (+ edge records): message count of hop l
    unsigned long long pull_work[RP_MAXL + 1];  // in-edges of A_l
    int pull[RP_MAXL + 1];
    int regather[RP_MAXL + 1];        // hop l rebuilds the aggregates of A_l from their in-lists instead of adding deltas
    int n_long[RP_MAXL + 1];          // bottom-up marking: vertices whose long in-list is scanned by a warp
    int n_rebuilt[RP_MAXL + 1];       // aggregate rows of hop l gathered anew because their rounding budget ran out
    int rebuild_items[RP_MAXL + 1];   // (vertex, chunk) work items of the long rows among them
    int max_items[RP_MAXL + 1];       // max / min: (long row, chunk) work items of hop l's recomputation
    int regather_ticket[RP_MAXL + 1]; // rebuilding form: next unassigned position of A_l
    int gather_ticket[RP_MAXL + 1];   // gathering form of the delta scatter: next unassigned position of A_l
    int gather_long_ticket[RP_MAXL + 1];  // ... and next unassigned work item of the long in-lists
    int gather_items[RP_MAXL + 1];    // gathering form of the delta scatter: (sink, chunk) work items of the long in-lists
    long long num_edges;              // current edge count (kept across batches)
    int work_counter[8];              // dynamic work distribution tickets (reset by the consumer)
};

// Start of a batch: everything back to zero except what lives across batches; params[0] = number of
// operations, params[1] = number of payload rows.
__device__ __forceinline__ void d_ctl_reset(Ctl* ctl, const int* params) {
    Ctl z;
    memset(&z, 0, sizeof(Ctl));
    for (int s = 0; s < 2; ++s) {
        z.pool_next[s] = ctl->pool_next[s];
        z.pool_free[s] = ctl->pool_free[s];
        z.pool_lost[s] = ctl->pool_lost[s];
    }
    z.num_edges = ctl->num_edges;
    z.n_ops = params[0];
    z.n_rows = params[1];
    *ctl = z;
}

// One direction of the adjacency: row r holds col[start[r] .. start[r] + deg[r]), capacity cap[r].
// Rows start in the base region; a row that outgrows its slack moves into the overflow pool
// (the tail of the same array) with doubled capacity.
struct Side {
    int32_t* col;
    float* w;          // stored weight of every entry of col (weighted sum with per-edge weights), else null
    int64_t* start;
    int32_t* cap;
    int32_t* deg;
    int64_t col_size;  // base region + pool, entries
    int64_t base_end;  // first pool entry
    // per-row scratch of the batched update (all zero between batches)
    int32_t* cnt_del;
    int32_t* cnt_add;
    int32_t* tick_a;
    int32_t* tick_b;
    int32_t* touch;
    // vacated blocks, by size class: free_blk[k * RP_POOL_LIST_CAP + i], i < free_cnt[k], is the first entry
    // of a block of 2^k entries.  A kernel either takes blocks or returns them, never both.
    int64_t* free_blk;
    int32_t* free_cnt;
};

// One net edge change.  side 0 = out-list of u (stores v), side 1 = in-list of v (stores u).
struct Rec {
    int32_t u, v;
    int32_t sign;        // +1 added, -1 deleted
    int32_t pos[2];      // deleted: slot of the entry inside its row
    int32_t rank[2];     // rank among the row's additions (resp. deletions) of this batch
    int32_t tail_val[2]; // deleted: entry found at tail slot new_deg + rank
    int32_t rep[2];      // 1 for the first record that touched the row
    int32_t deg_out_old; // out-degree of u before the batch
    int32_t silent;      // partitioned execution: the no-compute copy of a cut edge (the sink's worker sends nothing for it)
    float w;             // stored edge weights: weight of the added edge / weight the deleted edge had
    float tail_w[2];     // deleted: weight found at the tail slot
};

// transposed (K contiguous), tf32-split copy of a weight block for the tensor-core layer update
struct TcW {
    float* hi;
    float* lo;
    int k_pad, n_pad;
};

struct LayerDev {
    int kind, d_in, d_hid, d_out, act;
    float eps;
    int ld_in, ld_hid, ld_out;  // padded widths (multiples of 4)
    float* W1;   // SAGE: [W_self; W_neigh] (2 ld_in x ld_out); GRAPHCONV: ld_in x ld_out; GIN: ld_in x ld_hid;
                 // attention: the two logit vectors W a_src, W a_dst (2 x ld_in)
    float* b1;   // ld_out (SAGE, GRAPHCONV) or ld_hid (GIN)
    float* W2;   // GIN: d_hid x ld_out
    float* b2;   // GIN: ld_out
    TcW tc_main; // weights of the affected-row GEMM (GIN: first matrix)
    TcW tc_nbr;  // neighbour matrix, for layers that transform before the scatter
    TcW tc_2;    // GIN: second matrix
    TcW tc_self; // SAGE: self matrix, for the cached self projection
};

struct Ctx {
    int device;
    cudaStream_t stream;
    bool own_stream;
    int N, L, agg;
    bool self_term, src_norm;
    bool weighted;             // every edge carries a stored weight (RIPPLE_AGG_WSUM_EDGE)
    bool attention;            // attention layers (Sec. 3.4.1): S^l rows hold [numerator | denominator]
    int n_local;               // partitioned execution: ids below are this worker's vertices, the rest halo slots (0: not partitioned)
    int32_t* halo_owner;       // per halo slot: owning worker, or -1 while unassigned
    int32_t* halo_rid;         // per halo slot: the vertex's local id at its owner
    uint8_t* silent_dev;       // batch staging: no-compute flag per operation
    int has_silent;
    float* peer_dS[RIPPLE_MAX_PEERS][RP_MAXL + 1];   // peers' message accumulators (device addresses valid here)
    float* peer_H[RIPPLE_MAX_PEERS][RP_MAXL + 1];
    uint32_t* peer_bitmap[RIPPLE_MAX_PEERS];
    int32_t* peer_deg_out[RIPPLE_MAX_PEERS];
    void* ipc_opened[RIPPLE_MAX_PEERS * (2 * (RP_MAXL + 1) + 2)];   // mappings to close
    int n_ipc_opened;
    int32_t* halo_owner_h;     // host copies of the halo table, to check it against the peers' sizes
    int32_t* halo_rid_h;
    int halo_hi;               // halo slots below this index may be assigned
    int halo_dirty;            // the table or the peer set changed since it was last checked
    int64_t peer_n[RIPPLE_MAX_PEERS];   // local ids of every registered worker
    unsigned peer_mask;        // workers whose buffers have been registered
    unsigned halo_owner_mask;  // workers that own at least one assigned halo slot
    unsigned long long* rows_sent;   // device, per hop: halo rows shipped by the last batch
    int part_phase;            // 0 idle, else 1 + the number of phases of the current batch already run
    int part_nb;
    float* opw_dev;            // batch staging: one weight per operation (weighted only)
    int has_opw;               // the batch being applied came with weights
    int64_t E0;
    int64_t max_batch;
    int scatter_mode, gemm_mode, timing;
    int rebuild_armed[RP_MAXL + 1];   // per hop: the rebuilding form is enqueued for this batch (see arm_rebuild)
    int tc_armed;                     // the tensor-core form of the layer update is enqueued for this batch
    int pull_hop[RP_MAXL + 1];        // per hop: the delta scatter of this batch gathers per sink instead of pushing (see arm_rebuild)
    int gather_min_width;             // narrowest message row (floats) whose hop may gather (environment RIPPLE_GATHER_MIN_WIDTH)
    long long gather_min_messages;    // ... if the hop delivered at least this many messages in the batch before
    long long batches_done;
    int last_nb;
    int debug_tc_withhold;   // diagnostic (environment RIPPLE_DEBUG_TC_WITHHOLD=1): see ripple_create
    int pdl;                 // launch with programmatic stream serialisation (off: environment RIPPLE_NO_PDL=1)
    int may_expand;   // the batch being enqueued may hold vertex deletions (always assumed for device batches)
    long long regather_min_messages;   // default threshold only: hops with fewer messages always push
    float regather_threshold[RP_MAXL + 1];  // per hop: share of all edges from which the hop rebuilds its aggregates
    int n_sm;
    LayerDev layer[RP_MAXL + 1];
    int d[RP_MAXL + 1], ld[RP_MAXL + 1];
    Side side[2];
    float* H[RP_MAXL + 1];
    float* S[RP_MAXL + 1];
    float* Z[RP_MAXL + 1];    // cached self projection W_self^T h^{l-1} of SAGE layers (N x ld_l), else null
    uint32_t* bitmap2;         // monotonic aggregation: sinks whose cached maximum must be recomputed
    uint32_t* invmask;         // monotonic aggregation: per vertex, mw words: elements whose maximiser was lost
    int mw;
    int32_t* old_idx;          // monotonic aggregation: sender -> index of its previous row among the rows of A_{l-1}
    float* P[RP_MAXL + 1];    // cached neighbour projection W_n^T h^{l-1} of layers that transform before the scatter (N x ws_l), else null
    float* dS[RP_MAXL + 1];   // per-batch message accumulator, zero outside a batch (same shape as S)
    float* Eb[RP_MAXL + 1];   // per vertex: rounding budget spent on S^l_v since the row was last gathered (see k_fold_deltas), or null
    bool fused_fold[RP_MAXL + 1];   // S^l += dS^l happens inside the row update's epilogue (no budget kept)
    float rebuild_tau2;       // square of the budget, in roundings of the row's largest entry
    float* att_s[RP_MAXL + 1];   // attention: source half of the logit, (W a_src) . h^{l-1}_v, per vertex
    float* att_t[RP_MAXL + 1];   // attention: sink half, (W a_dst) . h^{l-1}_v
    float* att_so;               // attention: source halves the senders of the current hop had before the batch (list order)
    int2* att_items;             // attention: (vertex, in-list chunk) work items of the rows gathered anew
    float* T;          // GIN hidden rows (compact, N x ld_hid)
    float* D[2];       // delta rows, ping-pong (compact, N x max ld)
    float* Dt;         // delta rows after the neighbour transform (compact, N x max inbox width)
    bool pre[RP_MAXL + 1];   // layer applies its neighbour transform before the scatter
    int ws[RP_MAXL + 1];     // row width (floats, padded) of S^l and of hop-l messages
    int32_t* A[RP_MAXL + 1];   // affected lists
    int32_t* Clist[2];         // sender list, ping-pong (A_l followed by extra sources)
    int64_t* coff;             // exclusive prefix of out-degrees over the sender list (+1)
    uint32_t* bitmap;          // N bits
    int n_words;
    int32_t* posmap;           // vertex -> index in the current sender list, or -1
    int32_t* deg_out_old;      // vertex -> out-degree before the batch, or -1
    int32_t* feat_last;        // vertex -> index of its last SET_FEATURE op in the batch, or -1
    // batch staging
    ripple_update* ups_dev;
    float* feat_dev;
    unsigned long long* hkeys; // pair hash table
    unsigned long long* hwin;  // per hash slot: (position in the batch + 1) << 32 | op index of the winning op
    int32_t* op_seq;           // generated ops: position in the batch of the vertex deletion they come from
    int32_t* vdel_seq;         // vertex -> position of its last deletion in the batch, or -1
    int2* vjobs;               // (op index, first generated slot) per vertex deletion
    int32_t* op_slot;
    int hsize;
    Rec* rec;
    int32_t* grow_list[2];
    int32_t* shrink_list[2];
    int64_t* moved_start;      // per moved row (growing rows of both sides, then shrinking rows): the block it left
    int32_t* moved_cap;
    // scan scratch
    int64_t* tile_sums;
    int n_tile_sums;
    int* scan_done;    // blocks of a scan's first kernel that have finished (zero between scans)
    char* stage_host;  // pinned: sizes, operations, weights and payload rows of a small host batch, packed for one copy
    char* stage_dev;
    size_t stage_bytes;
    int packed_now;    // the batch being applied arrived through the packed staging buffer
    int few_rows_form; // the batch being applied is small: its row updates carry the few-row form (see k_update_rows)
    int* params_dev;   // {n_ops, n_rows} of the batch being applied
    int* params_host;  // pinned
    int no_graphs;
    cudaGraphExec_t graph_exec[RP_GRAPH_SLOTS];
    int graph_n[RP_GRAPH_SLOTS];
    int64_t graph_launches[RP_GRAPH_SLOTS];
    int graph_next;
    int seen_key[RP_GRAPH_SEEN];
    int seen_count[RP_GRAPH_SEEN];
    int seen_next;
    Ctl* ctl;        // device
    Ctl* ctl_host;   // pinned
    ripple_stats stats;
    cudaEvent_t ev[4 + 3 * (RP_MAXL + 1) + 2];
    cudaEvent_t ev_sc[2 * (RP_MAXL + 1)];  // tight brackets around each hop's main scatter kernel
    cudaEvent_t ev_rg[2 * (RP_MAXL + 1)];  // ... and around the gather of a rebuilding hop
    int64_t launches;
    char err[512];
};

// ---- helpers -----------------------------------------------------------------------------------
inline int div_up(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }
inline int pad4(int x) { return (x + 3) & ~3; }

// Every kernel of the library goes through this: programmatic stream serialisation (see pdl_enter)
// unless switched off for the context.
#define RP_LAUNCH(ctx, kernel, grid, block, smem, ...)                                            \
    do {                                                                                           \
        cudaLaunchConfig_t cfg_ = {};                                                              \
        cfg_.gridDim = dim3((unsigned)(grid));                                                     \
        cfg_.blockDim = dim3((unsigned)(block));                                                   \
        cfg_.dynamicSmemBytes = (size_t)(smem);                                                    \
        cfg_.stream = (ctx)->stream;                                                               \
        cudaLaunchAttribute attr_[1];                                                              \
        attr_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                          \
        attr_[0].val.programmaticStreamSerializationAllowed = 1;                                   \
        cfg_.attrs = attr_;                                                                        \
        cfg_.numAttrs = (ctx)->pdl ? 1 : 0;                                                        \
        cudaLaunchKernelEx(&cfg_, kernel, __VA_ARGS__);                                            \
        (ctx)->launches++;                                                                         \
    } while (0)

// dispatch on row width: ld <= 32 floats -> 8 lanes per row, <= 64 -> 16, else whole warp
#define RP_WIDTH_DISPATCH(ld, CALL)                       \
    do {                                                  \
        const int nv_ = div_up((ld), 128);                \
        if ((ld) <= 32) { CALL(1, 8); }                   \
        else if ((ld) <= 64) { CALL(1, 16); }             \
        else if (nv_ <= 1) { CALL(1, 32); }               \
        else if (nv_ <= 2) { CALL(2, 32); }               \
        else if (nv_ <= 4) { CALL(4, 32); }               \
        else { CALL(8, 32); }                             \
    } while (0)

// graph_store.cu
cudaError_t graph_build(Ctx* c, const int32_t* src_dev, const int32_t* dst_dev, const float* w_dev, int64_t E,
                        double slack, int64_t pool_edges);
void graph_batch_classify(Ctx* c, int n);   // validate, dedupe, find net changes, plan
void graph_batch_apply_small(Ctx* c, int n);            // a handful of updates: control block reset, Apply and the hop-0 senders in one block
void graph_batch_mutate(Ctx* c, int n);                 // apply the net changes to both directions
void graph_batch_cleanup(Ctx* c, int n);                // reset per-batch scratch
cudaError_t graph_export(Ctx* c, int64_t* rowptr, int32_t* col, float* weight, int64_t col_capacity, int64_t* n_edges);

// frontier.cu
void scan_degrees(Ctx* c, const int32_t* list, const int* n_dev, int n_host, const int32_t* deg,
                  int64_t* out, unsigned long long* total_dev);
void frontier_seed_features(Ctx* c, int n);             // A_0 from the batch's feature updates
void frontier_mark(Ctx* c, int l, bool walk, int n);    // bitmap of A_l: (walk) edge-record sinks, A_{l-1} and Out(C_{l-1}); rebuilding hops: bottom-up
void frontier_mark_extras(Ctx* c, int l);               // marks only what no walk finds (for hops whose message walk marks its sinks itself)
void frontier_compact(Ctx* c, int l);                   // bitmap -> ascending list A_l
void frontier_compact_small(Ctx* c, int l);              // the same in one block (tiny batches, small graphs)
void senders_build_small(Ctx* c, int l);                // C_l = A_l with its degree prefix, in one block
void senders_build(Ctx* c, int l, int n);               // C_l, posmap, coff, E_{l+1}
void senders_release(Ctx* c, int l);                    // clear posmap entries of C_l

// scatter.cu
void spmm_full(Ctx* c, int l);                          // S^l for every vertex (bootstrap)
void bitmap_to_list_from(Ctx* c, uint32_t* bitmap, int32_t* list, int* count_dev, unsigned long long* pull_work);
// monotonic.cu (max aggregation, Sec. 3.4.2)
void max_full(Ctx* c, int l);                           // bootstrap: cached maxima of every vertex
void max_hop(Ctx* c, int l, int n);                     // messages <old, new>, recomputation of invalidated sinks
void max_senders_build(Ctx* c, int l);                  // rows of A_l whose embedding changed, with their out-degree prefix
void max_prepare();
void choose_direction(Ctx* c, int l);                   // delta or rebuilding form of hop l (device-side decision)
void scatter_layer(Ctx* c, int l, int n);               // delta messages of hop l into dS^l
void regather_layer(Ctx* c, int l);                     // rebuilding form: S^l rows of A_l gathered anew
void fold_deltas(Ctx* c, int l);                        // S^l += dS^l, dS^l = 0 on the rows of A_l

// attention.cu (attention layers, Sec. 3.4.1)
void att_full(Ctx* c, int l);                           // bootstrap: logit halves, cached rows, embeddings of every vertex
void att_hop(Ctx* c, int l, int n, bool small);         // frontier, messages, recomputation: cached rows of A_l
void att_update(Ctx* c, int l, bool full);              // h^l = numerator / denominator on the rows of A_l; keeps the old rows

// partition.cu (partitioned execution, Sec. 4)
void part_ship(Ctx* c, int l);             // remote send: halo mailboxes of hop l into their owners' accumulators
void part_fetch_halo_rows(Ctx* c, int l);  // bootstrap: H^l of every assigned halo slot from its owner

// layer_update.cu
void update_rows(Ctx* c, int l, bool full);             // re-apply Update^l + activation, emit deltas
void self_project(Ctx* c, int l, bool full);            // refresh the cached self projection of a narrow SAGE layer
void sender_transform(Ctx* c, int l);                   // P^l rows of the senders of hop l, and their transformed deltas
void neighbour_transform(Ctx* c, int l, const float* rows_in, int ld_rows, const int* n_dev, int n_host,
                         float* rows_out);              // compact rows times the layer's neighbour matrix
void feature_rows(Ctx* c, int n);                       // hop 0: overwrite feature rows, emit deltas
void extra_sender_rows(Ctx* c, int l, int n);           // deltas of senders whose row did not change

// layer_update_tc.cu
cudaError_t tc_weights_build(TcW* out, const float* W_host, int K, int ldw);
void tc_prepare();   // one-time kernel attributes (not allowed inside a stream capture)
void narrow_prepare();   // likewise, for the update form for narrow outputs

}  // namespace rp
