// Router of the partitioned execution (Sec. 4.3, 4.4, Alg. 1): host code only.
//
// Keeps the vertex-partition map, per-partition load, in-degrees and the high in-degree set, places the
// vertices that edge additions create, splits a batch given in global ids into per-worker batches in
// local ids (an edge goes to its source's worker; if the sink lives elsewhere that worker gets a
// no-compute copy), and hands out halo slots: the first time a worker holds an edge whose other endpoint
// is remote, that endpoint gets the worker's next free halo slot.  Every worker process runs a replica
// on the same stream of batches; the replicas stay identical because nothing here depends on timing.
#include "../../include/ripple_part.h"

#include <algorithm>
#include <new>
#include <unordered_map>
#include <vector>

namespace {

struct Part {
    int64_t n_local = 0;         // local id capacity (multiple of 32)
    int64_t next_local = 0;      // next free local id
    int64_t halo_cap = 0;
    int64_t next_halo = 0;       // halo slots in use
    std::vector<int32_t> global_of;                 // local id -> global id (-1: unused)
    std::unordered_map<int32_t, int32_t> halo_of;   // remote global id -> halo slot
    std::vector<int32_t> halo_owner, halo_remote;   // per slot
    // the batch being routed
    std::vector<ripple_update> ops;
    std::vector<uint8_t> no_compute;
    std::vector<int32_t> op_of;      // position in the routed batch of the operation each local operation comes from
    std::vector<int32_t> row_of;
    int64_t first_new_halo = 0;
};

}  // namespace

struct ripple_router {
    int P = 0;
    int64_t N = 0;
    int routing = 0;
    int64_t hd_refresh = 0, seen = 0, n_edges = 0, placed = 0;
    std::vector<int32_t> owner, local_id, in_degree;
    std::vector<int64_t> load;
    std::vector<uint8_t> high;
    std::vector<Part> part;
    std::vector<int32_t> src0, dst0;      // the initial edges (for ripple_router_partition_fill)
    // the edge lists: whether an edge exists (in-degrees must not move under no-op updates), and the expansion
    // of vertex deletions
    std::vector<std::vector<int32_t>> out_adj, in_adj;

    int32_t cur_pos = 0;   // position in the batch of the operation being routed
    void count_update() { if (++seen % hd_refresh == 0) refresh_high(); }
    static bool drop(std::vector<int32_t>& a, int32_t x) {
        for (size_t i = 0; i < a.size(); ++i)
            if (a[i] == x) { a[i] = a.back(); a.pop_back(); return true; }
        return false;
    }
    bool has_edge(int32_t u, int32_t v) const {   // the shorter of the two lists is searched
        const std::vector<int32_t>& a = out_adj[u].size() <= in_adj[v].size() ? out_adj[u] : in_adj[v];
        const int32_t x = &a == &out_adj[u] ? v : u;
        return std::find(a.begin(), a.end(), x) != a.end();
    }
    // routes one edge operation (placing new endpoints first); false: a worker ran out of ids or halo slots
    bool route_edge(int32_t op, int32_t u, int32_t v) {
        const bool add = op == RIPPLE_OP_ADD_EDGE;
        if (add && !assign_edge(u, v)) return false;
        const int pu = owner[u], pv = owner[v];
        if (pu < 0 || pv < 0) return true;   // (deleting an edge of a vertex that was never placed: nothing exists)
        const int32_t lu = id_at(pu, u), lv = id_at(pu, v);
        if (lu < 0 || lv < 0) return false;
        part[pu].ops.push_back({op, lu, lv});
        part[pu].no_compute.push_back(0);
        part[pu].op_of.push_back(cur_pos);
        if (pv != pu) {
            const int32_t su = id_at(pv, u), sv = id_at(pv, v);
            if (su < 0 || sv < 0) return false;
            part[pv].ops.push_back({op, su, sv});
            part[pv].no_compute.push_back(1);
            part[pv].op_of.push_back(cur_pos);
        }
        if (add && !has_edge(u, v)) { in_degree[v]++; n_edges++; out_adj[u].push_back(v); in_adj[v].push_back(u); }
        else if (!add && drop(out_adj[u], v)) { in_degree[v]--; n_edges--; drop(in_adj[v], u); }
        return true;
    }
    void route_feature(int32_t u, int32_t row) {
        Part& q = part[owner[u]];
        q.ops.push_back({RIPPLE_OP_SET_FEATURE, local_id[u], (int32_t)q.row_of.size()});
        q.no_compute.push_back(0);
        q.op_of.push_back(cur_pos);
        q.row_of.push_back(row);
    }

    void refresh_high() {
        const double avg = (double)n_edges / (double)std::max<int64_t>(placed, 1);
        for (int64_t v = 0; v < N; ++v) high[v] = (double)in_degree[v] > 2.0 * avg;
    }
    int least_loaded() const {
        int best = 0;
        for (int p = 1; p < P; ++p)
            if (load[p] < load[best]) best = p;
        return best;
    }
    bool place(int32_t v, int p) {
        Part& q = part[p];
        if (q.next_local >= q.n_local) return false;
        owner[v] = p;
        local_id[v] = (int32_t)q.next_local;
        q.global_of[q.next_local++] = v;
        load[p]++;
        placed++;
        return true;
    }
    // Alg. 1 (or the hash rule): places whichever endpoint of an added edge does not exist yet
    bool assign_edge(int32_t u, int32_t v) {
        const bool eu = owner[u] >= 0, ev = owner[v] >= 0;
        if (eu && ev) return true;
        if (routing == RIPPLE_ROUTE_HASH) {
            if (!eu && !place(u, u % P)) return false;
            if (!ev && owner[v] < 0 && !place(v, v % P)) return false;
            return true;
        }
        if (!eu && ev) return place(u, high[v] ? owner[v] : least_loaded());
        const int p = least_loaded();   // the final Else: every remaining case
        if (!eu && !place(u, p)) return false;
        if (!ev && owner[v] < 0 && !place(v, p)) return false;
        return true;
    }
    // local id under which worker p knows global vertex g (a halo slot if g lives elsewhere), or -1 if full
    int32_t id_at(int p, int32_t g) {
        if (owner[g] == p) return local_id[g];
        Part& q = part[p];
        auto it = q.halo_of.find(g);
        if (it != q.halo_of.end()) return (int32_t)(q.n_local + it->second);
        if (q.next_halo >= q.halo_cap) return -1;
        const int32_t slot = (int32_t)q.next_halo++;
        q.halo_of.emplace(g, slot);
        q.halo_owner.push_back(owner[g]);
        q.halo_remote.push_back(local_id[g]);
        q.global_of[q.n_local + slot] = g;
        return (int32_t)(q.n_local + slot);
    }
};

extern "C" ripple_status ripple_router_create(int32_t n_partitions, int64_t num_vertices, const int32_t* owner,
                                              int64_t num_edges, const int32_t* src, const int32_t* dst,
                                              int32_t routing, int64_t hd_refresh, int64_t spare_local,
                                              int64_t halo_capacity, ripple_router** out) {
    if (out) *out = nullptr;
    if (!out || !owner || n_partitions < 1 || n_partitions > RIPPLE_MAX_PEERS || num_vertices < 1 || num_edges < 0 ||
        (num_edges > 0 && (!src || !dst)) || (routing != RIPPLE_ROUTE_LOCALITY && routing != RIPPLE_ROUTE_HASH) ||
        spare_local < 0 || halo_capacity < 0)
        return RIPPLE_ERR_INVALID_ARG;
    ripple_router* r = new (std::nothrow) ripple_router();
    if (!r) return RIPPLE_ERR_OOM;
    r->P = n_partitions; r->N = num_vertices; r->routing = routing;
    r->hd_refresh = hd_refresh > 0 ? hd_refresh : 500000;
    r->owner.assign(num_vertices, -1);
    r->local_id.assign(num_vertices, -1);
    r->in_degree.assign(num_vertices, 0);
    r->high.assign(num_vertices, 0);
    r->load.assign(n_partitions, 0);
    r->part.resize(n_partitions);
    r->out_adj.resize(num_vertices);
    r->in_adj.resize(num_vertices);
    std::vector<int64_t> count(n_partitions, 0);
    for (int64_t v = 0; v < num_vertices; ++v) {
        if (owner[v] >= n_partitions) { delete r; return RIPPLE_ERR_INVALID_ARG; }
        if (owner[v] >= 0) count[owner[v]]++;
    }
    for (int p = 0; p < n_partitions; ++p) {
        Part& q = r->part[p];
        q.n_local = (count[p] + spare_local + 31) / 32 * 32;
        if (q.n_local == 0) q.n_local = 32;
        q.halo_cap = halo_capacity;
        q.global_of.assign(q.n_local + q.halo_cap, -1);
    }
    for (int64_t v = 0; v < num_vertices; ++v)      // local ids in ascending global id
        if (owner[v] >= 0) r->place((int32_t)v, owner[v]);
    r->src0.assign(src, src + num_edges);
    r->dst0.assign(dst, dst + num_edges);
    for (int64_t e = 0; e < num_edges; ++e) {
        const int32_t u = src[e], v = dst[e];
        if (u < 0 || u >= num_vertices || v < 0 || v >= num_vertices || r->owner[u] < 0 || r->owner[v] < 0) {
            delete r;
            return RIPPLE_ERR_VERTEX_RANGE;
        }
        r->in_degree[v]++;
        r->out_adj[u].push_back(v);
        r->in_adj[v].push_back(u);
        if (r->owner[u] != r->owner[v] && (r->id_at(r->owner[u], v) < 0 || r->id_at(r->owner[v], u) < 0)) {
            delete r;
            return RIPPLE_ERR_CAPACITY;
        }
    }
    r->n_edges = num_edges;
    r->refresh_high();
    *out = r;
    return RIPPLE_OK;
}

extern "C" void ripple_router_destroy(ripple_router* r) { delete r; }

static int64_t edges_of(const ripple_router* r, int rank) {
    int64_t n = 0;
    for (size_t e = 0; e < r->src0.size(); ++e) n += r->owner[r->src0[e]] == rank || r->owner[r->dst0[e]] == rank;
    return n;
}

extern "C" ripple_status ripple_router_partition_shape(ripple_router* r, int32_t rank, int64_t* n_local,
                                                       int64_t* num_vertices, int64_t* num_edges,
                                                       int64_t* halos_used) {
    if (!r || rank < 0 || rank >= r->P || !n_local || !num_vertices || !num_edges || !halos_used) return RIPPLE_ERR_INVALID_ARG;
    const Part& q = r->part[rank];
    *n_local = q.n_local;
    *num_vertices = q.n_local + q.halo_cap;
    *num_edges = edges_of(r, rank);
    *halos_used = q.next_halo;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_router_partition_fill(ripple_router* r, int32_t rank, int32_t* src_local,
                                                      int32_t* dst_local, int64_t* edge_of, int32_t* global_of,
                                                      int32_t* halo_owner, int32_t* halo_remote_id) {
    if (!r || rank < 0 || rank >= r->P || !global_of) return RIPPLE_ERR_INVALID_ARG;
    Part& q = r->part[rank];
    int64_t n = 0;
    for (size_t e = 0; e < r->src0.size(); ++e) {
        const int32_t u = r->src0[e], v = r->dst0[e];
        if (r->owner[u] != rank && r->owner[v] != rank) continue;
        if (!src_local || !dst_local) return RIPPLE_ERR_INVALID_ARG;
        src_local[n] = r->id_at(rank, u);
        dst_local[n] = r->id_at(rank, v);
        if (edge_of) edge_of[n] = (int64_t)e;
        ++n;
    }
    std::copy(q.global_of.begin(), q.global_of.end(), global_of);
    for (int64_t h = 0; h < q.next_halo; ++h) {
        if (!halo_owner || !halo_remote_id) return RIPPLE_ERR_INVALID_ARG;
        halo_owner[h] = q.halo_owner[h];
        halo_remote_id[h] = q.halo_remote[h];
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_router_route(ripple_router* r, const ripple_update* ups, int64_t n) {
    if (!r || n < 0 || (n > 0 && !ups)) return RIPPLE_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; ++i) {     // checked before anything changes
        const ripple_update& x = ups[i];
        if (x.op < RIPPLE_OP_ADD_EDGE || x.op > RIPPLE_OP_DEL_VERTEX) return RIPPLE_ERR_INVALID_ARG;
        if (x.u < 0 || x.u >= r->N) return RIPPLE_ERR_VERTEX_RANGE;
        if ((x.op == RIPPLE_OP_ADD_EDGE || x.op == RIPPLE_OP_DEL_EDGE) && (x.v < 0 || x.v >= r->N)) return RIPPLE_ERR_VERTEX_RANGE;
    }
    for (Part& q : r->part) {
        q.ops.clear(); q.no_compute.clear(); q.op_of.clear(); q.row_of.clear();
        q.first_new_halo = q.next_halo;
    }
    for (int64_t i = 0; i < n; ++i) {
        const ripple_update& x = ups[i];
        r->cur_pos = (int32_t)i;
        if (x.op == RIPPLE_OP_SET_FEATURE) {
            if (r->owner[x.u] < 0) return RIPPLE_ERR_INVALID_ARG;   // a feature update of a vertex that is not in the graph
            r->route_feature(x.u, x.v);
        } else if (x.op == RIPPLE_OP_DEL_VERTEX) {
            // Replaced, at its position in the batch, by the deletions of the vertex's edges (out-edges in ascending
            // sink order, then in-edges in ascending source order: every replica generates the same sequence) and a
            // feature update with a row of zeros (payload row -1).
            r->count_update();
            if (r->owner[x.u] < 0) continue;
            std::vector<int32_t> outs = r->out_adj[x.u], ins = r->in_adj[x.u];
            std::sort(outs.begin(), outs.end());
            std::sort(ins.begin(), ins.end());
            for (int32_t v : outs) { if (!r->route_edge(RIPPLE_OP_DEL_EDGE, x.u, v)) return RIPPLE_ERR_CAPACITY; r->count_update(); }
            for (int32_t u : ins) { if (!r->route_edge(RIPPLE_OP_DEL_EDGE, u, x.u)) return RIPPLE_ERR_CAPACITY; r->count_update(); }
            r->route_feature(x.u, -1);
        } else if (!r->route_edge(x.op, x.u, x.v)) {
            return RIPPLE_ERR_CAPACITY;
        }
        r->count_update();
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_router_batch_shape(ripple_router* r, int32_t rank, int64_t* n_ops, int64_t* n_rows,
                                                   int64_t* n_new_halos) {
    if (!r || rank < 0 || rank >= r->P || !n_ops || !n_rows || !n_new_halos) return RIPPLE_ERR_INVALID_ARG;
    const Part& q = r->part[rank];
    *n_ops = (int64_t)q.ops.size();
    *n_rows = (int64_t)q.row_of.size();
    *n_new_halos = q.next_halo - q.first_new_halo;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_router_batch_fill(ripple_router* r, int32_t rank, ripple_update* ups_local,
                                                  uint8_t* no_compute, int32_t* op_of, int32_t* row_of,
                                                  int32_t* first_halo, int32_t* halo_owner, int32_t* halo_remote_id) {
    if (!r || rank < 0 || rank >= r->P || !first_halo) return RIPPLE_ERR_INVALID_ARG;
    const Part& q = r->part[rank];
    if ((!q.ops.empty() && (!ups_local || !no_compute)) || (!q.row_of.empty() && !row_of)) return RIPPLE_ERR_INVALID_ARG;
    std::copy(q.ops.begin(), q.ops.end(), ups_local);
    std::copy(q.no_compute.begin(), q.no_compute.end(), no_compute);
    if (op_of) std::copy(q.op_of.begin(), q.op_of.end(), op_of);
    std::copy(q.row_of.begin(), q.row_of.end(), row_of);
    *first_halo = (int32_t)q.first_new_halo;
    for (int64_t h = q.first_new_halo; h < q.next_halo; ++h) {
        if (!halo_owner || !halo_remote_id) return RIPPLE_ERR_INVALID_ARG;
        halo_owner[h - q.first_new_halo] = q.halo_owner[h];
        halo_remote_id[h - q.first_new_halo] = q.halo_remote[h];
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_router_global_ids(ripple_router* r, int32_t rank, int32_t* global_of, int64_t capacity) {
    if (!r || rank < 0 || rank >= r->P || !global_of) return RIPPLE_ERR_INVALID_ARG;
    const Part& q = r->part[rank];
    if (capacity < (int64_t)q.global_of.size()) return RIPPLE_ERR_CAPACITY;
    std::copy(q.global_of.begin(), q.global_of.end(), global_of);
    return RIPPLE_OK;
}

extern "C" int32_t ripple_router_owner(ripple_router* r, int32_t v) {
    return (r && v >= 0 && v < r->N) ? r->owner[v] : -1;
}
extern "C" int32_t ripple_router_local_id(ripple_router* r, int32_t v) {
    return (r && v >= 0 && v < r->N) ? r->local_id[v] : -1;
}
extern "C" int32_t ripple_router_global_id(ripple_router* r, int32_t rank, int32_t local_id) {
    if (!r || rank < 0 || rank >= r->P) return -1;
    const Part& q = r->part[rank];
    return (local_id >= 0 && (size_t)local_id < q.global_of.size()) ? q.global_of[local_id] : -1;
}
extern "C" int32_t ripple_router_is_high_degree(ripple_router* r, int32_t v) {
    return (r && v >= 0 && v < r->N) ? r->high[v] : 0;
}
extern "C" int64_t ripple_router_load(ripple_router* r, int32_t rank) {
    return (r && rank >= 0 && rank < r->P) ? r->load[rank] : -1;
}
