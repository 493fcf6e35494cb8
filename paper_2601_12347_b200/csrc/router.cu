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
#include <unordered_set>
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
    std::unordered_set<uint64_t> edges;   // u * N + v: keeps the in-degrees right under no-op updates
    std::vector<Part> part;
    std::vector<int32_t> src0, dst0;      // the initial edges (for ripple_router_partition_fill)

    uint64_t key(int32_t u, int32_t v) const { return (uint64_t)u * (uint64_t)N + (uint64_t)v; }

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
        r->edges.insert(r->key(u, v));
        r->in_degree[v]++;
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
                                                      int32_t* dst_local, int32_t* global_of, int32_t* halo_owner,
                                                      int32_t* halo_remote_id) {
    if (!r || rank < 0 || rank >= r->P || !global_of) return RIPPLE_ERR_INVALID_ARG;
    Part& q = r->part[rank];
    int64_t n = 0;
    for (size_t e = 0; e < r->src0.size(); ++e) {
        const int32_t u = r->src0[e], v = r->dst0[e];
        if (r->owner[u] != rank && r->owner[v] != rank) continue;
        if (!src_local || !dst_local) return RIPPLE_ERR_INVALID_ARG;
        src_local[n] = r->id_at(rank, u);
        dst_local[n] = r->id_at(rank, v);
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
        if (x.op != RIPPLE_OP_ADD_EDGE && x.op != RIPPLE_OP_DEL_EDGE && x.op != RIPPLE_OP_SET_FEATURE) return RIPPLE_ERR_INVALID_ARG;
        if (x.u < 0 || x.u >= r->N) return RIPPLE_ERR_VERTEX_RANGE;
        if (x.op != RIPPLE_OP_SET_FEATURE && (x.v < 0 || x.v >= r->N)) return RIPPLE_ERR_VERTEX_RANGE;
    }
    for (Part& q : r->part) {
        q.ops.clear(); q.no_compute.clear(); q.row_of.clear();
        q.first_new_halo = q.next_halo;
    }
    for (int64_t i = 0; i < n; ++i) {
        const ripple_update& x = ups[i];
        if (x.op == RIPPLE_OP_SET_FEATURE) {
            const int p = r->owner[x.u];
            if (p < 0) return RIPPLE_ERR_INVALID_ARG;   // a feature update of a vertex that is not in the graph
            Part& q = r->part[p];
            q.ops.push_back({x.op, r->local_id[x.u], (int32_t)q.row_of.size()});
            q.no_compute.push_back(0);
            q.row_of.push_back(x.v);
        } else {
            const bool add = x.op == RIPPLE_OP_ADD_EDGE;
            if (add && !r->assign_edge(x.u, x.v)) return RIPPLE_ERR_CAPACITY;
            const int pu = r->owner[x.u], pv = r->owner[x.v];
            if (pu >= 0 && pv >= 0) {   // (deleting an edge of a vertex that was never placed: nothing exists)
                const int32_t lu = r->id_at(pu, x.u), lv = r->id_at(pu, x.v);
                if (lu < 0 || lv < 0) return RIPPLE_ERR_CAPACITY;
                r->part[pu].ops.push_back({x.op, lu, lv});
                r->part[pu].no_compute.push_back(0);
                if (pv != pu) {
                    const int32_t su = r->id_at(pv, x.u), sv = r->id_at(pv, x.v);
                    if (su < 0 || sv < 0) return RIPPLE_ERR_CAPACITY;
                    r->part[pv].ops.push_back({x.op, su, sv});
                    r->part[pv].no_compute.push_back(1);
                }
                const uint64_t k = r->key(x.u, x.v);
                if (add && r->edges.insert(k).second) { r->in_degree[x.v]++; r->n_edges++; }
                else if (!add && r->edges.erase(k)) { r->in_degree[x.v]--; r->n_edges--; }
            }
        }
        if (++r->seen % r->hd_refresh == 0) r->refresh_high();
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
                                                  uint8_t* no_compute, int32_t* row_of, int32_t* first_halo,
                                                  int32_t* halo_owner, int32_t* halo_remote_id) {
    if (!r || rank < 0 || rank >= r->P || !first_halo) return RIPPLE_ERR_INVALID_ARG;
    const Part& q = r->part[rank];
    if ((!q.ops.empty() && (!ups_local || !no_compute)) || (!q.row_of.empty() && !row_of)) return RIPPLE_ERR_INVALID_ARG;
    std::copy(q.ops.begin(), q.ops.end(), ups_local);
    std::copy(q.no_compute.begin(), q.no_compute.end(), no_compute);
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
