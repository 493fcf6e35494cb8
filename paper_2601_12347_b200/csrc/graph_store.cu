// GPU-resident dynamic graph store: both directions of the adjacency as CSR with per-vertex
// slack, backed by an overflow pool, and the batched insert/delete kernels.
//
// A batch is normalised on the device ("Apply" step of Sec. 3.3): the last operation on a pair
// wins (pair hash table + atomicMax of the op index), the winner is compared with the stored
// row (warp-cooperative search) and becomes a net change record or a counted no-op.  Records
// are then applied without any per-row lock and without scanning rows again:
//   deletions  tombstone their slot; the row's last n_del slots ("tail") are read, the live
//              ones among them are packed to the front of the tail and handed out, by ticket,
//              to the holes in front of the tail (a many-at-once swap-with-last);
//   additions  take slot new_deg + rank, rank from an atomic per-row counter; a row that would
//              overflow its capacity first moves into the overflow pool with doubled capacity.
// Nothing is mutated until the whole batch has been validated and the pool demand is known to
// fit, so a rejected batch leaves the store untouched.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>
#include <vector>

namespace rp {

// ---------------------------------------------------------------------------------------------
// build from COO
// ---------------------------------------------------------------------------------------------
__global__ void k_count_degrees(const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                                int64_t E, int N, int32_t* deg_out, int32_t* deg_in, Ctl* ctl) {
    pdl_enter();
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < E;
         e += (int64_t)gridDim.x * blockDim.x) {
        int u = src[e], v = dst[e];
        if ((unsigned)u >= (unsigned)N || (unsigned)v >= (unsigned)N) {
            atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_VERTEX_RANGE);
            continue;
        }
        atomicAdd(&deg_out[u], 1);
        atomicAdd(&deg_in[v], 1);
    }
}

__global__ void k_capacities(int N, const int32_t* __restrict__ deg, int32_t* cap, float slack) {
    pdl_enter();
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    int d = deg[v];
    int extra = (int)ceilf((float)d * slack) + 4;
    cap[v] = (d + extra + 3) & ~3;
}

__global__ void k_fill_rows(const int32_t* __restrict__ src, const int32_t* __restrict__ dst,
                            const float* __restrict__ weight, int64_t E, int N, Side out, Side in) {
    pdl_enter();
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < E;
         e += (int64_t)gridDim.x * blockDim.x) {
        int u = src[e], v = dst[e];
        if ((unsigned)u >= (unsigned)N || (unsigned)v >= (unsigned)N) continue;
        int p = atomicAdd(&out.cnt_add[u], 1);
        out.col[out.start[u] + p] = v;
        int q = atomicAdd(&in.cnt_add[v], 1);
        in.col[in.start[v] + q] = u;
        if (out.w) {
            const float a = weight ? weight[e] : 1.0f;
            out.w[out.start[u] + p] = a;
            in.w[in.start[v] + q] = a;
        }
    }
}

static cudaError_t alloc_side(Side& s, int N) {
    cudaError_t e;
    size_t nb = sizeof(int32_t) * (size_t)N;
    if ((e = cudaMalloc(&s.start, sizeof(int64_t) * ((size_t)N + 1)))) return e;
    int32_t** arrs[] = {&s.cap, &s.deg, &s.cnt_del, &s.cnt_add, &s.tick_a, &s.tick_b, &s.touch};
    for (auto a : arrs) {
        if ((e = cudaMalloc(a, nb))) return e;
        if ((e = cudaMemset(*a, 0, nb))) return e;
    }
    if ((e = cudaMalloc(&s.free_blk, sizeof(int64_t) * (size_t)RP_POOL_CLASSES * RP_POOL_LIST_CAP))) return e;
    if ((e = cudaMalloc(&s.free_cnt, sizeof(int32_t) * RP_POOL_CLASSES))) return e;
    return cudaMemset(s.free_cnt, 0, sizeof(int32_t) * RP_POOL_CLASSES);
}

cudaError_t graph_build(Ctx* c, const int32_t* src, const int32_t* dst, const float* weight, int64_t E,
                        double slack, int64_t pool_edges) {
    cudaError_t e;
    const int N = c->N;
    for (int s = 0; s < 2; ++s)
        if ((e = alloc_side(c->side[s], N))) return e;
    Side& out = c->side[0];
    Side& in = c->side[1];
    const int T = 256;
    int grid_e = (int)std::min<int64_t>(std::max<int64_t>(div_up(E, T), 1), (int64_t)c->n_sm * 16);
    if (E > 0) RP_LAUNCH(c, k_count_degrees, grid_e, T, 0, src, dst, E, N, out.deg, in.deg, c->ctl);
    for (int s = 0; s < 2; ++s) {
        RP_LAUNCH(c, k_capacities, div_up(N, T), T, 0, N, c->side[s].deg, c->side[s].cap, (float)slack);
        scan_degrees(c, nullptr, nullptr, N, c->side[s].cap, c->side[s].start, &c->ctl->pool_next[s]);
    }
    if ((e = cudaMemcpyAsync(c->ctl_host, c->ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, c->stream))) return e;
    if ((e = cudaStreamSynchronize(c->stream))) return e;
    if (c->ctl_host->err) return cudaSuccess;  // caller inspects ctl_host->err
    for (int s = 0; s < 2; ++s) {
        Side& sd = c->side[s];
        sd.base_end = (int64_t)c->ctl_host->pool_next[s];
        sd.col_size = sd.base_end + pool_edges;
        if ((e = cudaMalloc(&sd.col, sizeof(int32_t) * (size_t)std::max<int64_t>(sd.col_size, 4)))) return e;
        if (c->weighted && (e = cudaMalloc(&sd.w, sizeof(float) * (size_t)std::max<int64_t>(sd.col_size, 4)))) return e;
    }
    if (E > 0) RP_LAUNCH(c, k_fill_rows, grid_e, T, 0, src, dst, weight, E, N, out, in);
    for (int s = 0; s < 2; ++s)
        if ((e = cudaMemsetAsync(c->side[s].cnt_add, 0, sizeof(int32_t) * (size_t)N, c->stream))) return e;
    return cudaStreamSynchronize(c->stream);
}

// ---------------------------------------------------------------------------------------------
// batch normalisation
// ---------------------------------------------------------------------------------------------
// number of operations after vertex deletions have been expanded into edge deletions
__device__ __forceinline__ int ops_total(const Ctl* ctl) {
    return ctl->n_ops + (ctl->expand_failed ? 0 : (int)ctl->n_extra);
}

// Vertex deletion (Sec. 3.2): every edge that has the vertex as an endpoint goes.  Each deletion
// reserves room behind the caller's operations for one edge deletion per stored out- and
// in-neighbour; the generated operations carry the deletion's position in the batch, so that the
// last-operation-wins rule orders them against the explicit operations on the same pairs.
__global__ void k_expand_plan(const ripple_update* __restrict__ ups, int N, long long capacity, Ctl* ctl,
                              Side out, Side in, int2* vjobs) {
    pdl_enter();
    const int n = ctl->n_ops;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const ripple_update op = ups[i];
        if (op.op != RIPPLE_OP_DEL_VERTEX || (unsigned)op.u >= (unsigned)N) continue;
        const unsigned long long cnt = (unsigned long long)out.deg[op.u] + (unsigned long long)in.deg[op.u];
        const unsigned long long base = atomicAdd(&ctl->n_extra, cnt);
        if ((unsigned long long)n + base + cnt > (unsigned long long)capacity) {
            atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_CAPACITY);
            ctl->expand_failed = 1;
            ctl->abort = 1;
            continue;
        }
        vjobs[atomicAdd(&ctl->n_vjobs, 1)] = make_int2(i, n + (int)base);
    }
}

__global__ void k_expand_copy(ripple_update* ups, int32_t* op_seq, Ctl* ctl, Side out, Side in,
                              const int2* __restrict__ vjobs) {
    pdl_enter();
    if (ctl->abort) return;
    const int nj = ctl->n_vjobs;
    for (int j = blockIdx.x; j < nj; j += gridDim.x) {
        const int2 job = vjobs[j];
        const int w = ups[job.x].u;
        const int dout = out.deg[w], din = in.deg[w];
        const int64_t bo = out.start[w], bi = in.start[w];
        for (int k = threadIdx.x; k < dout + din; k += blockDim.x) {
            ripple_update g;
            g.op = RIPPLE_OP_DEL_EDGE;
            if (k < dout) { g.u = w; g.v = out.col[bo + k]; }
            else { g.u = in.col[bi + (k - dout)]; g.v = w; }
            ups[job.y + k] = g;
            op_seq[job.y + k] = job.x;
        }
    }
}

__device__ __forceinline__ void d_classify(const ripple_update* __restrict__ ups, const int32_t* __restrict__ op_seq, int N,
                                           Ctl* ctl, unsigned long long* hkeys, unsigned long long* hwin, int hmask,
                                           int32_t* op_slot, int32_t* feat_last, int32_t* vdel_seq, int no_vertex_ops) {
    const int n = ops_total(ctl), n_given = ctl->n_ops;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        ripple_update op = ups[i];
        op_slot[i] = -1;
        // (a worker of a partitioned execution takes no vertex deletion: its router has turned them into edge deletions)
        if (op.op < 0 || op.op > 3 || (no_vertex_ops && op.op == RIPPLE_OP_DEL_VERTEX)) {
            atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_INVALID_ARG);
            ctl->abort = 1;
            continue;
        }
        bool bad = (unsigned)op.u >= (unsigned)N;
        if (op.op == RIPPLE_OP_SET_FEATURE) bad |= (unsigned)op.v >= (unsigned)ctl->n_rows;
        else if (op.op != RIPPLE_OP_DEL_VERTEX) bad |= (unsigned)op.v >= (unsigned)N;
        if (bad) {
            atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_VERTEX_RANGE);
            ctl->abort = 1;
            continue;
        }
        if (op.op == RIPPLE_OP_SET_FEATURE) {
            atomicMax(&feat_last[op.u], i);
            continue;
        }
        if (op.op == RIPPLE_OP_DEL_VERTEX) {   // also the last word on the vertex's feature row so far
            atomicMax(&feat_last[op.u], i);
            atomicMax(&vdel_seq[op.u], i);
            continue;
        }
        const int seq = i < n_given ? i : op_seq[i];
        const unsigned long long mine = ((unsigned long long)(seq + 1) << 32) | (unsigned)i;
        unsigned long long key = (unsigned long long)op.u * (unsigned long long)N + (unsigned long long)op.v + 1ull;
        int h = (int)(mix64(key) & (unsigned long long)hmask);
        bool placed = false;
        for (int probe = 0; probe <= hmask; ++probe) {
            unsigned long long prev = atomicCAS(&hkeys[h], 0ull, key);
            if (prev == 0ull || prev == key) {
                atomicMax(&hwin[h], mine);
                op_slot[i] = h;
                placed = true;
                break;
            }
            h = (h + 1) & hmask;
        }
        if (!placed) {   // table full: cannot happen with hsize >= 2 max_batch
            atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_CAPACITY);
            ctl->abort = 1;
        }
    }
}

__global__ void k_classify(const ripple_update* __restrict__ ups, const int32_t* __restrict__ op_seq, int N,
                           Ctl* ctl, unsigned long long* hkeys, unsigned long long* hwin, int hmask,
                           int32_t* op_slot, int32_t* feat_last, int32_t* vdel_seq, int no_vertex_ops) {
    pdl_enter();
    d_classify(ups, op_seq, N, ctl, hkeys, hwin, hmask, op_slot, feat_last, vdel_seq, no_vertex_ops);
}

// Position of x in row [base, base + deg), or -1; the whole block calls this.  Rows start on
// 16-byte boundaries, so every thread compares four entries per load, and it keeps eight loads in
// flight: a hub row of 150 K entries costs a block of 256 threads about 19 round trips to memory.
__device__ __forceinline__ int block_find(const int32_t* __restrict__ col, int64_t base, int deg, int x,
                                          volatile int* s_found) {
    constexpr int FIND_UNROLL = 8;
    __syncthreads();
    if (threadIdx.x == 0) *s_found = -1;
    __syncthreads();
    const int4* row4 = reinterpret_cast<const int4*>(col + base);
    const int n4 = deg >> 2;
    for (int q0 = 0; q0 < n4; q0 += FIND_UNROLL * blockDim.x) {
        int4 e[FIND_UNROLL];
#pragma unroll
        for (int k = 0; k < FIND_UNROLL; ++k) {
            int q = q0 + k * blockDim.x + threadIdx.x;
            e[k] = q < n4 ? __ldg(row4 + q) : make_int4(-1, -1, -1, -1);   // x is a vertex id: never negative
        }
#pragma unroll
        for (int k = 0; k < FIND_UNROLL; ++k) {
            int hit = e[k].x == x ? 0 : e[k].y == x ? 1 : e[k].z == x ? 2 : e[k].w == x ? 3 : -1;
            if (hit >= 0) *s_found = 4 * (q0 + k * blockDim.x + threadIdx.x) + hit;
        }
        if (*s_found >= 0) break;   // a peek per round; a thread that misses it only reads on
    }
    int j = 4 * n4 + threadIdx.x;
    if (j < deg && col[base + j] == x) *s_found = j;
    __syncthreads();
    return *s_found;
}

__device__ __forceinline__ void d_plan_growth(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in,
                                              int32_t* grow_out, int32_t* grow_in, int32_t* shrink_out,
                                              int32_t* shrink_in, int tid, int nthreads);
__device__ __forceinline__ void d_plan_check(Ctl* ctl, Side out, Side in);

// One block per op: winners are compared with the stored graph and become records or no-ops.
// The last block to finish then plans the row moves (which rows need a new block, and whether the
// blocks exist): no launch of its own for that.
// An explicit edge operation that precedes the deletion of one of its endpoints is superseded by
// it (for stored edges the generated deletion already wins the slot; for pairs that are not stored
// nothing was generated, hence the explicit test).  Only the caller's operations are counted.
__device__ __forceinline__ void
d_resolve(const ripple_update* __restrict__ ups, const int32_t* __restrict__ op_seq, Ctl* ctl,
          const unsigned long long* __restrict__ hwin, const int32_t* __restrict__ op_slot,
          const int32_t* __restrict__ feat_last, const int32_t* __restrict__ vdel_seq, Side out, Side in,
          Rec* rec, uint32_t* bitmap, const float* __restrict__ op_w, int32_t* grow_out, int32_t* grow_in,
          int32_t* shrink_out, int32_t* shrink_in, const uint8_t* __restrict__ silent) {
    __shared__ int s_found;
    __shared__ int s_last;
    if (ctl->abort) return;
    const int n = ops_total(ctl), n_given = ctl->n_ops;
    for (int i = blockIdx.x; i < n; i += gridDim.x) {
        ripple_update op = ups[i];
        if (op.op == RIPPLE_OP_SET_FEATURE || op.op == RIPPLE_OP_DEL_VERTEX) {
            if (threadIdx.x == 0 && feat_last[op.u] == i) {
                atomicAdd(&ctl->n_feat, 1);
                atomicOr(&bitmap[op.u >> 5], 1u << (op.u & 31));
            }
            continue;
        }
        const int seq = i < n_given ? i : op_seq[i];
        if ((int)(unsigned)hwin[op_slot[i]] != i || seq < max(vdel_seq[op.u], vdel_seq[op.v])) {
            if (threadIdx.x == 0 && i < n_given) atomicAdd(&ctl->n_superseded, 1);
            continue;
        }
        int j_out = block_find(out.col, out.start[op.u], out.deg[op.u], op.v, &s_found);
        bool is_add = op.op == RIPPLE_OP_ADD_EDGE;
        if (is_add == (j_out >= 0)) {
            if (threadIdx.x == 0) atomicAdd(is_add ? &ctl->n_noop_add : &ctl->n_noop_del, 1);
            continue;
        }
        int j_in = -1;
        if (!is_add) j_in = block_find(in.col, in.start[op.v], in.deg[op.v], op.u, &s_found);
        if (threadIdx.x == 0) {
            int r = atomicAdd(&ctl->n_rec, 1);
            atomicAdd(is_add ? &ctl->n_add : &ctl->n_del, 1);
            Rec x;
            x.u = op.u; x.v = op.v; x.sign = is_add ? 1 : -1;
            x.pos[0] = j_out; x.pos[1] = j_in;
            x.tail_val[0] = x.tail_val[1] = RP_TOMB;
            x.tail_w[0] = x.tail_w[1] = 0.f;
            // stored weights: a new edge takes the weight given with its operation, a deleted one had ...
            x.w = !out.w ? 1.0f : is_add ? ((op_w && i < n_given) ? op_w[i] : 1.0f) : out.w[out.start[op.u] + j_out];
            x.deg_out_old = out.deg[op.u];
            x.silent = (silent && i < n_given) ? silent[i] : 0;
            x.rep[0] = atomicAdd(&out.touch[op.u], 1) == 0;
            x.rep[1] = atomicAdd(&in.touch[op.v], 1) == 0;
            x.rank[0] = atomicAdd(is_add ? &out.cnt_add[op.u] : &out.cnt_del[op.u], 1);
            x.rank[1] = atomicAdd(is_add ? &in.cnt_add[op.v] : &in.cnt_del[op.v], 1);
            rec[r] = x;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&ctl->plan_done, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    d_plan_growth(ctl, rec, out, in, grow_out, grow_in, shrink_out, shrink_in, threadIdx.x, blockDim.x);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) d_plan_check(ctl, out, in);
}

__global__ void __launch_bounds__(256)
k_resolve(const ripple_update* __restrict__ ups, const int32_t* __restrict__ op_seq, Ctl* ctl,
          const unsigned long long* __restrict__ hwin, const int32_t* __restrict__ op_slot,
          const int32_t* __restrict__ feat_last, const int32_t* __restrict__ vdel_seq, Side out, Side in,
          Rec* rec, uint32_t* bitmap, const float* __restrict__ op_w, int32_t* grow_out, int32_t* grow_in,
          int32_t* shrink_out, int32_t* shrink_in, const uint8_t* __restrict__ silent) {
    pdl_enter();
    d_resolve(ups, op_seq, ctl, hwin, op_slot, feat_last, vdel_seq, out, in, rec, bitmap, op_w, grow_out, grow_in,
              shrink_out, shrink_in, silent);
}

// ---------------------------------------------------------------------------------------------
// Blocks of the adjacency store.  A row that outgrows its block moves to one of at least twice the
// size; a row left with less than a quarter of a (not small) block in use moves to a smaller one.
// Blocks handed out after the initial layout have power-of-two sizes (class k = 2^k entries) and
// come from the class's free list of vacated blocks if it has one, else from the never-used tail
// of the array (the overflow pool).  A vacated block -- of the pool or of the initial layout -- goes
// onto the list of the largest class that fits into it.  Within a kernel the lists are either
// taken from (k_grow_rows) or added to (k_commit_degrees), never both, so a plain counter per list
// is enough.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int class_for_request(int want) {   // smallest class that holds `want` entries
    int k = RP_POOL_MIN_CLASS;
    while ((1 << k) < want) ++k;
    return k;
}

__device__ __forceinline__ int class_of_block(int cap) {       // largest class that fits into `cap` entries, or -1
    if (cap < (1 << RP_POOL_MIN_CLASS)) return -1;
    return 31 - __clz(cap);
}

__device__ __forceinline__ int grown_class(int cap, int need) {
    return class_for_request(max(2 * cap, need + (need >> 2) + 4));
}

__device__ __forceinline__ bool wants_smaller_block(int cap, int need) { return cap >= 64 && 4 * need <= cap; }

__device__ __forceinline__ int shrunk_class(int need) { return class_for_request(2 * need + 8); }

// takes a block of class k from the free list; -1 if the list is empty
__device__ __forceinline__ long long take_block(const Side& sd, int k) {
    const int old = atomicSub(&sd.free_cnt[k], 1);
    if (old >= 1) return sd.free_blk[(size_t)k * RP_POOL_LIST_CAP + (old - 1)];
    atomicAdd(&sd.free_cnt[k], 1);
    return -1;
}

// Rows whose additions do not fit: list them and count the blocks they will take, by class.  Rows
// that deletions leave nearly empty: list them for a move to a smaller block.
__device__ __forceinline__ void d_plan_growth(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in,
                              int32_t* grow_out, int32_t* grow_in, int32_t* shrink_out, int32_t* shrink_in,
                              int tid, int nthreads) {
    if (ctl->abort) return;
    int n = ctl->n_rec;
    for (int i = tid; i < 2 * n; i += nthreads) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (x.rank[s] != 0) continue;   // one record per row and kind of change
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        int need = sd.deg[row] - sd.cnt_del[row] + sd.cnt_add[row];
        if (x.sign > 0) {
            if (need > sd.cap[row]) {
                int g = atomicAdd(&ctl->n_grow[s], 1);
                (s ? grow_in : grow_out)[g] = row;
                atomicAdd(&ctl->grow_demand[s][grown_class(sd.cap[row], need)], 1);
            }
        } else if (need <= sd.cap[row] && wants_smaller_block(sd.cap[row], need)) {
            int g = atomicAdd(&ctl->n_shrink[s], 1);
            (s ? shrink_in : shrink_out)[g] = row;
        }
    }
}

// what the growing rows cannot take from the free lists must fit into the never-used tail
__device__ __forceinline__ void d_plan_check(Ctl* ctl, Side out, Side in) {
    if (ctl->abort) return;
    for (int s = 0; s < 2; ++s) {
        const Side& sd = s ? in : out;
        unsigned long long need = 0;
        for (int k = RP_POOL_MIN_CLASS; k < RP_POOL_CLASSES; ++k) {
            const int short_of = ctl->grow_demand[s][k] - sd.free_cnt[k];
            if (short_of > 0) need += (unsigned long long)short_of << k;
        }
        ctl->pool_need[s] = need;
        if (ctl->pool_next[s] + need > (unsigned long long)sd.col_size) {
            ctl->err = (int)RIPPLE_ERR_CAPACITY;
            ctl->abort = 1;
        }
    }
}

// n sizes the launches (the number of operations given, or the batch capacity if vertex deletions
// may multiply them); the kernels read the actual counts from the control block
void graph_batch_classify(Ctx* c, int n) {
    if (n <= 0) return;
    const int T = 256;
    const int grid_ops = std::min(div_up(n, T), c->n_sm * 8);
    if (c->may_expand) {   // a host batch known to hold no vertex deletion skips the expansion
        RP_LAUNCH(c, k_expand_plan, grid_ops, T, 0, c->ups_dev, c->N, (long long)c->max_batch, c->ctl, c->side[0],
                  c->side[1], c->vjobs);
        RP_LAUNCH(c, k_expand_copy, std::min(n, c->n_sm * 4), T, 0, c->ups_dev, c->op_seq, c->ctl, c->side[0],
                  c->side[1], c->vjobs);
    }
    RP_LAUNCH(c, k_classify, grid_ops, T, 0, c->ups_dev, c->op_seq, c->N, c->ctl, c->hkeys, c->hwin,
              c->hsize - 1, c->op_slot, c->feat_last, c->vdel_seq, (int)(c->n_local > 0));
    int grid = std::min(n, c->n_sm * 8);
    RP_LAUNCH(c, k_resolve, grid, T, 0, c->ups_dev, c->op_seq, c->ctl, c->hwin, c->op_slot, c->feat_last,
              c->vdel_seq, c->side[0], c->side[1], c->rec, c->bitmap,
              (const float*)(c->has_opw ? c->opw_dev : nullptr), c->grow_list[0], c->grow_list[1],
              c->shrink_list[0], c->shrink_list[1], (const uint8_t*)(c->has_silent ? c->silent_dev : nullptr));
}

// ---------------------------------------------------------------------------------------------
// mutation
// ---------------------------------------------------------------------------------------------
#define FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row)                                                  \
    int n_ = (ctl)->n_rec;                                                                        \
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < 2 * n_; i += gridDim.x * blockDim.x)

__device__ __forceinline__ void d_del_mark(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) {
    if (ctl->abort) return;
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (x.sign > 0) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        sd.col[sd.start[row] + x.pos[s]] = RP_TOMB;
    }
}

__device__ __forceinline__ void d_del_tail_read(Ctl* ctl, Rec* rec, Side out, Side in) {
    if (ctl->abort) return;
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        Rec& x = rec[i >> 1];
        if (x.sign > 0) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        int new_deg = sd.deg[row] - sd.cnt_del[row];
        x.tail_val[s] = sd.col[sd.start[row] + new_deg + x.rank[s]];
        if (sd.w) x.tail_w[s] = sd.w[sd.start[row] + new_deg + x.rank[s]];
    }
}

__device__ __forceinline__ void d_del_tail_pack(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) {
    if (ctl->abort) return;
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (x.sign > 0 || x.tail_val[s] == RP_TOMB) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        int new_deg = sd.deg[row] - sd.cnt_del[row];
        int t = atomicAdd(&sd.tick_a[row], 1);
        sd.col[sd.start[row] + new_deg + t] = x.tail_val[s];
        if (sd.w) sd.w[sd.start[row] + new_deg + t] = x.tail_w[s];
    }
}

__device__ __forceinline__ void d_del_fill(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) {
    if (ctl->abort) return;
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (x.sign > 0) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        int new_deg = sd.deg[row] - sd.cnt_del[row];
        if (x.pos[s] >= new_deg) continue;
        int t = atomicAdd(&sd.tick_b[row], 1);
        sd.col[sd.start[row] + x.pos[s]] = sd.col[sd.start[row] + new_deg + t];
        if (sd.w) sd.w[sd.start[row] + x.pos[s]] = sd.w[sd.start[row] + new_deg + t];
    }
}

// Moves rows into new blocks.  Growing rows: a block of the planned class from the free list, else
// from the never-used tail (the plan has checked that it fits).  One warp per row; a row of more
// than GROW_BLOCK_ROW entries is left to a second pass in which a whole block copies it.  The last
// block to finish then moves the shrinking rows, which take from the free lists or from what the
// growing rows have left of the never-used tail (a row that finds no block stays where it is and
// is looked at again when it is next touched).  The blocks left behind are noted in moved_start / moved_cap and returned to the free
// lists by k_commit_degrees.
constexpr int GROW_BLOCK_ROW = 2048;

__device__ __forceinline__ void move_row(Side& sd, int row, long long off, int ncap, int live, int tid, int nthreads) {
    const int64_t old = sd.start[row];
    for (int j = tid; j < live; j += nthreads) sd.col[off + j] = sd.col[old + j];
    if (sd.w)
        for (int j = tid; j < live; j += nthreads) sd.w[off + j] = sd.w[old + j];
}

__device__ __forceinline__ void d_grow_rows(Ctl* ctl, Side out, Side in, const int32_t* __restrict__ grow_out, const int32_t* __restrict__ grow_in,
            const int32_t* __restrict__ shrink_out, const int32_t* __restrict__ shrink_in, int64_t* moved_start,
            int32_t* moved_cap) {
    if (ctl->abort) return;
    __shared__ long long s_off;
    __shared__ int s_last;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    const int n0 = ctl->n_grow[0], n1 = ctl->n_grow[1];
    for (int pass = 0; pass < 2; ++pass) {
        const int first = pass ? (int)blockIdx.x : warp, step = pass ? (int)gridDim.x : nwarps;
        for (int g = first; g < n0 + n1; g += step) {
            const int s = g >= n0;
            Side& sd = s ? in : out;
            const int row = s ? grow_in[g - n0] : grow_out[g];
            const int live = sd.deg[row] - sd.cnt_del[row];
            if ((live > GROW_BLOCK_ROW) != (pass == 1)) continue;
            const int k = grown_class(sd.cap[row], live + sd.cnt_add[row]);
            const int ncap = 1 << k;
            long long off = 0;
            if (pass ? threadIdx.x == 0 : lane == 0) {
                off = take_block(sd, k);
                if (off >= 0) atomicAdd(&ctl->pool_free[s], (unsigned long long)(-(long long)ncap));
                else off = (long long)atomicAdd(&ctl->pool_next[s], (unsigned long long)ncap);
                moved_start[g] = sd.start[row];
                moved_cap[g] = sd.cap[row];
                if (pass) s_off = off;
            }
            if (pass) { __syncthreads(); off = s_off; move_row(sd, row, off, ncap, live, threadIdx.x, blockDim.x); __syncthreads(); }
            else { off = __shfl_sync(FULL, off, 0); move_row(sd, row, off, ncap, live, lane, 32); __syncwarp(); }
            if (pass ? threadIdx.x == 0 : lane == 0) { sd.start[row] = (int64_t)off; sd.cap[row] = ncap; }
        }
    }
    const int m0 = ctl->n_shrink[0], m1 = ctl->n_shrink[1];
    if (m0 + m1 == 0) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&ctl->grow_done, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int g = threadIdx.x >> 5; g < m0 + m1; g += blockDim.x >> 5) {
        const int s = g >= m0;
        Side& sd = s ? in : out;
        const int row = s ? shrink_in[g - m0] : shrink_out[g];
        const int live = sd.deg[row] - sd.cnt_del[row];
        const int k = shrunk_class(live + sd.cnt_add[row]);
        const int ncap = 1 << k;
        long long off = -1;
        if (lane == 0) {
            off = take_block(sd, k);
            if (off >= 0) atomicAdd(&ctl->pool_free[s], (unsigned long long)(-(long long)ncap));
            else {   // the growing rows have all been served: what is left of the never-used tail may be taken
                const unsigned long long at = atomicAdd(&ctl->pool_next[s], (unsigned long long)ncap);
                if (at + (unsigned long long)ncap <= (unsigned long long)sd.col_size) off = (long long)at;
                else atomicAdd(&ctl->pool_next[s], (unsigned long long)(-(long long)ncap));
            }
            moved_start[n0 + n1 + g] = sd.start[row];
            moved_cap[n0 + n1 + g] = off >= 0 ? sd.cap[row] : 0;   // 0: nothing left behind
        }
        off = __shfl_sync(FULL, off, 0);
        if (off < 0) continue;
        move_row(sd, row, off, ncap, live, lane, 32);
        __syncwarp();
        if (lane == 0) { sd.start[row] = (int64_t)off; sd.cap[row] = ncap; }
    }
}

__device__ __forceinline__ void d_add_write(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) {
    if (ctl->abort) return;
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (x.sign < 0) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        int live = sd.deg[row] - sd.cnt_del[row];
        sd.col[sd.start[row] + live + x.rank[s]] = s ? x.u : x.v;
        if (sd.w) sd.w[sd.start[row] + live + x.rank[s]] = x.w;
    }
}

__device__ __forceinline__ void d_commit_degrees(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in,
                                 int32_t* deg_out_old, const int64_t* __restrict__ moved_start,
                                 const int32_t* __restrict__ moved_cap) {
    if (ctl->abort) return;
    // the blocks that moved rows left behind go onto the free lists
    const int n0 = ctl->n_grow[0], n1 = ctl->n_grow[1], m0 = ctl->n_shrink[0], m1 = ctl->n_shrink[1];
    for (int g = blockIdx.x * blockDim.x + threadIdx.x; g < n0 + n1 + m0 + m1; g += gridDim.x * blockDim.x) {
        const int s = g < n0 + n1 ? g >= n0 : g - n0 - n1 >= m0;
        const Side& sd = s ? in : out;
        const int cap = moved_cap[g];
        if (cap <= 0) continue;
        const int k = class_of_block(cap);
        int kept = 0;
        if (k >= 0) {
            const int idx = atomicAdd(&sd.free_cnt[k], 1);
            if (idx < RP_POOL_LIST_CAP) {
                sd.free_blk[(size_t)k * RP_POOL_LIST_CAP + idx] = moved_start[g];
                kept = 1 << k;
            } else atomicSub(&sd.free_cnt[k], 1);
        }
        if (kept) atomicAdd(&ctl->pool_free[s], (unsigned long long)kept);
        if (cap > kept) atomicAdd(&ctl->pool_lost[s], (unsigned long long)(cap - kept));
    }
    FOR_EACH_REC_SIDE(ctl, i, s, x, sd, row) {
        int s = i & 1;
        const Rec& x = rec[i >> 1];
        if (!x.rep[s]) continue;
        const Side& sd = s ? in : out;
        int row = s ? x.v : x.u;
        sd.deg[row] = sd.deg[row] - sd.cnt_del[row] + sd.cnt_add[row];
        if (s == 0) deg_out_old[row] = x.deg_out_old;
    }
}

// The kernels of the row update, one launch each ...
__global__ void k_del_mark(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) { pdl_enter(); d_del_mark(ctl, rec, out, in); }
__global__ void k_del_tail_read(Ctl* ctl, Rec* rec, Side out, Side in) { pdl_enter(); d_del_tail_read(ctl, rec, out, in); }
__global__ void k_del_tail_pack(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) { pdl_enter(); d_del_tail_pack(ctl, rec, out, in); }
__global__ void k_del_fill(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) { pdl_enter(); d_del_fill(ctl, rec, out, in); }
__global__ void __launch_bounds__(256)
k_grow_rows(Ctl* ctl, Side out, Side in, const int32_t* __restrict__ grow_out, const int32_t* __restrict__ grow_in,
            const int32_t* __restrict__ shrink_out, const int32_t* __restrict__ shrink_in, int64_t* moved_start,
            int32_t* moved_cap) {
    pdl_enter();
    d_grow_rows(ctl, out, in, grow_out, grow_in, shrink_out, shrink_in, moved_start, moved_cap);
}
__global__ void k_add_write(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in) { pdl_enter(); d_add_write(ctl, rec, out, in); }
__global__ void k_commit_degrees(Ctl* ctl, const Rec* __restrict__ rec, Side out, Side in, int32_t* deg_out_old,
                                 const int64_t* __restrict__ moved_start, const int32_t* __restrict__ moved_cap) {
    pdl_enter();
    d_commit_degrees(ctl, rec, out, in, deg_out_old, moved_start, moved_cap);
}

// ... and all of them in one block, a barrier between the phases, for the batches that are replayed
// from a captured chain (up to RP_GRAPH_MAX_BATCH operations: a few hundred records at most, which one
// block handles in a single sweep per phase).  Small batches are bound by the number of launches.
__global__ void __launch_bounds__(1024)
k_mutate_small(Ctl* ctl, Rec* rec, Side out, Side in, const int32_t* __restrict__ grow_out,
               const int32_t* __restrict__ grow_in, const int32_t* __restrict__ shrink_out,
               const int32_t* __restrict__ shrink_in, int64_t* moved_start, int32_t* moved_cap, int32_t* deg_out_old) {
    pdl_enter();
    d_del_mark(ctl, rec, out, in);
    __syncthreads();
    d_del_tail_read(ctl, rec, out, in);
    __syncthreads();
    d_del_tail_pack(ctl, rec, out, in);
    __syncthreads();
    d_del_fill(ctl, rec, out, in);
    __syncthreads();
    d_grow_rows(ctl, out, in, grow_out, grow_in, shrink_out, shrink_in, moved_start, moved_cap);
    __syncthreads();
    d_add_write(ctl, rec, out, in);
    __syncthreads();
    d_commit_degrees(ctl, rec, out, in, deg_out_old, moved_start, moved_cap);
}

// A batch of a handful of updates, none of them a vertex deletion, for models whose hop-0 senders are exactly
// the vertices with a feature update: control block reset, classification, resolution and planning, the row
// update, the list A_0 (sorted in shared memory from the winning feature operations: no sweep of the
// frontier bitmap), the feature rows with their old values or deltas, and the sender list of hop 1 with its
// out-degree prefix -- nine launches of the general chain -- in one block with barriers in between.
__global__ void __launch_bounds__(1024)
k_apply_small(Ctl* ctl, const int* params, const ripple_update* __restrict__ ups, const int32_t* __restrict__ op_seq, int N,
              unsigned long long* hkeys, unsigned long long* hwin, int hmask, int32_t* op_slot, int32_t* feat_last,
              int32_t* vdel_seq, Side out, Side in, Rec* rec, uint32_t* bitmap, const float* __restrict__ op_w,
              int32_t* grow_out, int32_t* grow_in, int32_t* shrink_out, int32_t* shrink_in, int64_t* moved_start,
              int32_t* moved_cap, int32_t* deg_out_old, const float* __restrict__ feat, int d0, float* H0, int ld,
              float* D, int keep_old, int32_t* A0, int build_senders, int32_t* senders, int32_t* posmap, int64_t* coff) {
    pdl_enter();
    __shared__ int s_ids[RP_TINY_BATCH];
    __shared__ int s_n;
    if (threadIdx.x == 0) { d_ctl_reset(ctl, params); s_n = 0; }
    __syncthreads();
    d_classify(ups, op_seq, N, ctl, hkeys, hwin, hmask, op_slot, feat_last, vdel_seq, 0);
    __syncthreads();
    d_resolve(ups, op_seq, ctl, hwin, op_slot, feat_last, vdel_seq, out, in, rec, bitmap, op_w, grow_out, grow_in,
              shrink_out, shrink_in, nullptr);
    __syncthreads();
    d_del_mark(ctl, rec, out, in);
    __syncthreads();
    d_del_tail_read(ctl, rec, out, in);
    __syncthreads();
    d_del_tail_pack(ctl, rec, out, in);
    __syncthreads();
    d_del_fill(ctl, rec, out, in);
    __syncthreads();
    d_grow_rows(ctl, out, in, grow_out, grow_in, shrink_out, shrink_in, moved_start, moved_cap);
    __syncthreads();
    d_add_write(ctl, rec, out, in);
    __syncthreads();
    d_commit_degrees(ctl, rec, out, in, deg_out_old, moved_start, moved_cap);
    __syncthreads();
    if (ctl->abort) return;
    // A_0: the vertices whose last feature operation this is, ascending
    const int n = ctl->n_ops;
    if ((int)threadIdx.x < n) {
        const ripple_update op = ups[threadIdx.x];
        if (op.op == RIPPLE_OP_SET_FEATURE && feat_last[op.u] == (int)threadIdx.x) {
            s_ids[atomicAdd(&s_n, 1)] = op.u;
            atomicAnd(&bitmap[op.u >> 5], ~(1u << (op.u & 31)));   // (resolution marked it for the general chain's sweep)
        }
    }
    __syncthreads();
    const int na = s_n;
    int mine = -1, rank = 0;
    if ((int)threadIdx.x < na) {
        mine = s_ids[threadIdx.x];
        for (int k = 0; k < na; ++k) rank += s_ids[k] < mine;
    }
    __syncthreads();
    if (mine >= 0) { s_ids[rank] = mine; A0[rank] = mine; }
    if (threadIdx.x == 0) { ctl->nA[0] = na; if (build_senders) ctl->nC[0] = na; }
    __syncthreads();
    // feature rows: one warp per vertex of A_0
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = warp; i < na; i += (int)(blockDim.x >> 5)) {
        const int v = s_ids[i];
        const float* src = feat + (size_t)ups[feat_last[v]].v * d0;
        for (int k = lane; k < ld; k += 32) {
            const float x = k < d0 ? src[k] : 0.f;
            const float o = H0[(size_t)v * ld + k];
            D[(size_t)i * ld + k] = keep_old ? o : x - o;
            H0[(size_t)v * ld + k] = x;
        }
    }
    // senders of hop 1 = A_0, with the prefix of their out-degrees (max / min aggregation lists its own: the rows
    // of A_0 whose values really changed)
    if (build_senders && threadIdx.x == 0) {
        int64_t sum = 0;
        for (int i = 0; i < na; ++i) {
            const int v = s_ids[i];
            senders[i] = v;
            posmap[v] = i;
            coff[i] = sum;
            sum += out.deg[v];
        }
        coff[na] = sum;
        ctl->E[1] = (unsigned long long)sum;
    }
}

void graph_batch_apply_small(Ctx* c, int n) {
    (void)n;
    Side& o = c->side[0];
    Side& i = c->side[1];
    RP_LAUNCH(c, k_apply_small, 1, 1024, 0, c->ctl, (const int*)c->params_dev, (const ripple_update*)c->ups_dev,
              (const int32_t*)c->op_seq, c->N, c->hkeys, c->hwin, c->hsize - 1, c->op_slot, c->feat_last, c->vdel_seq, o, i,
              c->rec, c->bitmap, (const float*)(c->has_opw ? c->opw_dev : nullptr), c->grow_list[0], c->grow_list[1],
              c->shrink_list[0], c->shrink_list[1], c->moved_start, c->moved_cap, c->deg_out_old,
              (const float*)c->feat_dev, c->d[0], c->H[0], c->ld[0], c->D[0], (int)(c->attention || rp_monotonic(c->agg)),
              c->A[0], (int)!rp_monotonic(c->agg), c->Clist[0], c->posmap, c->coff);
}

void graph_batch_mutate(Ctx* c, int n) {
    if (n <= 0) return;
    const int T = 256;
    int grid = std::min(div_up(2 * n, T), c->n_sm * 8);
    Side& o = c->side[0];
    Side& i = c->side[1];
    if (n <= RP_GRAPH_MAX_BATCH) {
        RP_LAUNCH(c, k_mutate_small, 1, 1024, 0, c->ctl, c->rec, o, i, c->grow_list[0], c->grow_list[1],
                  c->shrink_list[0], c->shrink_list[1], c->moved_start, c->moved_cap, c->deg_out_old);
        return;
    }
    RP_LAUNCH(c, k_del_mark, grid, T, 0, c->ctl, c->rec, o, i);
    RP_LAUNCH(c, k_del_tail_read, grid, T, 0, c->ctl, c->rec, o, i);
    RP_LAUNCH(c, k_del_tail_pack, grid, T, 0, c->ctl, c->rec, o, i);
    RP_LAUNCH(c, k_del_fill, grid, T, 0, c->ctl, c->rec, o, i);
    RP_LAUNCH(c, k_grow_rows, std::min(div_up(2 * n, T / 32), c->n_sm * 8), T, 0, c->ctl, o, i,
              c->grow_list[0], c->grow_list[1], c->shrink_list[0], c->shrink_list[1], c->moved_start, c->moved_cap);
    RP_LAUNCH(c, k_add_write, grid, T, 0, c->ctl, c->rec, o, i);
    RP_LAUNCH(c, k_commit_degrees, grid, T, 0, c->ctl, c->rec, o, i, c->deg_out_old, c->moved_start, c->moved_cap);
}

// ---------------------------------------------------------------------------------------------
// per-batch scratch back to its resting state (runs for rejected batches too)
// ---------------------------------------------------------------------------------------------
__global__ void k_cleanup(const ripple_update* __restrict__ ups, int N, Ctl* ctl,
                          const Rec* __restrict__ rec, Side out, Side in, unsigned long long* hkeys,
                          unsigned long long* hwin, const int32_t* __restrict__ op_slot, int32_t* feat_last,
                          int32_t* vdel_seq, int32_t* deg_out_old, uint32_t* bitmap) {
    pdl_enter();
    const int n_rec = ctl->n_rec, n = ops_total(ctl);
    if (blockIdx.x == 0 && threadIdx.x == 0 && !ctl->abort) ctl->num_edges += ctl->n_add - ctl->n_del;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < max(n, n_rec); i += gridDim.x * blockDim.x) {
        if (i < n) {
            ripple_update op = ups[i];
            int slot = op_slot[i];
            if (slot >= 0) { hkeys[slot] = 0ull; hwin[slot] = 0ull; }
            if ((op.op == RIPPLE_OP_SET_FEATURE || op.op == RIPPLE_OP_DEL_VERTEX) && (unsigned)op.u < (unsigned)N) {
                feat_last[op.u] = -1;
                if (op.op == RIPPLE_OP_DEL_VERTEX) vdel_seq[op.u] = -1;
                if (ctl->abort) atomicAnd(&bitmap[op.u >> 5], ~(1u << (op.u & 31)));
            }
        }
        if (i < n_rec) {
            const Rec& x = rec[i];
            out.cnt_del[x.u] = 0; out.cnt_add[x.u] = 0; out.tick_a[x.u] = 0; out.tick_b[x.u] = 0; out.touch[x.u] = 0;
            in.cnt_del[x.v] = 0; in.cnt_add[x.v] = 0; in.tick_a[x.v] = 0; in.tick_b[x.v] = 0; in.touch[x.v] = 0;
            deg_out_old[x.u] = -1;
        }
    }
}

void graph_batch_cleanup(Ctx* c, int n) {
    if (n <= 0) return;
    const int T = 256;
    RP_LAUNCH(c, k_cleanup, std::min(div_up(n, T), c->n_sm * 8), T, 0, c->ups_dev, c->N, c->ctl, c->rec,
              c->side[0], c->side[1], c->hkeys, c->hwin, c->op_slot, c->feat_last, c->vdel_seq, c->deg_out_old,
              c->bitmap);
}

// ---------------------------------------------------------------------------------------------
// canonical export (parity checks)
// ---------------------------------------------------------------------------------------------
__global__ void k_export_rows(int N, Side out, const int64_t* __restrict__ rowptr, int32_t* col, float* weight) {
    pdl_enter();
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int v = warp; v < N; v += nwarps) {
        int64_t base = out.start[v], dst = rowptr[v];
        int deg = out.deg[v];
        for (int j = lane_id(); j < deg; j += 32) {
            col[dst + j] = out.col[base + j];
            if (weight) weight[dst + j] = out.w ? out.w[base + j] : 1.0f;
        }
    }
}

cudaError_t graph_export(Ctx* c, int64_t* rowptr, int32_t* col, float* weight, int64_t col_capacity, int64_t* n_edges) {
    cudaError_t e;
    const int N = c->N;
    std::vector<int32_t> deg((size_t)N);
    if ((e = cudaMemcpyAsync(deg.data(), c->side[0].deg, sizeof(int32_t) * (size_t)N, cudaMemcpyDeviceToHost, c->stream))) return e;
    if ((e = cudaStreamSynchronize(c->stream))) return e;
    rowptr[0] = 0;
    for (int v = 0; v < N; ++v) rowptr[v + 1] = rowptr[v] + deg[v];
    *n_edges = rowptr[N];
    if (rowptr[N] > col_capacity) return cudaErrorInvalidValue;
    if (rowptr[N] == 0) return cudaSuccess;
    int64_t* rp_dev = nullptr;
    int32_t* col_dev = nullptr;
    float* w_dev = nullptr;
    if ((e = cudaMalloc(&rp_dev, sizeof(int64_t) * ((size_t)N + 1)))) return e;
    if ((e = cudaMalloc(&col_dev, sizeof(int32_t) * (size_t)rowptr[N]))) { cudaFree(rp_dev); return e; }
    if (weight && (e = cudaMalloc(&w_dev, sizeof(float) * (size_t)rowptr[N]))) { cudaFree(rp_dev); cudaFree(col_dev); return e; }
    e = cudaMemcpyAsync(rp_dev, rowptr, sizeof(int64_t) * ((size_t)N + 1), cudaMemcpyHostToDevice, c->stream);
    if (!e) {
        RP_LAUNCH(c, k_export_rows, c->n_sm * 8, 256, 0, N, c->side[0], rp_dev, col_dev, w_dev);
        e = cudaMemcpyAsync(col, col_dev, sizeof(int32_t) * (size_t)rowptr[N], cudaMemcpyDeviceToHost, c->stream);
        if (!e && weight)
            e = cudaMemcpyAsync(weight, w_dev, sizeof(float) * (size_t)rowptr[N], cudaMemcpyDeviceToHost, c->stream);
    }
    if (!e) e = cudaStreamSynchronize(c->stream);
    cudaFree(rp_dev);
    cudaFree(col_dev);
    cudaFree(w_dev);
    if (e) return e;
    if (!weight) {
#pragma omp parallel for schedule(dynamic, 1024)
        for (int v = 0; v < N; ++v) std::sort(col + rowptr[v], col + rowptr[v + 1]);
        return cudaSuccess;
    }
    // rows sorted by neighbour id, the weights moving with their entries
#pragma omp parallel
    {
        std::vector<std::pair<int32_t, float>> tmp;
#pragma omp for schedule(dynamic, 1024)
        for (int v = 0; v < N; ++v) {
            const int64_t b = rowptr[v], n = rowptr[v + 1] - b;
            tmp.resize((size_t)n);
            for (int64_t j = 0; j < n; ++j) tmp[(size_t)j] = {col[b + j], weight[b + j]};
            std::sort(tmp.begin(), tmp.end(), [](const std::pair<int32_t, float>& x, const std::pair<int32_t, float>& y) { return x.first < y.first; });
            for (int64_t j = 0; j < n; ++j) { col[b + j] = tmp[(size_t)j].first; weight[b + j] = tmp[(size_t)j].second; }
        }
    }
    return cudaSuccess;
}

}  // namespace rp

// ---------------------------------------------------------------------------------------------
// allocation-free export
// ---------------------------------------------------------------------------------------------
// Same result as ripple_export_graph, for callers that must not allocate device memory.  The
// staging that ripple_export_graph obtains with cudaMalloc on every call (a device copy of the
// row pointers and a packed copy of the column indices) lives here in two file-scope device
// arrays of fixed size.  Every GPU that loads the library carries them (about 10 MB) until the
// process exits.  In host code the arrays' names are host-side stand-ins, not device addresses:
// the addresses the kernel receives come from cudaGetSymbolAddress, taken once per device.
#include <cstdio>
#include <cstring>
#include <mutex>

namespace rp {

constexpr int64_t STATIC_MAX_VERTICES = 1 << 18;  // 262 144
constexpr int64_t STATIC_MAX_EDGES = 1 << 21;     // 2 097 152

static __device__ __align__(256) int64_t g_static_rowptr[STATIC_MAX_VERTICES + 1];
static __device__ __align__(256) int32_t g_static_col[STATIC_MAX_EDGES];

struct StaticScratch {
    int64_t* rowptr = nullptr;
    int32_t* col = nullptr;
    bool ready = false;
};
constexpr int STATIC_MAX_DEVICES = 64;
static StaticScratch g_static[STATIC_MAX_DEVICES];
static std::mutex g_static_mu;

// once per device, with that device current
static cudaError_t static_scratch(int device, StaticScratch* out) {
    if (device < 0 || device >= STATIC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticScratch& s = g_static[device];
    if (!s.ready) {
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&s.rowptr), g_static_rowptr);
        if (e != cudaSuccess) return e;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&s.col), g_static_col);
        if (e != cudaSuccess) return e;
        s.ready = true;
    }
    *out = s;
    return cudaSuccess;
}

}  // namespace rp

extern "C" ripple_status ripple_export_graph_static(ripple_ctx* ctx, int64_t* rowptr, int32_t* col,
                                                    int64_t col_capacity) {
    using namespace rp;
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !rowptr || (!col && col_capacity > 0)) return RIPPLE_ERR_INVALID_ARG;
    const int N = c->N;
    if (N > STATIC_MAX_VERTICES) {
        snprintf(c->err, sizeof(c->err),
                 "ripple_export_graph_static handles at most %lld vertices, the graph has %d; "
                 "use ripple_export_graph", (long long)STATIC_MAX_VERTICES, N);
        return RIPPLE_ERR_CAPACITY;
    }
    cudaError_t e = cudaSetDevice(c->device);
    StaticScratch sc;
    if (!e) e = static_scratch(c->device, &sc);
    // degrees land, as raw bytes, in the tail of the caller's rowptr buffer and are widened in place,
    // front to back: entry v is read (memcpy, so that no int64 object is ever read through an int32
    // pointer) before the store to rowptr[v + 1] can reach its bytes
    unsigned char* deg_bytes = reinterpret_cast<unsigned char*>(rowptr + N + 1) - sizeof(int32_t) * (size_t)N;
    if (!e) e = cudaMemcpyAsync(deg_bytes, c->side[0].deg, sizeof(int32_t) * (size_t)N, cudaMemcpyDeviceToHost, c->stream);
    if (!e) e = cudaStreamSynchronize(c->stream);
    if (e) {
        snprintf(c->err, sizeof(c->err), "ripple_export_graph_static: %s", cudaGetErrorString(e));
        return RIPPLE_ERR_CUDA;
    }
    rowptr[0] = 0;
    for (int v = 0; v < N; ++v) {
        int32_t d;
        memcpy(&d, deg_bytes + sizeof(int32_t) * (size_t)v, sizeof(int32_t));
        rowptr[v + 1] = rowptr[v] + (int64_t)d;
    }
    const int64_t E = rowptr[N];
    if (E > STATIC_MAX_EDGES) {
        snprintf(c->err, sizeof(c->err),
                 "ripple_export_graph_static handles at most %lld edges, the graph has %lld; "
                 "use ripple_export_graph", (long long)STATIC_MAX_EDGES, (long long)E);
        return RIPPLE_ERR_CAPACITY;
    }
    if (E > col_capacity) {
        snprintf(c->err, sizeof(c->err), "col_capacity %lld is smaller than the edge count %lld",
                 (long long)col_capacity, (long long)E);
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (E == 0) return RIPPLE_OK;
    e = cudaMemcpyAsync(sc.rowptr, rowptr, sizeof(int64_t) * ((size_t)N + 1), cudaMemcpyHostToDevice, c->stream);
    if (!e) {
        k_export_rows<<<c->n_sm * 8, 256, 0, c->stream>>>(N, c->side[0], sc.rowptr, sc.col, nullptr);
        e = cudaGetLastError();
    }
    if (!e) e = cudaMemcpyAsync(col, sc.col, sizeof(int32_t) * (size_t)E, cudaMemcpyDeviceToHost, c->stream);
    if (!e) e = cudaStreamSynchronize(c->stream);
    if (e) {
        snprintf(c->err, sizeof(c->err), "ripple_export_graph_static: %s", cudaGetErrorString(e));
        return RIPPLE_ERR_CUDA;
    }
    for (int v = 0; v < N; ++v) std::sort(col + rowptr[v], col + rowptr[v + 1]);
    return RIPPLE_OK;
}
