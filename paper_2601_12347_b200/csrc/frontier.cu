// Per-layer affected sets (the hops of the propagation tree, Sec. 3.3) and sender lists.
//
//   A_l = sinks(dE) U Out_new(C_{l-1}) U (self term ? A_{l-1} : {})        l = 1..L,  A_0 = F
//   C_l = A_l U (source coefficients depend on out-degree ? sources(dE) : {})
//
// Membership is collected in an N-bit bitmap (duplicates vanish in the OR) and turned into an
// ascending id list by a popcount scan; the bitmap is cleared by the same pass.  Out-lists are
// walked edge-balanced: the concatenated out-edges of the sender list are cut into equal chunks
// and each warp finds its rows by binary search in the degree prefix, so a hub costs what its
// edges cost, not one long warp.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>

namespace rp {

constexpr int SCAN_T = 256;
constexpr int SCAN_ITEMS = 4;
constexpr int SCAN_TILE = SCAN_T * SCAN_ITEMS;

// ---------------------------------------------------------------------------------------------
// exclusive prefix sum of deg[list[i]] (or deg[i]) over i < n, n known only on the device
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int scan_count(const int* n_dev, int n_host) { return n_dev ? *n_dev : n_host; }

// Tile sums; the last block to finish turns them into exclusive tile prefixes and writes the total
// (one launch instead of two: the chain of a small batch is bound by the number of launches).
// If `senders` is given the listed vertices are, in the same pass, copied there and entered into the
// position map, and their number into *n_senders: the sender list of a hop whose senders are exactly
// the affected vertices (no launch of its own for that).
__global__ void k_scan_tiles(const int32_t* __restrict__ list, const int* n_dev, int n_host,
                             const int32_t* __restrict__ deg, int64_t* tile_sums, int64_t* out,
                             unsigned long long* total_dev, int* done, int32_t* senders, int32_t* posmap,
                             int* n_senders) {
    pdl_enter();
    __shared__ int64_t scratch[33];
    __shared__ int s_last;
    int n = scan_count(n_dev, n_host);
    int n_tiles = (n + SCAN_TILE - 1) / SCAN_TILE;
    if (senders && blockIdx.x == 0 && threadIdx.x == 0) *n_senders = n;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        int64_t s = 0;
#pragma unroll
        for (int k = 0; k < SCAN_ITEMS; ++k) {
            int i = t * SCAN_TILE + k * SCAN_T + threadIdx.x;
            if (i < n) {
                const int v = list ? list[i] : i;
                s += deg[v];
                if (senders) { senders[i] = v; posmap[v] = i; }
            }
        }
        int64_t total;
        block_exclusive_scan<int64_t>(s, scratch, total);
        if (threadIdx.x == 0) tile_sums[t] = total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(done, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x == 0) *done = 0;   // ready for the next scan
    int64_t carry = 0;
    for (int t0 = 0; t0 < n_tiles; t0 += blockDim.x) {
        int t = t0 + threadIdx.x;
        int64_t x = t < n_tiles ? tile_sums[t] : 0, total;
        int64_t ex = block_exclusive_scan<int64_t>(x, scratch, total);
        if (t < n_tiles) tile_sums[t] = carry + ex;
        carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        out[n] = carry;
        if (total_dev) *total_dev = (unsigned long long)carry;
    }
}

__global__ void k_scan_write(const int32_t* __restrict__ list, const int* n_dev, int n_host,
                             const int32_t* __restrict__ deg, const int64_t* __restrict__ tile_sums,
                             int64_t* out) {
    pdl_enter();
    __shared__ int64_t scratch[33];
    int n = scan_count(n_dev, n_host);
    int n_tiles = (n + SCAN_TILE - 1) / SCAN_TILE;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        // thread owns SCAN_ITEMS consecutive items so the block scan yields their base directly
        int i0 = t * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
        int64_t x[SCAN_ITEMS], s = 0;
#pragma unroll
        for (int k = 0; k < SCAN_ITEMS; ++k) {
            int i = i0 + k;
            x[k] = i < n ? deg[list ? list[i] : i] : 0;
            s += x[k];
        }
        int64_t total;
        int64_t base = tile_sums[t] + block_exclusive_scan<int64_t>(s, scratch, total);
#pragma unroll
        for (int k = 0; k < SCAN_ITEMS; ++k) {
            int i = i0 + k;
            if (i < n) out[i] = base;
            base += x[k];
        }
        __syncthreads();
    }
}

static void scan_degrees_and_copy(Ctx* c, const int32_t* list, const int* n_dev, int n_host, const int32_t* deg,
                                  int64_t* out, unsigned long long* total_dev, int32_t* senders, int* n_senders) {
    int max_tiles = std::max(1, div_up(c->N, SCAN_TILE));
    int grid = std::min(max_tiles, c->n_sm * 8);
    RP_LAUNCH(c, k_scan_tiles, grid, SCAN_T, 0, list, n_dev, n_host, deg, c->tile_sums, out, total_dev, c->scan_done,
              senders, c->posmap, n_senders);
    RP_LAUNCH(c, k_scan_write, grid, SCAN_T, 0, list, n_dev, n_host, deg, c->tile_sums, out);
}

void scan_degrees(Ctx* c, const int32_t* list, const int* n_dev, int n_host, const int32_t* deg,
                  int64_t* out, unsigned long long* total_dev) {
    scan_degrees_and_copy(c, list, n_dev, n_host, deg, out, total_dev, nullptr, nullptr);
}

// ---------------------------------------------------------------------------------------------
// bitmap -> ascending id list (clears the bitmap)
// ---------------------------------------------------------------------------------------------
constexpr int CMP_T = 256;  // one word per thread

__global__ void k_bitmap_tile_counts(const uint32_t* __restrict__ bitmap, int n_words, int* tile_cnt) {
    pdl_enter();
    __shared__ int scratch[33];
    int w = blockIdx.x * CMP_T + threadIdx.x;
    int pc = w < n_words ? __popc(bitmap[w]) : 0;
    int total;
    block_exclusive_scan<int>(pc, scratch, total);
    if (threadIdx.x == 0) tile_cnt[blockIdx.x] = total;
}

__global__ void k_bitmap_compact(uint32_t* bitmap, int n_words, const int* __restrict__ tile_cnt,
                                 int32_t* list, int* count_out, const int32_t* __restrict__ deg_in,
                                 unsigned long long* pull_work) {
    pdl_enter();
    __shared__ int scratch[33];
    __shared__ int tile_base;
    __shared__ unsigned long long work;
    // base of this tile: sum of the counts of the tiles before it
    int part = 0;
    for (int t = threadIdx.x; t < (int)blockIdx.x; t += CMP_T) part += tile_cnt[t];
    int total;
    block_exclusive_scan<int>(part, scratch, total);
    if (threadIdx.x == 0) { tile_base = total; work = 0ull; }
    __syncthreads();
    int w = blockIdx.x * CMP_T + threadIdx.x;
    uint32_t bits = w < n_words ? bitmap[w] : 0u;
    if (bits) bitmap[w] = 0u;
    int pc = __popc(bits);
    int off = tile_base + block_exclusive_scan<int>(pc, scratch, total);
    unsigned long long my_work = 0;
    while (bits) {
        int b = __ffs(bits) - 1;
        bits &= bits - 1;
        int v = (w << 5) + b;
        list[off++] = v;
        if (deg_in) my_work += (unsigned long long)deg_in[v];
    }
    if (pull_work) {
        my_work = warp_sum(my_work);
        if (lane_id() == 0 && my_work) atomicAdd(&work, my_work);
        __syncthreads();
        if (threadIdx.x == 0 && work) atomicAdd(pull_work, work);
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) *count_out = tile_base + total;
}

void bitmap_to_list_from(Ctx* c, uint32_t* bitmap, int32_t* list, int* count_dev, unsigned long long* pull_work) {
    int tiles = div_up(c->n_words, CMP_T);
    int* tile_cnt = reinterpret_cast<int*>(c->tile_sums);  // scan scratch is free here
    RP_LAUNCH(c, k_bitmap_tile_counts, tiles, CMP_T, 0, bitmap, c->n_words, tile_cnt);
    RP_LAUNCH(c, k_bitmap_compact, tiles, CMP_T, 0, bitmap, c->n_words, tile_cnt, list, count_dev,
              pull_work ? c->side[1].deg : nullptr, pull_work);
}

static void bitmap_to_list(Ctx* c, int32_t* list, int* count_dev, unsigned long long* pull_work) {
    bitmap_to_list_from(c, c->bitmap, list, count_dev, pull_work);
}

// ---------------------------------------------------------------------------------------------
// marking
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_bit(uint32_t* bitmap, int v) {
    uint32_t m = 1u << (v & 31);
    if (!(bitmap[v >> 5] & m)) atomicOr(&bitmap[v >> 5], m);
}

constexpr int WALK_CHUNK = 256;  // edges per warp work item

__global__ void k_mark_frontier(Ctl* ctl, int l, int self_term, int walk, const int32_t* __restrict__ senders,
                                const int64_t* __restrict__ coff, Side out, const Rec* __restrict__ rec,
                                const int32_t* __restrict__ A_prev, uint32_t* bitmap) {
    pdl_enter();
    if (ctl->abort) return;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsize = gridDim.x * blockDim.x;
    // sinks of net edge changes are affected at every hop
    for (int i = gtid; i < ctl->n_rec; i += gsize) set_bit(bitmap, rec[i].v);
    if (self_term)
        for (int i = gtid; i < ctl->nA[l - 1]; i += gsize) set_bit(bitmap, A_prev[i]);
    // out-neighbours of the senders of the previous hop (the push scatter marks them itself)
    if (!walk || ctl->regather[l]) return;   // (a rebuilding hop marks bottom-up)
    const int nC = ctl->nC[l - 1];
    if (nC == 0) return;
    const int64_t E = coff[nC];
    const int warp = gtid >> 5, nwarps = gsize >> 5, lane = lane_id();
    for (int64_t e0 = (int64_t)warp * WALK_CHUNK; e0 < E; e0 += (int64_t)nwarps * WALK_CHUNK) {
        int64_t e1 = min(e0 + WALK_CHUNK, E);
        int i = upper_row(coff, nC, e0);
        int64_t e = e0;
        while (e < e1) {
            int64_t row_end = coff[i + 1];
            if (row_end <= e) { ++i; continue; }
            int64_t seg_end = min(e1, row_end);
            int64_t base = out.start[senders[i]] + (e - coff[i]);
            for (int64_t j = lane; j < seg_end - e; j += 32) set_bit(bitmap, out.col[base + j]);
            e = seg_end;
            ++i;
        }
    }
}

// Rebuilding hops mark bottom-up (the direction switch of a frontier search that has reached most
// of the graph): v belongs to Out_new(C_{l-1}) iff one of its in-neighbours is a sender.  With the
// senders owning most edges the first few probes of the position map settle almost every vertex,
// where walking the senders' out-lists would look up the bitmap once per edge (measured 1.2 ms on
// 123 M edges against 0.1 ms).  Four lanes per vertex probe the first 64 in-neighbours; the few
// vertices still undecided with longer lists are queued for a warp each.
constexpr int BU_LANES = 4, BU_FIRST = 64;

__global__ void __launch_bounds__(256)
k_mark_bottom_up(Ctl* ctl, int l, int N, Side in, const int32_t* __restrict__ posmap, uint32_t* bitmap,
                 int32_t* overflow, int* n_overflow) {
    pdl_enter();
    if (ctl->abort || !ctl->regather[l]) return;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, groups = (gridDim.x * blockDim.x) / BU_LANES;
    const int sub = threadIdx.x & (BU_LANES - 1);
    const unsigned group = 0xFu << ((threadIdx.x & 31) & ~(BU_LANES - 1));   // the four lanes that share a vertex
    for (int v = gtid / BU_LANES; v < N; v += groups) {
        const int deg = in.deg[v];
        if (deg == 0 || (bitmap[v >> 5] & (1u << (v & 31)))) continue;   // same outcome in all four lanes
        const int64_t base = in.start[v];
        const int lim = min(deg, BU_FIRST);
        bool hit = false;
        for (int j0 = 0; j0 < lim && !hit; j0 += BU_LANES) {
            const int j = j0 + sub;
            const bool mine = j < lim && posmap[in.col[base + j]] >= 0;
            hit = __any_sync(group, mine);
        }
        if (sub == 0) {
            if (hit) set_bit(bitmap, v);
            else if (deg > BU_FIRST) overflow[atomicAdd(n_overflow, 1)] = v;
        }
    }
}

__global__ void __launch_bounds__(256)
k_mark_bottom_up_long(Ctl* ctl, int l, Side in, const int32_t* __restrict__ posmap, uint32_t* bitmap,
                      const int32_t* __restrict__ overflow, const int* __restrict__ n_overflow) {
    pdl_enter();
    if (ctl->abort || !ctl->regather[l]) return;
    const int n = *n_overflow;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int i = warp; i < n; i += nwarps) {
        const int v = overflow[i];
        const int deg = in.deg[v];
        const int64_t base = in.start[v];
        bool hit = false;
        for (int j0 = BU_FIRST; j0 < deg && !hit; j0 += 32) {
            bool mine = j0 + lane < deg && posmap[in.col[base + j0 + lane]] >= 0;
            hit = __any_sync(FULL, mine);
        }
        if (hit && lane == 0) set_bit(bitmap, v);
    }
}

void frontier_seed_features(Ctx* c, int n) {
    (void)n;
    bitmap_to_list(c, c->A[0], &c->ctl->nA[0], nullptr);
}

// Marks the members of A_l that do not come from walking the senders' out-lists (sinks of edge
// changes, A_{l-1} for models with a self term) and, if `walk`, those that do.
void frontier_mark(Ctx* c, int l, bool walk, int n) {
    // without a walk of its own (the push scatter marks the sinks it reaches) the rest of the marking rides
    // along with the last kernel of the hop's delta form; an empty batch has nothing to mark
    if (walk)
        RP_LAUNCH(c, k_mark_frontier, c->n_sm * 8, 256, 0, c->ctl, l, (int)c->self_term,
                  (int)walk, c->Clist[(l - 1) & 1], c->coff, c->side[0], c->rec, c->A[l - 1], c->bitmap);
    (void)n;
    if (!c->rebuild_armed[l]) return;
    // the list A_l is not built yet: its buffer holds the queue of undecided long rows
    RP_LAUNCH(c, k_mark_bottom_up, c->n_sm * 8, 256, 0, c->ctl, l, c->N, c->side[1], c->posmap, c->bitmap, c->A[l],
              &c->ctl->n_long[l]);
    RP_LAUNCH(c, k_mark_bottom_up_long, c->n_sm * 4, 256, 0, c->ctl, l, c->side[1], c->posmap, c->bitmap, c->A[l],
              &c->ctl->n_long[l]);
}

// The frontier of a hop in one block: words of the bitmap are dealt out in contiguous runs, one per thread, so
// that a block scan of the popcounts places every id.  For batches of a handful of updates on graphs whose
// bitmap one block can sweep (two launches of the general chain otherwise).
__global__ void __launch_bounds__(1024)
k_frontier_small(Ctl* ctl, int l, uint32_t* bitmap, int n_words, int32_t* list, const int32_t* __restrict__ deg_in) {
    pdl_enter();
    __shared__ int scratch_i[33];
    __shared__ unsigned long long s_work;
    if (ctl->abort) return;
    if (threadIdx.x == 0) s_work = 0ull;
    const int per = (n_words + (int)blockDim.x - 1) / (int)blockDim.x;
    const int w0 = min(n_words, (int)threadIdx.x * per), w1 = min(n_words, w0 + per);
    int pc = 0;
    for (int w = w0; w < w1; ++w) pc += __popc(bitmap[w]);
    int total;
    int off = block_exclusive_scan<int>(pc, scratch_i, total);
    unsigned long long work = 0;
    for (int w = w0; w < w1; ++w) {
        uint32_t bits = bitmap[w];
        if (!bits) continue;
        bitmap[w] = 0u;
        while (bits) {
            const int v = (w << 5) + __ffs(bits) - 1;
            bits &= bits - 1;
            list[off++] = v;
            work += (unsigned long long)deg_in[v];
        }
    }
    work = warp_sum(work);
    if (lane_id() == 0 && work) atomicAdd(&s_work, work);
    __syncthreads();
    if (threadIdx.x == 0) { ctl->nA[l] = total; ctl->pull_work[l] = s_work; }
}

// ... and the sender list made from it (C_l = A_l) with the prefix of the out-degrees, likewise in one block
__global__ void __launch_bounds__(1024)
k_senders_small(Ctl* ctl, int l, const int32_t* __restrict__ list, const int32_t* __restrict__ deg_out, int32_t* senders,
                int32_t* posmap, int64_t* coff) {
    pdl_enter();
    __shared__ int64_t scratch_l[33];
    if (ctl->abort) return;
    const int total = ctl->nA[l];
    int64_t carry = 0;
    for (int i0 = 0; i0 < total; i0 += (int)blockDim.x) {
        const int i = i0 + (int)threadIdx.x;
        int v = -1;
        int64_t d = 0;
        if (i < total) { v = list[i]; d = deg_out[v]; }
        int64_t sum;
        const int64_t ex = block_exclusive_scan<int64_t>(d, scratch_l, sum);
        if (i < total) { senders[i] = v; posmap[v] = i; coff[i] = carry + ex; }
        carry += sum;
    }
    if (threadIdx.x == 0) {
        coff[total] = carry;
        ctl->E[l + 1] = (unsigned long long)carry;
        ctl->nC[l] = total;
    }
}

// the members of A_l that no walk of out-lists finds: sinks of edge changes, A_{l-1} for models with a self term
void frontier_mark_extras(Ctx* c, int l) {
    RP_LAUNCH(c, k_mark_frontier, c->n_sm * 2, 256, 0, c->ctl, l, (int)c->self_term, 0, c->Clist[(l - 1) & 1], c->coff,
              c->side[0], c->rec, c->A[l - 1], c->bitmap);
}

void frontier_compact_small(Ctx* c, int l) {
    RP_LAUNCH(c, k_frontier_small, 1, 1024, 0, c->ctl, l, c->bitmap, c->n_words, c->A[l], (const int32_t*)c->side[1].deg);
}

void senders_build_small(Ctx* c, int l) {
    RP_LAUNCH(c, k_senders_small, 1, 1024, 0, c->ctl, l, (const int32_t*)c->A[l], (const int32_t*)c->side[0].deg,
              c->Clist[l & 1], c->posmap, c->coff);
}

void frontier_compact(Ctx* c, int l) {
    bitmap_to_list(c, c->A[l], &c->ctl->nA[l], &c->ctl->pull_work[l]);
}

// ---------------------------------------------------------------------------------------------
// sender lists
// ---------------------------------------------------------------------------------------------
__global__ void k_senders_from_affected(Ctl* ctl, int l, const int32_t* __restrict__ A, int32_t* senders,
                                        int32_t* posmap) {
    pdl_enter();
    if (ctl->abort) return;
    int n = ctl->nA[l];
    if (blockIdx.x == 0 && threadIdx.x == 0) ctl->nC[l] = n;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        int v = A[i];
        senders[i] = v;
        posmap[v] = i;
    }
}

__global__ void k_senders_release(Ctl* ctl, int l, const int32_t* __restrict__ senders, int32_t* posmap) {
    pdl_enter();
    int n = ctl->nC[l];
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        posmap[senders[i]] = -1;
}

void senders_build(Ctx* c, int l, int n) {
    int32_t* senders = c->Clist[l & 1];
    if (!c->src_norm) {
        // the senders are exactly the affected vertices: listed while their out-degrees are summed
        // (after a rejected batch every list is empty, so nothing needs the abort flag here)
        scan_degrees_and_copy(c, c->A[l], &c->ctl->nA[l], 0, c->side[0].deg, c->coff, &c->ctl->E[l + 1], senders,
                              &c->ctl->nC[l]);
        return;
    }
    RP_LAUNCH(c, k_senders_from_affected, c->n_sm * 4, 256, 0, c->ctl, l, c->A[l], senders, c->posmap);
    if (n > 0) extra_sender_rows(c, l, n);
    scan_degrees(c, senders, &c->ctl->nC[l], 0, c->side[0].deg, c->coff, &c->ctl->E[l + 1]);
}

void senders_release(Ctx* c, int l) {
    RP_LAUNCH(c, k_senders_release, c->n_sm * 4, 256, 0, c->ctl, l, c->Clist[l & 1], c->posmap);
}

}  // namespace rp
