// Monotonic aggregation (Sec. 3.4.2), max and min, for GraphConv and SAGE layers.
//
// The cached aggregate S^l_v is the element-wise maximum of h^{l-1}_u over In(v) (zeros if v has no
// in-neighbour).  A local delta cannot update it; instead a message carries the sender's old and
// new row, <old, new>, and the sink takes one of three actions per element:
//   raise       new > cached maximum: the cache moves up to it (an atomic maximum);
//   invalidate  old == cached maximum and new < old (or the edge is gone): the maximum is no longer
//               known, the sink is queued and recomputes its row over all current in-neighbours;
//   nothing     otherwise.
// A sink whose cached row ends up unchanged is not affected: it is not recomputed and sends
// nothing on (with a self term it is also affected when its own previous-layer row changed).  Senders of the next hop are the affected rows whose embedding really changed.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>
#include <cfloat>

namespace rp {

constexpr int MAX_HUB_DEGREE = 256;    // longer in-lists are recomputed in chunks, one warp per chunk
constexpr int MAX_HUB_CHUNK = 256;     // in-list entries per chunk
constexpr int MAX_FULL_PASS_DEGREE = 4096;   // a full pass has rows enough to keep every warp busy: only longer lists are chunked
constexpr int MAX_CHUNK = 64;          // edges per warp work item of the message walk

// The same code serves min: every comparison goes through these helpers (is_min = 0: maximum).
// worst() is the value every real one improves on.
__device__ __forceinline__ float worst(int is_min) { return __int_as_float(is_min ? 0x7f800000 : 0xff800000); }
__device__ __forceinline__ float pick(float a, float b, int is_min) { return is_min ? fminf(a, b) : fmaxf(a, b); }
__device__ __forceinline__ bool beats(float a, float b, int is_min) { return is_min ? a < b : a > b; }

// atomic maximum / minimum of an IEEE float: non-negative values order like signed integers,
// negative ones like unsigned integers in reverse
__device__ __forceinline__ void atomic_pick_f32(float* addr, float val, int is_min) {
    if (!is_min) {
        if (val >= 0.f) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(val));
        else atomicMin(reinterpret_cast<unsigned int*>(addr), __float_as_uint(val));
    } else {
        if (val >= 0.f) atomicMin(reinterpret_cast<int*>(addr), __float_as_int(val));
        else atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(val));
    }
}

__device__ __forceinline__ void mark_bit(uint32_t* bitmap, int v) {
    const uint32_t m = 1u << (v & 31);
    if (!(bitmap[v >> 5] & m)) atomicOr(&bitmap[v >> 5], m);
}

__device__ __forceinline__ float4 pick4(const float4& a, const float4& b, int is_min) {
    return make_float4(pick(a.x, b.x, is_min), pick(a.y, b.y, is_min), pick(a.z, b.z, is_min), pick(a.w, b.w, is_min));
}

// acc = max(acc, rows of the in-neighbours [j_begin, j_end) of v); LPR lanes hold one row (NV float4
// slots each), a warp works on 32 / LPR neighbours per step; on return every lane group holds the
// maximum over all groups
template <int NV, int LPR>
__device__ __forceinline__ void max_accumulate(float4 (&acc)[NV], const Side& in, int v, int j_begin, int j_end,
                                               const float* __restrict__ M, int ld, int is_min) {
    const int lane = lane_id(), nq = ld >> 2;
    constexpr int EPI = 32 / LPR;
    const int sub = lane / LPR, ql = lane % LPR;
    const int64_t base = in.start[v];
    for (int j0 = j_begin; j0 < j_end; j0 += 32) {
        const int mine = j0 + lane < j_end ? in.col[base + j0 + lane] : 0;
        const int cnt = min(32, j_end - j0);
        constexpr int UNR = 4;   // neighbour rows in flight per lane group
        for (int j = 0; j < cnt; j += UNR * EPI) {
            int u[UNR];
            float4 x[UNR][NV];
#pragma unroll
            for (int t = 0; t < UNR; ++t) {
                const int jj = j + t * EPI + sub;
                u[t] = __shfl_sync(FULL, mine, jj & 31);
                if (jj >= cnt) u[t] = -1;
            }
#pragma unroll
            for (int t = 0; t < UNR; ++t) {
                const float4* row = reinterpret_cast<const float4*>(M + (size_t)max(u[t], 0) * ld);
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    const int q = ql + LPR * k;
                    if (u[t] >= 0 && q < nq) x[t][k] = __ldg(row + q);
                }
            }
#pragma unroll
            for (int t = 0; t < UNR; ++t)
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    const int q = ql + LPR * k;
                    if (u[t] >= 0 && q < nq) acc[k] = pick4(acc[k], x[t][k], is_min);
                }
        }
    }
#pragma unroll
    for (int k = 0; k < NV; ++k) {
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
            acc[k].x = pick(acc[k].x, __shfl_xor_sync(FULL, acc[k].x, o), is_min);
            acc[k].y = pick(acc[k].y, __shfl_xor_sync(FULL, acc[k].y, o), is_min);
            acc[k].z = pick(acc[k].z, __shfl_xor_sync(FULL, acc[k].z, o), is_min);
            acc[k].w = pick(acc[k].w, __shfl_xor_sync(FULL, acc[k].w, o), is_min);
        }
    }
}

template <int NV>
__device__ __forceinline__ void fill(float4 (&acc)[NV], float x) {
#pragma unroll
    for (int k = 0; k < NV; ++k) acc[k] = make_float4(x, x, x, x);
}

// ---------------------------------------------------------------------------------------------
// Invalidated elements.  A sink with thousands of in-neighbours is rarely invalidated in more than
// a few of its elements (a changed neighbour is the maximiser of about d / deg_in of them), and
// gathering whole rows for it would move hundreds of bytes per neighbour where a few suffice.  The
// messages therefore record WHICH elements lost their maximiser (a bit mask per row); a row with
// at most MAX_EL such elements re-reads only those, any other row is gathered in full.
// ---------------------------------------------------------------------------------------------
constexpr int MAX_EL = 16;

// set elements of a row's mask -> ascending indices; returns their number, or -1 if there are more
// than MAX_EL (or the whole row was flagged).  Same result in every thread.
__device__ __forceinline__ int mask_elements(const uint32_t* __restrict__ mask, int mw, int ld, int (&el)[MAX_EL]) {
    int cnt = 0;
    for (int w = 0; w < mw; ++w) {
        uint32_t bits = mask[w];
        while (bits) {
            const int e = (w << 5) + __ffs(bits) - 1;
            bits &= bits - 1;
            if (e >= ld || cnt == MAX_EL) return -1;
            el[cnt++] = e;
        }
    }
    return cnt;
}

// ---------------------------------------------------------------------------------------------
// the maximum of one row over its whole in-list: a warp, or for long lists a block
// ---------------------------------------------------------------------------------------------
// mode 0 (bootstrap): rows = all vertices, the result is stored.
// mode 1 (recomputation): rows = list; the result is compared with the cached row, stored if it
//         differs, and the vertex is marked affected.
template <int NV, int LPR>
__global__ void __launch_bounds__(256)
k_max_rows(Ctl* ctl, int l, int mode, const int32_t* __restrict__ list, const int* n_dev, int n_host, Side in,
           const float* __restrict__ M, int ld, float* __restrict__ S, uint32_t* bitmapA, int32_t* long_rows,
           int* n_long, uint32_t* invmask, int mw, int is_min) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = n_dev ? *n_dev : n_host;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    const int sub = lane / LPR, ql = lane % LPR;
    for (int i = warp; i < n; i += nwarps) {
        const int v = list ? list[i] : i;
        const int deg = in.deg[v];
        if (deg > (mode ? MAX_HUB_DEGREE : MAX_FULL_PASS_DEGREE)) {
            if (lane == 0) long_rows[atomicAdd(n_long, 1)] = v;
            continue;
        }
        if (mode) {   // few invalidated elements: re-read only those
            uint32_t* mask = invmask + (size_t)v * mw;
            int el[MAX_EL];
            const int cnt = mask_elements(mask, mw, ld, el);
            __syncwarp();
            for (int w = lane; w < mw; w += 32) mask[w] = 0u;
            if (cnt >= 0 && deg > 0) {
                float acc[MAX_EL];
#pragma unroll
                for (int t = 0; t < MAX_EL; ++t) acc[t] = worst(is_min);
                const int64_t base = in.start[v];
                for (int j = lane; j < deg; j += 32) {
                    const float* row = M + (size_t)in.col[base + j] * ld;
#pragma unroll
                    for (int t = 0; t < MAX_EL; ++t)
                        if (t < cnt) acc[t] = pick(acc[t], __ldg(row + el[t]), is_min);
                }
                bool differs = false;
#pragma unroll
                for (int t = 0; t < MAX_EL; ++t) {
                    if (t < cnt) {
                        float m = acc[t];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) m = pick(m, __shfl_xor_sync(FULL, m, o), is_min);
                        if (lane == 0) {
                            float* dst = S + (size_t)v * ld + el[t];
                            if (*dst != m) { *dst = m; differs = true; }
                        }
                    }
                }
                if (lane == 0 && differs) mark_bit(bitmapA, v);
                continue;
            }
        }
        float4 acc[NV];
        fill<NV>(acc, deg > 0 ? worst(is_min) : 0.f);
        max_accumulate<NV, LPR>(acc, in, v, 0, deg, M, ld, is_min);
        float4* dst = reinterpret_cast<float4*>(S + (size_t)v * ld);
        bool differs = false;
        if (sub == 0) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int q = ql + LPR * k;
                if (q < nq) {
                    if (mode) {
                        const float4 o = dst[q];
                        differs |= o.x != acc[k].x || o.y != acc[k].y || o.z != acc[k].z || o.w != acc[k].w;
                    }
                    dst[q] = acc[k];
                }
            }
        }
        if (mode && __any_sync(FULL, differs) && lane == 0) mark_bit(bitmapA, v);
    }
    (void)l;
}

// Long rows, in three steps so that a hub's in-list is spread over the whole device instead of one block
// (a row of 150 000 in-neighbours took a block 4 to 14 ms: the 99th percentile of a batch):
//   begin   one warp per long row: the row as it is goes to a scratch copy, the elements to be recomputed
//           (those flagged in the row's mask if they are few, else all) are reset to the worst value, and
//           the in-list is queued in chunks;
//   chunks  one warp per (row, chunk): the maximum over the chunk, for those elements, raises the row by
//           atomic maxima;
//   end     one warp per long row: compares the row with its scratch copy, marks the vertex affected if
//           anything differs, clears the mask.
__global__ void __launch_bounds__(256)
k_max_long_begin(Ctl* ctl, int mode, const int32_t* __restrict__ long_rows, const int* __restrict__ n_long, Side in,
                 int ld, float* __restrict__ S, float* __restrict__ saved, const uint32_t* __restrict__ invmask, int mw,
                 int is_min, int2* items, int* n_items) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = *n_long;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int i = warp; i < n; i += nwarps) {
        const int v = long_rows[i];
        float* srow = S + (size_t)v * ld;
        int el[MAX_EL];
        const int cnt = mode ? mask_elements(invmask + (size_t)v * mw, mw, ld, el) : -1;
        for (int k = lane; k < ld; k += 32) {
            if (mode) saved[(size_t)i * ld + k] = srow[k];
            if (cnt < 0) srow[k] = worst(is_min);
        }
        __syncwarp();   // every element is saved before any is reset
        if (cnt >= 0 && lane < cnt) srow[el[lane]] = worst(is_min);
        const int nch = (in.deg[v] + MAX_HUB_CHUNK - 1) / MAX_HUB_CHUNK;
        int first = 0;
        if (lane == 0) first = atomicAdd(n_items, nch);
        first = __shfl_sync(FULL, first, 0);
        for (int ch = lane; ch < nch; ch += 32) items[first + ch] = make_int2(i, ch);
    }
}

template <int NV>
__global__ void __launch_bounds__(256)
k_max_long_chunks(Ctl* ctl, int mode, const int32_t* __restrict__ long_rows, const int2* __restrict__ items,
                  const int* __restrict__ n_items, Side in, const float* __restrict__ M, int ld, float* S,
                  const uint32_t* __restrict__ invmask, int mw, int is_min) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = *n_items;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int it = warp; it < n; it += nwarps) {
        const int v = long_rows[items[it].x], ch = items[it].y;
        const int deg = in.deg[v];
        const int j0 = ch * MAX_HUB_CHUNK, j1 = min(deg, j0 + MAX_HUB_CHUNK);
        float* srow = S + (size_t)v * ld;
        int el[MAX_EL];
        const int cnt = mode ? mask_elements(invmask + (size_t)v * mw, mw, ld, el) : -1;
        if (cnt >= 0) {   // few elements: every lane strides over the chunk for those alone
            float acc[MAX_EL];
#pragma unroll
            for (int t = 0; t < MAX_EL; ++t) acc[t] = worst(is_min);
            const int64_t base = in.start[v];
            for (int j = j0 + lane; j < j1; j += 32) {
                const float* row = M + (size_t)in.col[base + j] * ld;
#pragma unroll
                for (int t = 0; t < MAX_EL; ++t)
                    if (t < cnt) acc[t] = pick(acc[t], __ldg(row + el[t]), is_min);
            }
#pragma unroll
            for (int t = 0; t < MAX_EL; ++t) {
                if (t < cnt) {
                    float m = acc[t];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) m = pick(m, __shfl_xor_sync(FULL, m, o), is_min);
                    if (lane == 0) atomic_pick_f32(srow + el[t], m, is_min);
                }
            }
            continue;
        }
        float4 acc[NV];
        fill<NV>(acc, worst(is_min));
        max_accumulate<NV, 32>(acc, in, v, j0, j1, M, ld, is_min);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int q = lane + 32 * k;
            if (q < nq) {
                atomic_pick_f32(srow + 4 * q + 0, acc[k].x, is_min);
                atomic_pick_f32(srow + 4 * q + 1, acc[k].y, is_min);
                atomic_pick_f32(srow + 4 * q + 2, acc[k].z, is_min);
                atomic_pick_f32(srow + 4 * q + 3, acc[k].w, is_min);
            }
        }
    }
}

__global__ void __launch_bounds__(256)
k_max_long_end(Ctl* ctl, const int32_t* __restrict__ long_rows, const int* __restrict__ n_long, int ld,
               const float* __restrict__ S, const float* __restrict__ saved, uint32_t* bitmapA, uint32_t* invmask,
               int mw) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = *n_long;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int i = warp; i < n; i += nwarps) {
        const int v = long_rows[i];
        bool differs = false;
        for (int k = lane; k < ld; k += 32) differs |= S[(size_t)v * ld + k] != saved[(size_t)i * ld + k];
        for (int w = lane; w < mw; w += 32) invmask[(size_t)v * mw + w] = 0u;
        if (__any_sync(FULL, differs) && lane == 0) mark_bit(bitmapA, v);
    }
}

// ---------------------------------------------------------------------------------------------
// messages <old, new> along the out-edges of the senders
// ---------------------------------------------------------------------------------------------
// in-degree of v before the batch: a sink that had no in-neighbour caches zeros, not a maximum
__device__ __forceinline__ int deg_in_before(const Side& in, int v) {
    return in.deg[v] - in.cnt_add[v] + in.cnt_del[v];
}

template <int NV, int LPR>
__global__ void __launch_bounds__(256)
k_max_messages(Ctl* ctl, int l, const int32_t* __restrict__ senders, const int32_t* __restrict__ old_idx,
               const int64_t* __restrict__ coff, Side out, Side in, const float* __restrict__ Hprev,
               const float* __restrict__ Old, int ld, float* S, uint32_t* bitmapA, uint32_t* bitmapR,
               uint32_t* invmask, int mw, int is_min) {
    pdl_enter();
    if (ctl->abort) return;
    const int nC = ctl->nC[l - 1];
    if (nC == 0) return;
    const int64_t E = coff[nC];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    constexpr int EPI = 32 / LPR;
    const int sub = lane / LPR, ql = lane % LPR;
    const unsigned group = LPR == 32 ? FULL : (((1u << LPR) - 1u) << (sub * LPR));
    for (int64_t e0 = (int64_t)warp * MAX_CHUNK; e0 < E; e0 += (int64_t)nwarps * MAX_CHUNK) {
        const int64_t e1 = min(e0 + MAX_CHUNK, E);
        int i = upper_row(coff, nC, e0);
        int64_t e = e0;
        while (e < e1) {
            const int64_t row_end = coff[i + 1];
            if (row_end <= e) { ++i; continue; }
            const int64_t seg_end = min(e1, row_end);
            const int u = senders[i];
            const int64_t base = out.start[u] + (e - coff[i]);
            const int cnt = (int)(seg_end - e);
            float4 hn[NV], ho[NV];
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int q = ql + LPR * k;
                hn[k] = q < nq ? __ldg(reinterpret_cast<const float4*>(Hprev + (size_t)u * ld) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                ho[k] = q < nq ? __ldg(reinterpret_cast<const float4*>(Old + (size_t)old_idx[i] * ld) + q) : hn[k];
            }
            // the sink of the next edge, its in-degree before the batch and its cached row are fetched
            // while the current edge is classified (every edge is a dependent chain of loads otherwise)
            int v_nx = 0, db_nx = 1;
            bool live_nx = false;
            float4 s_nx[NV];
            auto fetch = [&](int j) {
                const int jj = j + sub;
                live_nx = jj < cnt;
                v_nx = live_nx ? out.col[base + jj] : 0;
                db_nx = live_nx ? deg_in_before(in, v_nx) : 1;
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    const int q = ql + LPR * k;
                    s_nx[k] = (live_nx && db_nx != 0 && q < nq)
                                  ? *reinterpret_cast<const float4*>(S + (size_t)v_nx * ld + 4 * q)
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            };
            fetch(0);
            for (int j = 0; j < cnt; j += EPI) {
                const int v = v_nx, db = db_nx;
                const bool live = live_nx;
                float4 s_cur[NV];
#pragma unroll
                for (int k = 0; k < NV; ++k) s_cur[k] = s_nx[k];
                if (j + EPI < cnt) fetch(j + EPI);
                bool raise = false, invalid = false;
                if (live) {
                    uint32_t* mask = invmask + (size_t)v * mw;
                    if (db == 0) {   // zeros cached: gather the real maximum, every element
                        invalid = true;
                        for (int w = ql; w < mw; w += LPR) atomicOr(&mask[w], 0xffffffffu);
                    } else {
                        float* srow = S + (size_t)v * ld;
#pragma unroll
                        for (int k = 0; k < NV; ++k) {
                            const int q = ql + LPR * k;
                            if (q < nq) {
                                const float4 s = s_cur[k];
                                const float nn[4] = {hn[k].x, hn[k].y, hn[k].z, hn[k].w};
                                const float oo[4] = {ho[k].x, ho[k].y, ho[k].z, ho[k].w};
                                const float ss[4] = {s.x, s.y, s.z, s.w};
#pragma unroll
                                for (int t = 0; t < 4; ++t) {
                                    if (beats(nn[t], ss[t], is_min)) { atomic_pick_f32(srow + 4 * q + t, nn[t], is_min); raise = true; }
                                    else if (oo[t] == ss[t] && beats(oo[t], nn[t], is_min)) {
                                        invalid = true;
                                        const int e_ = 4 * q + t;
                                        atomicOr(&mask[e_ >> 5], 1u << (e_ & 31));
                                    }
                                }
                            }
                        }
                    }
                }
                raise = __any_sync(group, raise);
                invalid = __any_sync(group, invalid);
                if (live && ql == 0) {
                    if (raise) mark_bit(bitmapA, v);
                    if (invalid) mark_bit(bitmapR, v);
                }
            }
            e = seg_end;
            ++i;
        }
    }
}

// edge records: <-, new> along an added edge, <old, -> along a deleted one; one warp per record
__global__ void k_max_records(Ctl* ctl, const Rec* __restrict__ rec, Side in, const int32_t* __restrict__ posmap,
                              const int32_t* __restrict__ old_idx, const float* __restrict__ Hprev,
                              const float* __restrict__ Old, int ld, float* S, uint32_t* bitmapA, uint32_t* bitmapR,
                              uint32_t* invmask, int mw, int is_min) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->n_rec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int r = warp; r < n; r += nwarps) {
        const int u = rec[r].u, v = rec[r].v;
        float* srow = S + (size_t)v * ld;
        uint32_t* mask = invmask + (size_t)v * mw;
        bool raise = false, invalid = false, whole = false;
        if (rec[r].sign > 0) {
            if (deg_in_before(in, v) == 0) whole = true;
            else
                for (int k = lane; k < ld; k += 32) {
                    const float x = Hprev[(size_t)u * ld + k];
                    if (beats(x, srow[k], is_min)) { atomic_pick_f32(srow + k, x, is_min); raise = true; }
                }
        } else {
            if (in.deg[v] == 0) whole = true;
            else {
                const int p = posmap[u];
                const float* orow = p >= 0 ? Old + (size_t)old_idx[p] * ld : Hprev + (size_t)u * ld;
                for (int k = lane; k < ld; k += 32)
                    if (orow[k] == srow[k]) { invalid = true; atomicOr(&mask[k >> 5], 1u << (k & 31)); }
            }
        }
        if (whole) {   // every element
            invalid = true;
            for (int w = lane; w < mw; w += 32) atomicOr(&mask[w], 0xffffffffu);
        }
        raise = __any_sync(FULL, raise);
        invalid = __any_sync(FULL, invalid);
        if (lane == 0) {
            if (raise) mark_bit(bitmapA, v);
            if (invalid) mark_bit(bitmapR, v);
        }
    }
}

// self term: a vertex whose own previous-layer row changed recomputes its embedding as well
__global__ void k_max_mark_self(Ctl* ctl, int l, const int32_t* __restrict__ senders, uint32_t* bitmapA) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->nC[l - 1];
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) mark_bit(bitmapA, senders[i]);
}

// senders of the next hop: affected rows whose embedding really changed (old rows are kept compact,
// in the order of A_l); one warp per affected row
__global__ void k_max_senders(Ctl* ctl, int l, const int32_t* __restrict__ A, const float* __restrict__ H,
                              const float* __restrict__ Old, int ld, int32_t* senders, int32_t* old_idx,
                              int32_t* posmap) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->nA[l];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int i = warp; i < n; i += nwarps) {
        const int v = A[i];
        bool differs = false;
        for (int k = lane; k < ld; k += 32) differs |= H[(size_t)v * ld + k] != Old[(size_t)i * ld + k];
        if (__any_sync(FULL, differs) && lane == 0) {
            const int idx = atomicAdd(&ctl->nC[l], 1);
            senders[idx] = v;
            old_idx[idx] = i;
            posmap[v] = idx;
        }
    }
}

static void launch_long_rows(Ctx* c, int l, int mode, const float* M, int ld, float* S, int32_t* long_rows, int* n_long) {
    const int nv = div_up(ld, 128), is_min = (int)(c->agg == RIPPLE_AGG_MIN);
    int2* items = reinterpret_cast<int2*>(c->coff);   // the senders' degree prefix is not needed at this point
    int* n_items = &c->ctl->max_items[l];
    float* saved = c->Dt;                              // compact scratch rows (no layer transforms before a max)
    RP_LAUNCH(c, k_max_long_begin, c->n_sm * 2, 256, 0, c->ctl, mode, long_rows, n_long, c->side[1], ld, S, saved,
              c->invmask, c->mw, is_min, items, n_items);
#define CHUNKS(NV) RP_LAUNCH(c, k_max_long_chunks<NV>, c->n_sm * 8, 256, 0, c->ctl, mode, long_rows, items, n_items, c->side[1], M, ld, S, c->invmask, c->mw, is_min)
    if (nv <= 1) CHUNKS(1); else if (nv <= 2) CHUNKS(2); else if (nv <= 4) CHUNKS(4); else CHUNKS(8);
#undef CHUNKS
    if (mode)
        RP_LAUNCH(c, k_max_long_end, c->n_sm * 2, 256, 0, c->ctl, long_rows, n_long, ld, S, saved, c->bitmap,
                  c->invmask, c->mw);
}

// bootstrap: S^l_v for every vertex
void max_full(Ctx* c, int l) {
    const int ld = c->ws[l];
    int32_t* long_rows = c->Clist[0];
    int* n_long = &c->ctl->work_counter[(l - 1) & 7];
#define ROWS(NV, LPR) RP_LAUNCH(c, (k_max_rows<NV, LPR>), c->n_sm * 16, 256, 0, c->ctl, l, 0, (const int32_t*)nullptr, (const int*)nullptr, c->N, c->side[1], c->H[l - 1], ld, c->S[l], c->bitmap, long_rows, n_long, c->invmask, c->mw, (int)(c->agg == RIPPLE_AGG_MIN))
    RP_WIDTH_DISPATCH(ld, ROWS);
#undef ROWS
    launch_long_rows(c, l, 0, c->H[l - 1], ld, c->S[l], long_rows, n_long);
}

// hop l of a batch: messages, recomputation of the invalidated sinks, the list A_l
void max_hop(Ctx* c, int l, int n) {
    const int ld = c->ws[l];
    const float* Old = c->D[(l - 1) & 1];            // previous values of the rows of A_{l-1}, in its order
    const int32_t* senders = c->Clist[(l - 1) & 1];
    const int T = 256;
#define MSG(NV, LPR) RP_LAUNCH(c, (k_max_messages<NV, LPR>), c->n_sm * 8, T, 0, c->ctl, l, senders, c->old_idx, c->coff, c->side[0], c->side[1], c->H[l - 1], Old, ld, c->S[l], c->bitmap, c->bitmap2, c->invmask, c->mw, (int)(c->agg == RIPPLE_AGG_MIN))
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l], c->stream);
    RP_WIDTH_DISPATCH(ld, MSG);
#undef MSG
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l + 1], c->stream);
    if (n > 0)
        RP_LAUNCH(c, k_max_records, std::min(div_up(n, T / 32), c->n_sm * 8), T, 0, c->ctl, c->rec, c->side[1], c->posmap,
                  c->old_idx, c->H[l - 1], Old, ld, c->S[l], c->bitmap, c->bitmap2, c->invmask, c->mw, (int)(c->agg == RIPPLE_AGG_MIN));
    // invalidated sinks -> list (the buffer of A_l serves until A_l itself is compacted), then their rows
    int32_t* rlist = c->A[l];
    int* n_r = &c->ctl->n_long[l];
    bitmap_to_list_from(c, c->bitmap2, rlist, n_r, nullptr);
    int32_t* long_rows = c->Clist[l & 1];            // the next hop's sender list is not built yet
    int* n_long = &c->ctl->work_counter[(l - 1) & 7];
#define ROWS(NV, LPR) RP_LAUNCH(c, (k_max_rows<NV, LPR>), c->n_sm * 8, T, 0, c->ctl, l, 1, rlist, n_r, 0, c->side[1], c->H[l - 1], ld, c->S[l], c->bitmap, long_rows, n_long, c->invmask, c->mw, (int)(c->agg == RIPPLE_AGG_MIN))
    RP_WIDTH_DISPATCH(ld, ROWS);
#undef ROWS
    launch_long_rows(c, l, 1, c->H[l - 1], ld, c->S[l], long_rows, n_long);
    if (c->self_term) RP_LAUNCH(c, k_max_mark_self, c->n_sm * 2, T, 0, c->ctl, l, senders, c->bitmap);
}

// senders of hop l + 1 (l = 0: the vertices whose feature row really changed)
void max_senders_build(Ctx* c, int l) {
    int32_t* senders = c->Clist[l & 1];
    RP_LAUNCH(c, k_max_senders, c->n_sm * 8, 256, 0, c->ctl, l, c->A[l], c->H[l], c->D[l & 1], c->ld[l], senders,
              c->old_idx, c->posmap);
    scan_degrees(c, senders, &c->ctl->nC[l], 0, c->side[0].deg, c->coff, &c->ctl->E[l + 1]);
}

void max_prepare() {}

}  // namespace rp
