// Attention layers (Sec. 3.4.1, Eq. 3) and their hybrid-incremental hop.
//
//   h^l_v = sum_{u in In(v)} alpha_uv h^{l-1}_u,   alpha_uv = exp(z_uv) / sum_u exp(z_uv),
//   z_uv  = rect(a_src . W h_u + a_dst . W h_v),   rect(z) = z for z >= 0, slope * z below
//
// (slope = 1: the linear logit that Eq. 3 prints; slope < 1: the leaky rectifier of the architecture
// it cites).  The two halves of the logit are per-vertex scalars, s_u = (W a_src) . h_u and
// t_v = (W a_dst) . h_v, cached for every vertex and refreshed where h^{l-1} changed.
//
// Cached per vertex: the row [ sum_u e_uv h_u  |  sum_u e_uv ] with e_uv = exp(z_uv): numerator in the
// first d columns, denominator in column d.  A hop updates it in one of two ways:
//   recompute    a vertex whose own h^{l-1} changed (it was in the tree one hop earlier): its t_v moved,
//                so every e_uv it is the sink of moved; the row is gathered anew over its in-list;
//   incremental  any other hop-l vertex takes <numerator, denominator> messages: e_new h_new - e_old h_old
//                from a changed in-neighbour, the whole new term along an added edge, minus the whole
//                old term along a deleted one.
// e_old is recomputed from the cached (s_old, t_v) by the very expression that produced it when the
// term was added, so the weight that leaves the sum is bit for bit the one that entered it.  Messages of a batch meet in
// the accumulator dS first and reach the cached row as one addition; every row keeps the rounding
// budget of the linear aggregators (see k_fold_deltas) and is gathered anew when it runs out.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>

namespace rp {

constexpr int ATT_CHUNK = 64;     // out-edges per warp work item of the message walk
constexpr int ATT_GATHER = RP_ATT_CHUNK;   // in-list entries per warp work item of a recomputation

__device__ __forceinline__ float att_weight(float s_u, float t_v, float slope) {
    float z = s_u + t_v;
    z = z < 0.f ? slope * z : z;
    return expf(z);
}

// s_v = q_src . h_v, t_v = q_dst . h_v for the listed rows (all rows if list is null); one warp per row.
// s_old (if given) receives the value s_v had before, in list order: the old logit half of a sender.
__global__ void __launch_bounds__(256)
k_att_scalars(Ctl* ctl, const int32_t* __restrict__ list, const int* n_dev, int n_host, const float* __restrict__ H,
              int ld_h, const float* __restrict__ q, float* att_s, float* att_t, float* s_old) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = n_dev ? *n_dev : n_host;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld_h >> 2;
    const float4* qs = reinterpret_cast<const float4*>(q);
    const float4* qt = reinterpret_cast<const float4*>(q + ld_h);
    for (int i = warp; i < n; i += nwarps) {
        const int v = list ? list[i] : i;
        const float4* row = reinterpret_cast<const float4*>(H + (size_t)v * ld_h);
        float s = 0.f, t = 0.f;
        for (int k = lane; k < nq; k += 32) {
            const float4 h = row[k], a = __ldg(qs + k), b = __ldg(qt + k);
            s += h.x * a.x + h.y * a.y + h.z * a.z + h.w * a.w;
            t += h.x * b.x + h.y * b.y + h.z * b.z + h.w * b.w;
        }
        s = warp_sum(s);
        t = warp_sum(t);
        if (lane == 0) {
            if (s_old) s_old[i] = att_s[v];
            att_s[v] = s;
            att_t[v] = t;
        }
    }
}

// Messages along the current out-edges of the senders (the rows of A_{l-1}): e_new h_new - e_old h_old
// into the accumulator row of every sink that is not itself a sender (those recompute).  An edge added
// by this batch is walked like any other; its record then adds e_old h_old, which leaves the new term.
template <int NV, int LPR>
__global__ void __launch_bounds__(256)
k_att_push(Ctl* ctl, int l, const int32_t* __restrict__ senders, const int64_t* __restrict__ coff, Side out,
           const int32_t* __restrict__ posmap, const float* __restrict__ Hprev, const float* __restrict__ Old, int ld_h,
           const float* __restrict__ s_old, const float* __restrict__ att_s, const float* __restrict__ att_t,
           float slope, int d, int ld, float* dS, uint32_t* bitmap) {
    pdl_enter();
    if (ctl->abort) return;
    const int nC = ctl->nC[l - 1];
    if (nC == 0) return;
    const int64_t E = coff[nC];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2, nqh = ld_h >> 2;
    constexpr int EPI = 32 / LPR;
    const int sub = lane / LPR, ql = lane % LPR;
    const int qden = d >> 2, cden = d & 3;   // the denominator's place in the row
    for (int64_t e0 = (int64_t)warp * ATT_CHUNK; e0 < E; e0 += (int64_t)nwarps * ATT_CHUNK) {
        const int64_t e1 = min(e0 + ATT_CHUNK, E);
        int i = upper_row(coff, nC, e0);
        int64_t e = e0;
        while (e < e1) {
            const int64_t row_end = coff[i + 1];
            if (row_end <= e) { ++i; continue; }
            const int64_t seg_end = min(e1, row_end);
            const int u = senders[i];
            const int64_t base = out.start[u] + (e - coff[i]);
            float4 hn[NV], ho[NV];
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int q = ql + LPR * k;
                hn[k] = q < nqh ? __ldg(reinterpret_cast<const float4*>(Hprev + (size_t)u * ld_h) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                ho[k] = q < nqh ? __ldg(reinterpret_cast<const float4*>(Old + (size_t)i * ld_h) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const float sn = att_s[u], so = s_old[i];
            const int cnt_total = (int)(seg_end - e);
            for (int j0 = 0; j0 < cnt_total; j0 += 32) {
                const bool have = j0 + lane < cnt_total;
                const int mine = have ? out.col[base + j0 + lane] : 0;
                const float mine_t = have ? att_t[mine] : 0.f;
                const int mine_skip = have ? (posmap[mine] >= 0) : 1;
                const int cnt = min(32, cnt_total - j0);
                if (have) {   // every sink joins the hop's frontier: the same walk as the frontier's own
                    const uint32_t m = 1u << (mine & 31);
                    if (!(bitmap[mine >> 5] & m)) atomicOr(&bitmap[mine >> 5], m);
                }
                for (int j = 0; j < cnt; j += EPI) {
                    const int jj = j + sub;
                    const int v = __shfl_sync(FULL, mine, jj & 31);
                    const float t = __shfl_sync(FULL, mine_t, jj & 31);
                    const int skip = __shfl_sync(FULL, mine_skip, jj & 31);
                    if (jj < cnt && !skip) {
                        const float en = att_weight(sn, t, slope), eo = att_weight(so, t, slope);
                        float* dst = dS + (size_t)v * ld;
#pragma unroll
                        for (int k = 0; k < NV; ++k) {
                            const int q = ql + LPR * k;
                            if (q < nq) {
                                float m[4] = {en * hn[k].x - eo * ho[k].x, en * hn[k].y - eo * ho[k].y,
                                              en * hn[k].z - eo * ho[k].z, en * hn[k].w - eo * ho[k].w};
                                if (q == qden) m[cden] = en - eo;
                                red_add_v4(dst + 4 * q, make_float4(m[0], m[1], m[2], m[3]));
                            }
                        }
                    }
                }
            }
            e = seg_end;
            ++i;
        }
    }
}

// Edge records.  Added edge (u, v): plus the term of u as it was before this hop's changes (the walk
// above has already brought the difference to the new one if u is a sender).  Deleted edge: minus that
// term.  A sink that recomputes takes neither.  One warp per record.
__global__ void k_att_records(Ctl* ctl, const Rec* __restrict__ rec, const int32_t* __restrict__ posmap,
                              const float* __restrict__ Hprev, const float* __restrict__ Old, int ld_h,
                              const float* __restrict__ s_old, const float* __restrict__ att_s,
                              const float* __restrict__ att_t, float slope, int d, int ld, float* dS) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->n_rec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int r = warp; r < n; r += nwarps) {
        const int u = rec[r].u, v = rec[r].v;
        if (posmap[v] >= 0) continue;
        const int p = posmap[u];
        const float* row = p >= 0 ? Old + (size_t)p * ld_h : Hprev + (size_t)u * ld_h;
        const float s = p >= 0 ? s_old[p] : att_s[u];
        const float e = (rec[r].sign > 0 ? 1.f : -1.f) * att_weight(s, att_t[v], slope);
        float* dst = dS + (size_t)v * ld;
        for (int k = lane; k <= d; k += 32) atomicAdd(dst + k, k < d ? e * row[k] : e);
    }
}

// Per hop-l vertex (or per vertex, `all`): either fold the accumulated messages into the cached row,
// keeping the row's rounding budget, and write the new embedding row at once; or -- the vertex is a
// sender (its own h^{l-1} changed), the budget has run out, no in-neighbour is left, or `all` -- zero
// the row, queue its in-list, in chunks, for k_att_gather and flag the vertex for k_att_update.
__global__ void __launch_bounds__(256)
k_att_fold(Ctl* ctl, int l, const int32_t* __restrict__ A, const int* n_dev, int n_host, int all, int ld, float* S,
           float* dS, float* budget, float tau2, const int32_t* __restrict__ deg_in,
           const int32_t* __restrict__ posmap, int2* items, int d, int act, float* H, int ld_h, float* Old,
           uint32_t* gathered) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = n_dev ? *n_dev : n_host;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int i = warp; i < n; i += nwarps) {
        const int v = A ? A[i] : i;
        const size_t off = (size_t)v * ld;
        float4* s = reinterpret_cast<float4*>(S + off);
        float4* dd = reinterpret_cast<float4*>(dS + off);
        const bool fast = !all && nq <= 32 && (ld_h & 3) == 0;
        // (the fast form asks for the row together with the two words that decide whether it is used)
        float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), y0 = x0, hold0 = x0;
        float spent0 = 0.f;
        if (fast) {
            if (lane < nq) { x0 = s[lane]; y0 = dd[lane]; }
            if (lane < (ld_h >> 2)) hold0 = reinterpret_cast<const float4*>(H + (size_t)v * ld_h)[lane];
            if (budget) spent0 = budget[v];
        }
        bool anew = all || posmap[v] >= 0 || deg_in[v] == 0;   // (no in-neighbour left: exact zeros)
        bool on_budget = false;
        if (!anew && fast) {
            // Rows of up to 128 floats: one 16-byte piece per lane, so the row, its accumulator, its budget and the
            // old embedding are requested together and the new embedding is made from registers.  (A warp works
            // through its rows one after the other: the loop form below pays five dependent trips to memory per
            // row, this one two.)
            const int nqh = ld_h >> 2;
            float4 x = x0;
            const float4 y = y0, hold = hold0;
            float4* hrow4 = reinterpret_cast<float4*>(H + (size_t)v * ld_h);
            const float spent_before = spent0;
            float m_old = fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w)));
            x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
            float m_new = fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w)));
            if (lane < nq) { s[lane] = x; dd[lane] = make_float4(0.f, 0.f, 0.f, 0.f); }
            bool keep = true;
            if (budget) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    m_old = fmaxf(m_old, __shfl_xor_sync(FULL, m_old, o));
                    m_new = fmaxf(m_new, __shfl_xor_sync(FULL, m_new, o));
                }
                const float m = fmaxf(m_old, m_new);
                const float spent = spent_before + m * m;
                const float limit = tau2 * (0.5f + (float)(mix64((uint64_t)v) & 255u) * (1.0f / 512.0f)) * m_new * m_new;
                keep = !(spent > limit);
                if (keep && lane == 0) budget[v] = spent;
            }
            if (keep) {
                const int c = d & 3;
                const float mine = c == 0 ? x.x : c == 1 ? x.y : c == 2 ? x.z : x.w;
                const float den = __shfl_sync(FULL, mine, d >> 2);
                if (lane < nqh) {
                    const float e[4] = {x.x, x.y, x.z, x.w};
                    float h[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        h[t] = (den > 0.f && 4 * lane + t < d) ? e[t] / den : 0.f;
                        if (act == RIPPLE_ACT_RELU) h[t] = fmaxf(h[t], 0.f);
                    }
                    if (Old) *reinterpret_cast<float4*>(Old + (size_t)i * ld_h + 4 * lane) = hold;
                    hrow4[lane] = make_float4(h[0], h[1], h[2], h[3]);
                }
                continue;
            }
            __syncwarp();
            anew = on_budget = true;
        }
        if (!anew) {
            float m_old = 0.f, m_new = 0.f;
            for (int q = lane; q < nq; q += 32) {
                float4 x = s[q], y = dd[q];
                m_old = fmaxf(m_old, fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))));
                x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
                m_new = fmaxf(m_new, fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w))));
                s[q] = x;
                dd[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            bool keep = true;
            if (budget) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    m_old = fmaxf(m_old, __shfl_xor_sync(FULL, m_old, o));
                    m_new = fmaxf(m_new, __shfl_xor_sync(FULL, m_new, o));
                }
                const float m = fmaxf(m_old, m_new);
                const float spent = budget[v] + m * m;
                const float limit = tau2 * (0.5f + (float)(mix64((uint64_t)v) & 255u) * (1.0f / 512.0f)) * m_new * m_new;
                keep = !(spent > limit);
                if (keep && lane == 0) budget[v] = spent;
            }
            __syncwarp();
            if (keep) {   // the row is final: its embedding follows at once
                const float den = S[off + d];
                float* hrow = H + (size_t)v * ld_h;
                for (int k = lane; k < ld_h; k += 32) {
                    float x = (den > 0.f && k < d) ? S[off + k] / den : 0.f;
                    if (act == RIPPLE_ACT_RELU) x = fmaxf(x, 0.f);
                    if (Old) Old[(size_t)i * ld_h + k] = hrow[k];
                    hrow[k] = x;
                }
                continue;
            }
            anew = on_budget = true;
        }
        for (int q = lane; q < nq; q += 32) {
            s[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!all) dd[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const int deg = deg_in[v];
        const int nch = (deg + ATT_GATHER - 1) / ATT_GATHER;
        int first = 0;
        if (lane == 0) {
            if (nch) first = atomicAdd(&ctl->rebuild_items[l], nch);
            if (budget) budget[v] = 0.f;
            if (on_budget) atomicAdd(&ctl->n_rebuilt[l], 1);
            if (gathered) atomicOr(&gathered[v >> 5], 1u << (v & 31));
        }
        first = __shfl_sync(FULL, first, 0);
        for (int ch = lane; ch < nch; ch += 32) items[first + ch] = make_int2(v, ch);
    }
}

// One warp per (vertex, chunk of its in-list): sum_u e_uv [h_u | 1] over the chunk, added to the zeroed row.
template <int NV, int LPR>
__global__ void __launch_bounds__(256)
k_att_gather(Ctl* ctl, int l, const int2* __restrict__ items, Side in, const float* __restrict__ Hprev, int ld_h,
             const float* __restrict__ att_s, const float* __restrict__ att_t, float slope, int d, int ld, float* S) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->rebuild_items[l];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2, nqh = ld_h >> 2;
    constexpr int EPI = 32 / LPR;
    const int sub = lane / LPR, ql = lane % LPR;
    const int qden = d >> 2, cden = d & 3;
    for (int it = warp; it < n; it += nwarps) {
        const int v = items[it].x, ch = items[it].y;
        const int deg = in.deg[v];
        const int j_begin = ch * ATT_GATHER, j_end = min(deg, j_begin + ATT_GATHER);
        const int64_t base = in.start[v];
        const float t = att_t[v];
        float4 acc[NV];
#pragma unroll
        for (int k = 0; k < NV; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j0 = j_begin; j0 < j_end; j0 += 32) {
            const bool have = j0 + lane < j_end;
            const int mine = have ? in.col[base + j0 + lane] : 0;
            const float mine_e = have ? att_weight(att_s[mine], t, slope) : 0.f;
            const int cnt = min(32, j_end - j0);
            constexpr int UNR = NV == 1 ? 8 : 4;   // neighbour rows in flight per lane group
            for (int j = 0; j < cnt; j += UNR * EPI) {
                int u[UNR];
                float e[UNR];
                float4 x[UNR][NV];
#pragma unroll
                for (int r = 0; r < UNR; ++r) {
                    const int jj = j + r * EPI + sub;
                    u[r] = __shfl_sync(FULL, mine, jj & 31);
                    e[r] = __shfl_sync(FULL, mine_e, jj & 31);
                    if (jj >= cnt) { u[r] = -1; e[r] = 0.f; }
                }
#pragma unroll
                for (int r = 0; r < UNR; ++r) {
                    const float4* row = reinterpret_cast<const float4*>(Hprev + (size_t)max(u[r], 0) * ld_h);
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        const int q = ql + LPR * k;
                        x[r][k] = (u[r] >= 0 && q < nqh) ? __ldg(row + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
#pragma unroll
                for (int r = 0; r < UNR; ++r)
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        const int q = ql + LPR * k;
                        float m[4] = {e[r] * x[r][k].x, e[r] * x[r][k].y, e[r] * x[r][k].z, e[r] * x[r][k].w};
                        if (q == qden) m[cden] = e[r];
                        acc[k].x += m[0]; acc[k].y += m[1]; acc[k].z += m[2]; acc[k].w += m[3];
                    }
            }
        }
#pragma unroll
        for (int k = 0; k < NV; ++k) {
#pragma unroll
            for (int o = LPR; o < 32; o <<= 1) {
                acc[k].x += __shfl_xor_sync(FULL, acc[k].x, o);
                acc[k].y += __shfl_xor_sync(FULL, acc[k].y, o);
                acc[k].z += __shfl_xor_sync(FULL, acc[k].z, o);
                acc[k].w += __shfl_xor_sync(FULL, acc[k].w, o);
            }
        }
        if (sub == 0) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int q = ql + LPR * k;
                if (q < nq) red_add_v4(S + (size_t)v * ld + 4 * q, acc[k]);
            }
        }
    }
}

// h^l_v = numerator / denominator (zeros without in-neighbours), activation; the row it replaces is
// kept, compact and in list order, for the next hop's messages.  One warp per row.  With `gathered`
// only the flagged rows are written (the others got theirs from k_att_fold) and the flags are cleared.
__global__ void __launch_bounds__(256)
k_att_update(Ctl* ctl, const int32_t* __restrict__ list, const int* n_dev, int n_host, const float* __restrict__ S,
             int ld, int d, const int32_t* __restrict__ deg_in, int act, float* H, int ld_h, float* Old,
             uint32_t* gathered) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = n_dev ? *n_dev : n_host;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id();
    for (int i = warp; i < n; i += nwarps) {
        const int v = list ? list[i] : i;
        if (gathered) {
            if (!(gathered[v >> 5] & (1u << (v & 31)))) continue;
            __syncwarp();
            if (lane == 0) atomicAnd(&gathered[v >> 5], ~(1u << (v & 31)));
        }
        const float* srow = S + (size_t)v * ld;
        const float den = srow[d];
        const bool live = deg_in[v] > 0 && den > 0.f;
        float* hrow = H + (size_t)v * ld_h;
        for (int k = lane; k < ld_h; k += 32) {
            float x = (live && k < d) ? srow[k] / den : 0.f;
            if (act == RIPPLE_ACT_RELU) x = fmaxf(x, 0.f);
            if (Old) Old[(size_t)i * ld_h + k] = hrow[k];
            hrow[k] = x;
        }
    }
}

// ---------------------------------------------------------------------------------------------
static void launch_gather(Ctx* c, int l) {
    const LayerDev& ly = c->layer[l];
    const int ld = c->ws[l];
#define GATHER(NV, LPR) RP_LAUNCH(c, (k_att_gather<NV, LPR>), c->n_sm * 8, 256, 0, c->ctl, l, c->att_items, c->side[1], c->H[l - 1], c->ld[l - 1], c->att_s[l], c->att_t[l], ly.eps, ly.d_in, ld, c->S[l])
    RP_WIDTH_DISPATCH(ld, GATHER);
#undef GATHER
}

void att_update(Ctx* c, int l, bool full) {
    const LayerDev& ly = c->layer[l];
    float* old_rows = (full || l == c->L) ? nullptr : c->D[l & 1];   // the last hop sends nothing
    RP_LAUNCH(c, k_att_update, c->n_sm * 8, 256, 0, c->ctl, full ? (const int32_t*)nullptr : c->A[l],
              full ? (const int*)nullptr : &c->ctl->nA[l], c->N, c->S[l], c->ws[l], ly.d_in, c->side[1].deg, ly.act,
              c->H[l], c->ld[l], old_rows, full ? (uint32_t*)nullptr : c->bitmap);
}

// bootstrap: logit halves, cached rows and outputs of every vertex
void att_full(Ctx* c, int l) {
    const LayerDev& ly = c->layer[l];
    RP_LAUNCH(c, k_att_scalars, c->n_sm * 8, 256, 0, c->ctl, (const int32_t*)nullptr, (const int*)nullptr, c->N,
              c->H[l - 1], c->ld[l - 1], ly.W1, c->att_s[l], c->att_t[l], (float*)nullptr);
    RP_LAUNCH(c, k_att_fold, c->n_sm * 8, 256, 0, c->ctl, l, (const int32_t*)nullptr, (const int*)nullptr, c->N, 1,
              c->ws[l], c->S[l], c->dS[l], c->Eb[l], c->rebuild_tau2, c->side[1].deg, c->posmap, c->att_items, ly.d_in,
              ly.act, c->H[l], c->ld[l], (float*)nullptr, (uint32_t*)nullptr);
    launch_gather(c, l);
    att_update(c, l, true);
}

// hop l of a batch, up to the cached rows; att_update then writes the embeddings
void att_hop(Ctx* c, int l, int n, bool small) {
    const LayerDev& ly = c->layer[l];
    const int ld = c->ws[l], T = 256;
    const int32_t* senders = c->Clist[(l - 1) & 1];   // = A_{l-1}, entered in the position map
    const float* Old = c->D[(l - 1) & 1];             // their rows before this batch, in list order
    RP_LAUNCH(c, k_att_scalars, c->n_sm * 4, T, 0, c->ctl, senders, (const int*)&c->ctl->nC[l - 1], 0, c->H[l - 1],
              c->ld[l - 1], ly.W1, c->att_s[l], c->att_t[l], c->att_so);
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l], c->stream);
#define PUSH(NV, LPR) RP_LAUNCH(c, (k_att_push<NV, LPR>), c->n_sm * 8, T, 0, c->ctl, l, senders, c->coff, c->side[0], c->posmap, c->H[l - 1], Old, c->ld[l - 1], c->att_so, c->att_s[l], c->att_t[l], ly.eps, ly.d_in, ld, c->dS[l], c->bitmap)
    RP_WIDTH_DISPATCH(ld, PUSH);
#undef PUSH
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l + 1], c->stream);
    if (n > 0)
        RP_LAUNCH(c, k_att_records, std::min(div_up(n, T / 32), c->n_sm * 8), T, 0, c->ctl, c->rec, c->posmap,
                  c->H[l - 1], Old, c->ld[l - 1], c->att_so, c->att_s[l], c->att_t[l], ly.eps, ly.d_in, ld, c->dS[l]);
    // the list A_l: the message walk has marked the sinks it reached, the rest is marked here
    frontier_mark_extras(c, l);
    if (small) frontier_compact_small(c, l);   // (a handful of updates on a graph whose bitmap one block can sweep)
    else frontier_compact(c, l);
    RP_LAUNCH(c, k_att_fold, c->n_sm * 8, T, 0, c->ctl, l, c->A[l], (const int*)&c->ctl->nA[l], 0, 0, ld, c->S[l],
              c->dS[l], c->Eb[l], c->rebuild_tau2, c->side[1].deg, c->posmap, c->att_items, ly.d_in, ly.act, c->H[l],
              c->ld[l], l == c->L ? (float*)nullptr : c->D[l & 1], c->bitmap);   // (the bitmap is free between two hops' markings)
    launch_gather(c, l);
    senders_release(c, l - 1);
}

}  // namespace rp
