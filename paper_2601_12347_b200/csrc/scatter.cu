// Delta-message scatter (Send + Aggregate of Sec. 3.3.1) and the bootstrap aggregation.
//
// S^l is the persistent, un-normalised inbox: S^l_v = sum_{u in In(v)} c_u h^{l-1}_u.  For hop l
//   S_v += sum over surviving and added edges (u, v) with u in C_{l-1} of D_u
//        + sum over added edges   (u, v) of M_u       (M_u = c_old(u) h_old(u): what the walk
//        - sum over deleted edges (u, v) of M_u        above did not, or wrongly did, deliver)
// with D_u = c_new h_new - c_old h_old the sender's delta row (Sec. 3.3.3: changed vertex; added
// edge = old contribution 0; deleted edge = new contribution 0; weighted form alpha h - alpha h-).
//
// push: the out-edges of the senders are cut into equal chunks; a warp keeps the sender's delta
//       row in registers and issues one 16-byte vector reduction per lane and edge.
// pull: a warp per affected sink walks its in-list, keeps only sources that are senders
//       (position map), sums their delta rows in registers and touches S_v once.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>

namespace rp {

__device__ __forceinline__ float coef_from_degree(int deg) {
    return deg > 0 ? 1.0f / sqrtf((float)deg) : 0.0f;
}

// ---------------------------------------------------------------------------------------------
// bootstrap: S_v for every vertex by gathering over in-edges (Eq. 1)
// ---------------------------------------------------------------------------------------------
template <int NV>  // float4 slots per lane: row width <= 128 * NV floats
__global__ void k_spmm_pull(int N, Side in, const int32_t* __restrict__ deg_out, int src_norm,
                            const float* __restrict__ Hprev, int ld, float* __restrict__ S) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int v = warp; v < N; v += nwarps) {
        float4 acc[NV];
#pragma unroll
        for (int k = 0; k < NV; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int64_t base = in.start[v];
        const int deg = in.deg[v];
        for (int j0 = 0; j0 < deg; j0 += 32) {
            int mine = j0 + lane < deg ? in.col[base + j0 + lane] : 0;
            int cnt = min(32, deg - j0);
            for (int j = 0; j < cnt; ++j) {
                int u = __shfl_sync(FULL, mine, j);
                float cu = src_norm ? coef_from_degree(deg_out[u]) : 1.0f;
                const float4* row = reinterpret_cast<const float4*>(Hprev + (size_t)u * ld);
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    int q = lane + 32 * k;
                    if (q < nq) {
                        float4 x = __ldg(row + q);
                        acc[k].x += cu * x.x; acc[k].y += cu * x.y; acc[k].z += cu * x.z; acc[k].w += cu * x.w;
                    }
                }
            }
        }
        float4* dst = reinterpret_cast<float4*>(S + (size_t)v * ld);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            int q = lane + 32 * k;
            if (q < nq) dst[q] = acc[k];
        }
    }
}

void spmm_full(Ctx* c, int l) {
    const int ld = c->ld[l - 1];
    const int nv = div_up(ld, 128);
    const int grid = c->n_sm * 16, T = 256;
#define SPMM(NV) RP_LAUNCH(c, k_spmm_pull<NV>, grid, T, 0, c->N, c->side[1], c->side[0].deg, (int)c->src_norm, c->H[l - 1], ld, c->S[l])
    if (nv <= 1) SPMM(1); else if (nv <= 2) SPMM(2); else if (nv <= 4) SPMM(4); else SPMM(8);
#undef SPMM
}

// ---------------------------------------------------------------------------------------------
// push scatter
// ---------------------------------------------------------------------------------------------
constexpr int PUSH_CHUNK = 64;  // edges per warp work item

template <int NV>
__global__ void __launch_bounds__(256)
k_scatter_push(Ctl* ctl, int l, const int32_t* __restrict__ senders, const int64_t* __restrict__ coff,
               Side out, const float* __restrict__ D, int ld, float* S) {
    if (ctl->abort || ctl->pull[l]) return;
    const int nC = ctl->nC[l - 1];
    if (nC == 0) return;
    const int64_t E = coff[nC];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int64_t e0 = (int64_t)warp * PUSH_CHUNK; e0 < E; e0 += (int64_t)nwarps * PUSH_CHUNK) {
        const int64_t e1 = min(e0 + PUSH_CHUNK, E);
        int i = upper_row(coff, nC, e0);
        int64_t e = e0;
        while (e < e1) {
            const int64_t row_end = coff[i + 1];
            if (row_end <= e) { ++i; continue; }
            const int64_t seg_end = min(e1, row_end);
            const int64_t base = out.start[senders[i]] + (e - coff[i]);
            float4 d[NV];
            const float4* drow = reinterpret_cast<const float4*>(D + (size_t)i * ld);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                int q = lane + 32 * k;
                d[k] = q < nq ? __ldg(drow + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const int cnt_total = (int)(seg_end - e);
            for (int j0 = 0; j0 < cnt_total; j0 += 32) {
                int mine = j0 + lane < cnt_total ? out.col[base + j0 + lane] : 0;
                int cnt = min(32, cnt_total - j0);
                for (int j = 0; j < cnt; ++j) {
                    int v = __shfl_sync(FULL, mine, j);
                    float* dst = S + (size_t)v * ld;
#pragma unroll
                    for (int k = 0; k < NV; ++k) {
                        int q = lane + 32 * k;
                        if (q < nq) red_add_v4(dst + 4 * q, d[k]);
                    }
                }
            }
            e = seg_end;
            ++i;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// pull scatter
// ---------------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(256)
k_scatter_pull(Ctl* ctl, int l, const int32_t* __restrict__ A, Side in, const int32_t* __restrict__ posmap,
               const float* __restrict__ D, int ld, float* S) {
    if (ctl->abort || !ctl->pull[l]) return;
    const int nA = ctl->nA[l];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int i = warp; i < nA; i += nwarps) {
        const int v = A[i];
        float4 acc[NV];
#pragma unroll
        for (int k = 0; k < NV; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int64_t base = in.start[v];
        const int deg = in.deg[v];
        bool any = false;
        for (int j0 = 0; j0 < deg; j0 += 32) {
            int p = -1;
            if (j0 + lane < deg) p = posmap[in.col[base + j0 + lane]];
            unsigned m = __ballot_sync(FULL, p >= 0);
            any |= m != 0;
            while (m) {
                int j = __ffs(m) - 1;
                m &= m - 1;
                int pj = __shfl_sync(FULL, p, j);
                const float4* drow = reinterpret_cast<const float4*>(D + (size_t)pj * ld);
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    int q = lane + 32 * k;
                    if (q < nq) {
                        float4 x = __ldg(drow + q);
                        acc[k].x += x.x; acc[k].y += x.y; acc[k].z += x.z; acc[k].w += x.w;
                    }
                }
            }
        }
        if (!any) continue;
        float4* dst = reinterpret_cast<float4*>(S + (size_t)v * ld);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            int q = lane + 32 * k;
            if (q < nq) {
                float4 s = dst[q];
                s.x += acc[k].x; s.y += acc[k].y; s.z += acc[k].z; s.w += acc[k].w;
                dst[q] = s;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// edge-change records: +- M_u into the sink's aggregate; one warp per record
// ---------------------------------------------------------------------------------------------
__global__ void k_scatter_records(Ctl* ctl, const Rec* __restrict__ rec, int src_norm,
                                  const int32_t* __restrict__ deg_out, const int32_t* __restrict__ posmap,
                                  const float* __restrict__ Hprev, const float* __restrict__ D, int ld,
                                  float* S) {
    if (ctl->abort) return;
    const int n = ctl->n_rec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int r = warp; r < n; r += nwarps) {
        const Rec x = rec[r];
        const float sgn = (float)x.sign;
        const int p = posmap[x.u];
        const float4* hrow = reinterpret_cast<const float4*>(Hprev + (size_t)x.u * ld);
        float* dst = S + (size_t)x.v * ld;
        // M_u = c_old h_old = c_new h_new - D_u for a sender, c h otherwise
        const float cn = src_norm ? coef_from_degree(deg_out[x.u]) : 1.0f;
        for (int q = lane; q < nq; q += 32) {
            float4 h = __ldg(hrow + q);
            float4 m = make_float4(cn * h.x, cn * h.y, cn * h.z, cn * h.w);
            if (p >= 0) {
                float4 d = __ldg(reinterpret_cast<const float4*>(D + (size_t)p * ld) + q);
                m.x -= d.x; m.y -= d.y; m.z -= d.z; m.w -= d.w;
            }
            red_add_v4(dst + 4 * q, make_float4(sgn * m.x, sgn * m.y, sgn * m.z, sgn * m.w));
        }
    }
}

// decide the direction of hop l on the device
__global__ void k_choose_direction(Ctl* ctl, int l, int mode, int ld) {
    if (mode == RIPPLE_SCATTER_PULL) { ctl->pull[l] = 1; return; }
    if (mode == RIPPLE_SCATTER_PUSH) { ctl->pull[l] = 0; return; }
    // bytes moved from DRAM: push reads and writes one aggregate row per message; pull reads the
    // in-lists of all affected sinks and touches each aggregate row once
    double push = (double)ctl->E[l] * (8.0 * ld);
    double pull = (double)ctl->pull_work[l] * 8.0 + (double)ctl->nA[l] * (8.0 * ld) +
                  (double)ctl->E[l] * (0.5 * ld);
    ctl->pull[l] = pull < push;
}

void scatter_layer(Ctx* c, int l, int n) {
    const int ld = c->ld[l - 1];
    const int nv = div_up(ld, 128);
    const float* D = c->D[(l - 1) & 1];
    const int32_t* senders = c->Clist[(l - 1) & 1];
    RP_LAUNCH(c, k_choose_direction, 1, 1, 0, c->ctl, l, c->scatter_mode, ld);
    const int T = 256;
    const int grid = c->n_sm * 8;
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l], c->stream);
#define PUSH(NV) RP_LAUNCH(c, k_scatter_push<NV>, grid, T, 0, c->ctl, l, senders, c->coff, c->side[0], D, ld, c->S[l])
#define PULL(NV) RP_LAUNCH(c, k_scatter_pull<NV>, grid, T, 0, c->ctl, l, c->A[l], c->side[1], c->posmap, D, ld, c->S[l])
    if (c->scatter_mode != RIPPLE_SCATTER_PULL) {
        if (nv <= 1) PUSH(1); else if (nv <= 2) PUSH(2); else if (nv <= 4) PUSH(4); else PUSH(8);
    }
    if (c->scatter_mode != RIPPLE_SCATTER_PUSH) {
        if (nv <= 1) PULL(1); else if (nv <= 2) PULL(2); else if (nv <= 4) PULL(4); else PULL(8);
    }
#undef PUSH
#undef PULL
    if (c->timing) cudaEventRecord(c->ev_sc[2 * l + 1], c->stream);
    if (n > 0)
        RP_LAUNCH(c, k_scatter_records, std::min(div_up(n, T / 32), c->n_sm * 8), T, 0, c->ctl, c->rec,
                  (int)c->src_norm, c->side[0].deg, c->posmap, c->H[l - 1], D, ld, c->S[l]);
}

}  // namespace rp
