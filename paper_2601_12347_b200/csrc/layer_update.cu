// Affected-row layer update (Compute + Prepare of Sec. 3.3.1): gather [h^{l-1}_v || x_v] for the
// rows of A_l, multiply by the layer weights, add bias, apply the activation, write h^l_v in
// place and emit the delta row D_v = c_new h_new - c_old h_old for the next hop (Sec. 3.3.3).
// fp32 SIMT path: register-tiled GEMM whose A operand is gathered by row id.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>

namespace rp {

__device__ __forceinline__ float coef_deg(int deg) { return deg > 0 ? 1.0f / sqrtf((float)deg) : 0.0f; }

enum { A_CONCAT = 0, A_SUM = 1, A_AGG = 2, A_DENSE = 3, A_SELF = 4 };
enum { EPI_COMMIT = 0, EPI_TEMP = 1 };

struct UpdParams {
    const int32_t* list;  // row ids (null: identity)
    const int* n_dev;     // row count on the device (null: n_host)
    int n_host;
    int a_mode, epi_mode;
    // A operand
    const float* Hprev; int ld_h;   // previous-layer rows (CONCAT, SUM) or dense rows (DENSE)
    const float* S; int ld_s;       // aggregate rows
    float alpha;                    // SUM: (1 + eps)
    int agg;                        // sink-side normalisation
    const int32_t* deg_in;
    int K;                          // reduction length (CONCAT: 2 * ld_h)
    // B operand
    const float* W; int ldw;        // K x ldw
    const float* bias;
    int n_cols;                     // ldw (padded output width)
    int act;
    // epilogue
    float* Hout; int ld_o;          // COMMIT: rows by id; TEMP: compact rows
    float* Dout;                    // COMMIT: compact delta rows (may be null)
    const float* addend; int ld_add; // rows by id added as row_scale * addend before bias (may be null)
    int src_norm;
    const int32_t* deg_out;
    const int32_t* deg_out_old;
};

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

__global__ void __launch_bounds__(256)
k_update_rows(const Ctl* ctl, UpdParams p) {
    if (ctl->abort) return;
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN];
    __shared__ int row_id[BM];
    __shared__ float row_scale[BM];
    const int n = p.n_dev ? *p.n_dev : p.n_host;
    const int row_tiles = (n + BM - 1) / BM, col_tiles = (p.n_cols + BN - 1) / BN;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    for (int tile = blockIdx.x; tile < row_tiles * col_tiles; tile += gridDim.x) {
        const int rt = tile / col_tiles, ct = tile - rt * col_tiles;
        const int r0 = rt * BM, c0 = ct * BN;
        __syncthreads();
        if (tid < BM) {
            int i = r0 + tid, v = -1;
            float sc = 0.f;
            if (i < n) {
                v = p.list ? p.list[i] : i;
                if (p.a_mode != A_DENSE) {
                    sc = 1.0f;
                    if (p.agg == RIPPLE_AGG_MEAN) { int d = p.deg_in[v]; sc = d > 0 ? 1.0f / (float)d : 0.f; }
                    else if (p.agg == RIPPLE_AGG_WSUM_GCN) sc = coef_deg(p.deg_in[v]);
                }
            }
            row_id[tid] = v;
            row_scale[tid] = sc;
        }
        __syncthreads();
        float acc[TM][TN];
#pragma unroll
        for (int a = 0; a < TM; ++a)
#pragma unroll
            for (int b = 0; b < TN; ++b) acc[a][b] = 0.f;

        const int ar = tid >> 2, ak = (tid & 3) * 4;   // A tile: row ar, k offset ak..ak+3
        const int bk = tid >> 4, bn = (tid & 15) * 4;  // B tile: k row bk, cols bn..bn+3
        for (int k0 = 0; k0 < p.K; k0 += BK) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            {
                const int v = row_id[ar], k = k0 + ak;
                if (v >= 0 && k < p.K) {
                    if (p.a_mode == A_DENSE) {
                        a = *reinterpret_cast<const float4*>(p.Hprev + (size_t)(r0 + ar) * p.ld_h + k);
                    } else if (p.a_mode == A_SELF) {
                        float4 h = __ldg(reinterpret_cast<const float4*>(p.Hprev + (size_t)v * p.ld_h + k));
                        a = make_float4(p.alpha * h.x, p.alpha * h.y, p.alpha * h.z, p.alpha * h.w);
                    } else if (p.a_mode == A_CONCAT) {
                        if (k < p.ld_h) a = __ldg(reinterpret_cast<const float4*>(p.Hprev + (size_t)v * p.ld_h + k));
                        else {
                            float4 s = *reinterpret_cast<const float4*>(p.S + (size_t)v * p.ld_s + (k - p.ld_h));
                            float sc = row_scale[ar];
                            a = make_float4(sc * s.x, sc * s.y, sc * s.z, sc * s.w);
                        }
                    } else {
                        float4 s = *reinterpret_cast<const float4*>(p.S + (size_t)v * p.ld_s + k);
                        float sc = row_scale[ar];
                        a = make_float4(sc * s.x, sc * s.y, sc * s.z, sc * s.w);
                        if (p.a_mode == A_SUM) {
                            float4 h = __ldg(reinterpret_cast<const float4*>(p.Hprev + (size_t)v * p.ld_h + k));
                            a.x += p.alpha * h.x; a.y += p.alpha * h.y; a.z += p.alpha * h.z; a.w += p.alpha * h.w;
                        }
                    }
                }
            }
            float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + bk < p.K && c0 + bn < p.n_cols)
                b = __ldg(reinterpret_cast<const float4*>(p.W + (size_t)(k0 + bk) * p.ldw + c0 + bn));
            __syncthreads();
            As[ak + 0][ar] = a.x; As[ak + 1][ar] = a.y; As[ak + 2][ar] = a.z; As[ak + 3][ar] = a.w;
            *reinterpret_cast<float4*>(&Bs[bk][bn]) = b;
            __syncthreads();
#pragma unroll
            for (int k = 0; k < BK; ++k) {
                float4 av = *reinterpret_cast<const float4*>(&As[k][ty * TM]);
                float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * TN]);
                const float ar4[4] = {av.x, av.y, av.z, av.w};
                const float br4[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                for (int a2 = 0; a2 < TM; ++a2)
#pragma unroll
                    for (int b2 = 0; b2 < TN; ++b2) acc[a2][b2] = fmaf(ar4[a2], br4[b2], acc[a2][b2]);
            }
        }
        // epilogue
        const int col = c0 + tx * TN;
        if (col < p.n_cols) {
            float4 bias = p.bias ? __ldg(reinterpret_cast<const float4*>(p.bias + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int a2 = 0; a2 < TM; ++a2) {
                const int lr = ty * TM + a2, v = row_id[lr];
                if (v < 0) continue;
                float4 h = make_float4(acc[a2][0] + bias.x, acc[a2][1] + bias.y, acc[a2][2] + bias.z, acc[a2][3] + bias.w);
                if (p.addend) {
                    float4 s = *reinterpret_cast<const float4*>(p.addend + (size_t)v * p.ld_add + col);
                    float sc = row_scale[lr];
                    h.x += sc * s.x; h.y += sc * s.y; h.z += sc * s.z; h.w += sc * s.w;
                }
                if (p.act == RIPPLE_ACT_RELU) { h.x = fmaxf(h.x, 0.f); h.y = fmaxf(h.y, 0.f); h.z = fmaxf(h.z, 0.f); h.w = fmaxf(h.w, 0.f); }
                if (p.epi_mode == EPI_TEMP) {
                    *reinterpret_cast<float4*>(p.Hout + (size_t)(r0 + lr) * p.ld_o + col) = h;
                } else {
                    float4* dst = reinterpret_cast<float4*>(p.Hout + (size_t)v * p.ld_o + col);
                    if (p.Dout) {
                        float4 o = *dst;
                        float cn = 1.f, co = 1.f;
                        if (p.src_norm) {
                            int dn = p.deg_out[v], dold = p.deg_out_old[v];
                            cn = coef_deg(dn);
                            co = dold >= 0 ? coef_deg(dold) : cn;
                        }
                        float4 d = make_float4(cn * h.x - co * o.x, cn * h.y - co * o.y, cn * h.z - co * o.z, cn * h.w - co * o.w);
                        *reinterpret_cast<float4*>(p.Dout + (size_t)(r0 + lr) * p.ld_o + col) = d;
                    }
                    *dst = h;
                }
            }
        }
    }
}

// rows_out[i] = rows_in[i] * W_n for i < n: the neighbour part of layer l applied to compact rows
// (sender deltas, record rows, or every embedding row at bootstrap)
void neighbour_transform(Ctx* c, int l, const float* rows_in, int ld_rows, const int* n_dev, int n_host,
                         float* rows_out) {
    const LayerDev& ly = c->layer[l];
    UpdParams p{};
    p.list = nullptr; p.n_dev = n_dev; p.n_host = n_host;
    p.a_mode = A_DENSE; p.epi_mode = EPI_TEMP;
    p.Hprev = rows_in; p.ld_h = ld_rows;
    p.K = ly.ld_in;
    p.W = ly.kind == RIPPLE_LAYER_SAGE ? ly.W1 + (size_t)ly.ld_in * ly.ld_out : ly.W1;
    p.ldw = c->ws[l]; p.bias = nullptr; p.n_cols = c->ws[l];
    p.act = RIPPLE_ACT_IDENTITY; p.Hout = rows_out; p.ld_o = c->ws[l];
    RP_LAUNCH(c, k_update_rows, c->n_sm * 4, 256, 0, c->ctl, p);
}

void update_rows(Ctx* c, int l, bool full) {
    const LayerDev& ly = c->layer[l];
    const bool pre = c->pre[l];
    UpdParams p{};
    p.list = full ? nullptr : c->A[l];
    p.n_dev = full ? nullptr : &c->ctl->nA[l];
    p.n_host = c->N;
    p.Hprev = c->H[l - 1]; p.ld_h = c->ld[l - 1];
    p.S = c->S[l]; p.ld_s = c->ws[l];
    p.alpha = 1.0f;
    p.agg = c->agg;
    p.deg_in = c->side[1].deg;
    p.src_norm = c->src_norm;
    p.deg_out = c->side[0].deg;
    p.deg_out_old = c->deg_out_old;
    if (pre) { p.addend = c->S[l]; p.ld_add = c->ws[l]; }
    const int grid = c->n_sm * 4;
    if (ly.kind == RIPPLE_LAYER_GIN) {
        // hidden = relu(W1^T ((1 + eps) h + x) + b1), kept as compact rows
        p.a_mode = pre ? A_SELF : A_SUM; p.epi_mode = EPI_TEMP; p.alpha = 1.0f + ly.eps;
        p.K = ly.ld_in; p.W = ly.W1; p.ldw = ly.ld_hid; p.bias = ly.b1; p.n_cols = ly.ld_hid;
        p.act = RIPPLE_ACT_RELU; p.Hout = c->T; p.ld_o = ly.ld_hid; p.Dout = nullptr;
        RP_LAUNCH(c, k_update_rows, grid, 256, 0, c->ctl, p);
        p.a_mode = A_DENSE; p.epi_mode = EPI_COMMIT; p.addend = nullptr;
        p.Hprev = c->T; p.ld_h = ly.ld_hid;
        p.K = ly.ld_hid; p.W = ly.W2; p.ldw = ly.ld_out; p.bias = ly.b2; p.n_cols = ly.ld_out;
        p.act = ly.act; p.Hout = c->H[l]; p.ld_o = ly.ld_out; p.Dout = (full || l == c->L) ? nullptr : c->D[l & 1];  // the last hop sends nothing
        RP_LAUNCH(c, k_update_rows, grid, 256, 0, c->ctl, p);
        return;
    }
    p.epi_mode = EPI_COMMIT;
    if (ly.kind == RIPPLE_LAYER_SAGE) {
        p.a_mode = pre ? A_SELF : A_CONCAT;
        p.K = pre ? ly.ld_in : 2 * ly.ld_in;
    } else {
        p.a_mode = A_AGG;
        p.K = pre ? 0 : ly.ld_in;   // transformed inbox: nothing left to multiply
    }
    p.W = ly.W1; p.ldw = ly.ld_out; p.bias = ly.b1; p.n_cols = ly.ld_out;
    p.act = ly.act; p.Hout = c->H[l]; p.ld_o = ly.ld_out; p.Dout = (full || l == c->L) ? nullptr : c->D[l & 1];  // the last hop sends nothing
    RP_LAUNCH(c, k_update_rows, grid, 256, 0, c->ctl, p);
}

// ---------------------------------------------------------------------------------------------
// hop 0: feature replacement rows and their deltas; one warp per vertex of A_0
// ---------------------------------------------------------------------------------------------
__global__ void k_feature_rows(Ctl* ctl, const ripple_update* __restrict__ ups, const float* __restrict__ feat,
                               int d0, const int32_t* __restrict__ A0, const int32_t* __restrict__ feat_last,
                               int src_norm, const int32_t* __restrict__ deg_out,
                               const int32_t* __restrict__ deg_out_old, float* H0, int ld, float* D) {
    if (ctl->abort) return;
    const int n = ctl->nA[0];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int i = warp; i < n; i += nwarps) {
        const int v = A0[i];
        const float* src = feat + (size_t)ups[feat_last[v]].v * d0;
        float cn = 1.f, co = 1.f;
        if (src_norm) {
            cn = coef_deg(deg_out[v]);
            co = deg_out_old[v] >= 0 ? coef_deg(deg_out_old[v]) : cn;
        }
        for (int k = lane_id(); k < ld; k += 32) {
            float x = k < d0 ? src[k] : 0.f;
            float o = H0[(size_t)v * ld + k];
            D[(size_t)i * ld + k] = cn * x - co * o;
            H0[(size_t)v * ld + k] = x;
        }
    }
}

void feature_rows(Ctx* c, int n) {
    if (n <= 0) return;
    RP_LAUNCH(c, k_feature_rows, std::min(div_up(n, 8), c->n_sm * 8), 256, 0, c->ctl, c->ups_dev, c->feat_dev,
              c->d[0], c->A[0], c->feat_last, (int)c->src_norm, c->side[0].deg, c->deg_out_old, c->H[0],
              c->ld[0], c->D[0]);
}

// ---------------------------------------------------------------------------------------------
// senders whose row did not change but whose source coefficient did: D_u = (c_new - c_old) h_u
// ---------------------------------------------------------------------------------------------
__global__ void k_extra_senders(Ctl* ctl, int l, const Rec* __restrict__ rec, int32_t* senders,
                                int32_t* posmap, const int32_t* __restrict__ deg_out,
                                const float* __restrict__ H, int ld, float* D) {
    if (ctl->abort) return;
    const int n = ctl->n_rec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int r = warp; r < n; r += nwarps) {
        const Rec x = rec[r];
        if (!x.rep[0]) continue;           // one record per distinct source
        if (posmap[x.u] >= 0) continue;    // already a sender: its delta came from the row update
        int idx = 0;
        if (lane_id() == 0) idx = atomicAdd(&ctl->nC[l], 1);
        idx = __shfl_sync(FULL, idx, 0);
        const float dc = coef_deg(deg_out[x.u]) - coef_deg(x.deg_out_old);
        for (int k = lane_id(); k < ld; k += 32) D[(size_t)idx * ld + k] = dc * H[(size_t)x.u * ld + k];
        if (lane_id() == 0) { senders[idx] = x.u; posmap[x.u] = idx; }
    }
}

void extra_sender_rows(Ctx* c, int l, int n) {
    RP_LAUNCH(c, k_extra_senders, std::min(div_up(n, 8), c->n_sm * 8), 256, 0, c->ctl, l, c->rec,
              c->Clist[l & 1], c->posmap, c->side[0].deg, c->H[l], c->ld[l], c->D[l & 1]);
}

}  // namespace rp
