// Shared between the SIMT and the tensor-core form of the affected-row layer update: the
// parameter block, the gathered A operand and the fused epilogue.
#pragma once

#include "device_utils.cuh"
#include "ripple_internal.cuh"

namespace rp {

// A operand: SUM = alpha h_v + scale S_v (GIN); AGG = scale S_v; DENSE = compact rows; SELF = alpha h_v
enum { A_SUM = 1, A_AGG = 2, A_DENSE = 3, A_SELF = 4 };
enum { EPI_COMMIT = 0, EPI_TEMP = 1 };
enum { TC_OFF = 0, TC_TF32X3 = 1, TC_TF32 = 2 };

struct UpdParams {
    const int32_t* list;  // row ids (null: identity)
    const int* n_dev;     // row count on the device (null: n_host)
    int n_host;
    int a_mode, epi_mode;
    // A operand
    const float* Hprev; int ld_h;   // previous-layer rows (SUM, SELF) or dense rows (DENSE)
    const float* S; int ld_s;       // aggregate rows
    float alpha;                    // SUM, SELF: factor on the self row
    int agg;                        // sink-side normalisation
    const int32_t* deg_in;
    int K;                          // reduction length
    // B operand
    const float* W; int ldw;        // K x ldw, row-major (SIMT form)
    const float* Wt_hi;             // tensor-core form: transposed (n_pad x k_pad, K contiguous), split
    const float* Wt_lo;             //   into a tf32-exact part and the remainder
    int k_pad, n_pad;
    const float* bias;
    int n_cols;                     // ldw (padded output width)
    int act;
    // epilogue
    float* Hout; int ld_o;          // COMMIT: rows by id; TEMP: compact rows
    float* Dout;                    // COMMIT: compact delta rows (may be null)
    const float* addend; int ld_add; // rows by id added as row_scale * addend (may be null)
    const float* addend2;           // rows by id added as they are, same leading dimension (may be null)
    float* addend_rw;               // if set: addend with its pending per-batch sums folded in on the way
    float* addend_delta;            //   (addend_rw += addend_delta, addend_delta = 0); replaces addend
    int dout_old;                   // Dout receives the row's previous value instead of a delta (monotonic aggregation)
    int src_norm;
    const int32_t* deg_out;
    const int32_t* deg_out_old;
    // form selection (decided on the device from the row count)
    int tc_mode;                    // TC_OFF: SIMT only
    int tc_min_rows;
    int tc_withhold;                // diagnostic: the tensor-core kernel never signals its first finished tile
    int narrow_min_rows;            // > 0: launches of at least this many rows belong to the form for narrow outputs
};

__device__ __forceinline__ float coef_deg(int deg) { return deg > 0 ? 1.0f / sqrtf((float)deg) : 0.0f; }

__device__ __forceinline__ int upd_rows(const UpdParams& p) { return p.n_dev ? *p.n_dev : p.n_host; }

// true if this launch's row count belongs to the tensor-core kernel
__device__ __forceinline__ bool upd_use_tc(const UpdParams& p, int n) {
    return p.tc_mode != TC_OFF && n >= p.tc_min_rows;
}

// true if this launch's row count belongs to the SIMT form for narrow outputs (k_update_rows_narrow)
__device__ __forceinline__ bool upd_use_narrow(const UpdParams& p, int n) {
    return p.narrow_min_rows > 0 && n >= p.narrow_min_rows;
}

__device__ __forceinline__ float upd_row_scale(const UpdParams& p, int v) {
    if (p.a_mode == A_DENSE) return 0.f;
    if (p.agg == RIPPLE_AGG_MEAN) { int d = p.deg_in[v]; return d > 0 ? 1.0f / (float)d : 0.f; }
    if (p.agg == RIPPLE_AGG_WSUM_GCN) return coef_deg(p.deg_in[v]);
    return 1.0f;
}

// four consecutive entries k..k+3 of the A operand's row for vertex v (compact index i), k < K
__device__ __forceinline__ float4 upd_load_a(const UpdParams& p, int v, int i, int k, float sc) {
    if (p.a_mode == A_DENSE) return *reinterpret_cast<const float4*>(p.Hprev + (size_t)i * p.ld_h + k);
    if (p.a_mode == A_SELF) {
        float4 h = __ldg(reinterpret_cast<const float4*>(p.Hprev + (size_t)v * p.ld_h + k));
        return make_float4(p.alpha * h.x, p.alpha * h.y, p.alpha * h.z, p.alpha * h.w);
    }
    float4 s = *reinterpret_cast<const float4*>(p.S + (size_t)v * p.ld_s + k);
    float4 a = make_float4(sc * s.x, sc * s.y, sc * s.z, sc * s.w);
    if (p.a_mode == A_SUM) {
        float4 h = __ldg(reinterpret_cast<const float4*>(p.Hprev + (size_t)v * p.ld_h + k));
        a.x += p.alpha * h.x; a.y += p.alpha * h.y; a.z += p.alpha * h.z; a.w += p.alpha * h.w;
    }
    return a;
}

// true if the epilogue needs the row's previous value (to emit a delta row)
__device__ __forceinline__ bool upd_needs_old(const UpdParams& p) { return p.epi_mode == EPI_COMMIT && p.Dout; }

__device__ __forceinline__ float4 upd_load_old(const UpdParams& p, int v, int col) {
    return *reinterpret_cast<const float4*>(p.Hout + (size_t)v * p.ld_o + col);
}

// bias, optional addend, activation, then either a compact temp row or commit + delta row;
// `old` / `zpre` are the previously stored value and the addend2 value if the caller has
// prefetched them (has_old / has_z)
__device__ __forceinline__ void upd_epilogue4(const UpdParams& p, int v, int i, int col, float4 h, float sc,
                                              bool has_old = false,
                                              float4 old = make_float4(0.f, 0.f, 0.f, 0.f),
                                              bool has_z = false,
                                              float4 zpre = make_float4(0.f, 0.f, 0.f, 0.f)) {
    if (p.bias) {
        float4 b = __ldg(reinterpret_cast<const float4*>(p.bias + col));
        h.x += b.x; h.y += b.y; h.z += b.z; h.w += b.w;
    }
    if (p.addend_rw) {
        // every (row, column) of the aggregate is touched by exactly one thread, so the batch's
        // message sums can be folded into it here instead of in a pass of their own
        float4* sp = reinterpret_cast<float4*>(p.addend_rw + (size_t)v * p.ld_add + col);
        float4* dp = reinterpret_cast<float4*>(p.addend_delta + (size_t)v * p.ld_add + col);
        float4 s = *sp, d = *dp;
        s.x += d.x; s.y += d.y; s.z += d.z; s.w += d.w;
        *sp = s;
        *dp = make_float4(0.f, 0.f, 0.f, 0.f);
        h.x += sc * s.x; h.y += sc * s.y; h.z += sc * s.z; h.w += sc * s.w;
    } else if (p.addend) {
        float4 s = *reinterpret_cast<const float4*>(p.addend + (size_t)v * p.ld_add + col);
        h.x += sc * s.x; h.y += sc * s.y; h.z += sc * s.z; h.w += sc * s.w;
    }
    if (p.addend2) {
        float4 z = has_z ? zpre : *reinterpret_cast<const float4*>(p.addend2 + (size_t)v * p.ld_add + col);
        h.x += z.x; h.y += z.y; h.z += z.z; h.w += z.w;
    }
    if (p.act == RIPPLE_ACT_RELU) {
        h.x = fmaxf(h.x, 0.f); h.y = fmaxf(h.y, 0.f); h.z = fmaxf(h.z, 0.f); h.w = fmaxf(h.w, 0.f);
    }
    if (p.epi_mode == EPI_TEMP) {
        *reinterpret_cast<float4*>(p.Hout + (size_t)i * p.ld_o + col) = h;
        return;
    }
    float4* dst = reinterpret_cast<float4*>(p.Hout + (size_t)v * p.ld_o + col);
    if (p.Dout) {
        float4 o = has_old ? old : *dst;
        float cn = 1.f, co = 1.f;
        if (p.src_norm) {
            int dold = p.deg_out_old[v];
            cn = coef_deg(p.deg_out[v]);
            co = dold >= 0 ? coef_deg(dold) : cn;
        }
        *reinterpret_cast<float4*>(p.Dout + (size_t)i * p.ld_o + col) =
            p.dout_old ? o
                       : make_float4(cn * h.x - co * o.x, cn * h.y - co * o.y, cn * h.z - co * o.z, cn * h.w - co * o.w);
    }
    *dst = h;
}

// layer_update_tc.cu
void launch_update_tc(Ctx* c, const UpdParams& p);

}  // namespace rp
