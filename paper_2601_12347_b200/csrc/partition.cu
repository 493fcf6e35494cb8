// Partitioned execution (Sec. 4): the device side of the exchange between workers.
//
// A worker's halo slots are the remote endpoints of its cut edges.  During a hop the local sends of
// the push scatter land in the accumulator rows of local sinks and of halo slots alike; a halo slot's
// row is the mailbox in which the partition's messages for that remote vertex are combined (Sec. 4.2).
// The remote send (Sec. 4.5) is one kernel: every marked halo mailbox is added to the owner's
// accumulator row through a peer pointer, the vertex is marked in the owner's frontier bitmap, and
// the mailbox and its mark are cleared.  The owner's fold then aggregates what arrived from all
// partitions together with its own local messages.  Nothing here waits for another GPU.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>

namespace rp {

struct PeerTab {
    float* dS[RIPPLE_MAX_PEERS];
    const float* H[RIPPLE_MAX_PEERS];
    uint32_t* bitmap[RIPPLE_MAX_PEERS];
    const int32_t* deg_out[RIPPLE_MAX_PEERS];
};

// 16-byte vector reduction that another GPU's memory may be the target of
__device__ __forceinline__ void red_add_v4_sys(float* addr, float4 v) {
    asm volatile("red.relaxed.sys.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y),
                 "f"(v.z), "f"(v.w)
                 : "memory");
}

// one warp per bitmap word of the halo range (n_local is a multiple of 32)
__global__ void __launch_bounds__(256)
k_part_ship(Ctl* ctl, int l, int n_local, int n_words, uint32_t* bitmap, float* dS, int ld,
            const int32_t* __restrict__ halo_owner, const int32_t* __restrict__ halo_rid, PeerTab peers,
            unsigned long long* rows_sent) {
    pdl_enter();
    if (ctl->abort) return;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int w = (n_local >> 5) + warp; w < n_words; w += nwarps) {
        uint32_t bits = bitmap[w];
        if (!bits) continue;
        __syncwarp();
        if (lane == 0) {
            bitmap[w] = 0u;
            atomicAdd(&rows_sent[l], (unsigned long long)__popc(bits));
        }
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            const int lid = (w << 5) + b, h = lid - n_local;
            const int owner = halo_owner[h], rid = halo_rid[h];
            float4* row = reinterpret_cast<float4*>(dS + (size_t)lid * ld);
            if (owner >= 0 && peers.dS[owner] && peers.bitmap[owner]) {   // (the host refuses a hop whose peers are not all registered)
                float* dst = peers.dS[owner] + (size_t)rid * ld;
                for (int q = lane; q < nq; q += 32) red_add_v4_sys(dst + 4 * q, row[q]);
                if (lane == 0) atomicOr_system(&peers.bitmap[owner][rid >> 5], 1u << (rid & 31));
            }
            for (int q = lane; q < nq; q += 32) row[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

// One warp per assigned halo slot: its row of H^l is copied from the owner.  With coefficients on the source
// side (src_norm: 1 / sqrt of the out-degree) the gather that follows would scale the row by this worker's
// partial out-degree of the halo vertex; the copy is pre-scaled so that the product is the owner's coefficient.
__global__ void __launch_bounds__(256)
k_part_fetch(int n_local, int n_halo, float* H, int ld, const int32_t* __restrict__ halo_owner,
             const int32_t* __restrict__ halo_rid, PeerTab peers, int src_norm, const int32_t* __restrict__ deg_out) {
    pdl_enter();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    const int lane = lane_id(), nq = ld >> 2;
    for (int h = warp; h < n_halo; h += nwarps) {
        const int owner = halo_owner[h];
        if (owner < 0 || !peers.H[owner]) continue;
        const float4* src = reinterpret_cast<const float4*>(peers.H[owner] + (size_t)halo_rid[h] * ld);
        float4* dst = reinterpret_cast<float4*>(H + (size_t)(n_local + h) * ld);
        float a = 1.f;
        if (src_norm) {
            const int d_here = deg_out[n_local + h], d_true = peers.deg_out[owner][halo_rid[h]];
            a = (d_here > 0 && d_true > 0) ? sqrtf((float)d_here / (float)d_true) : 0.f;
        }
        for (int q = lane; q < nq; q += 32) {
            float4 x = src[q];
            dst[q] = make_float4(a * x.x, a * x.y, a * x.z, a * x.w);
        }
    }
}

static PeerTab peer_table(const Ctx* c, int l) {
    PeerTab t{};
    for (int p = 0; p < RIPPLE_MAX_PEERS; ++p) {
        t.dS[p] = c->peer_dS[p][l];
        t.H[p] = c->peer_H[p][l];
        t.bitmap[p] = c->peer_bitmap[p];
        t.deg_out[p] = c->peer_deg_out[p];
    }
    return t;
}

void part_ship(Ctx* c, int l) {
    const int halo_words = c->n_words - (c->n_local >> 5);
    if (halo_words <= 0) return;
    RP_LAUNCH(c, k_part_ship, std::min(div_up(halo_words, 8), c->n_sm * 8), 256, 0, c->ctl, l, c->n_local, c->n_words,
              c->bitmap, c->dS[l], c->ws[l], c->halo_owner, c->halo_rid, peer_table(c, l), c->rows_sent);
}

void part_fetch_halo_rows(Ctx* c, int l) {
    const int n_halo = c->N - c->n_local;
    if (n_halo <= 0) return;
    RP_LAUNCH(c, k_part_fetch, std::min(div_up(n_halo, 8), c->n_sm * 8), 256, 0, c->n_local, n_halo, c->H[l], c->ld[l],
              c->halo_owner, c->halo_rid, peer_table(c, l), (int)c->src_norm, c->side[0].deg);
}

}  // namespace rp
