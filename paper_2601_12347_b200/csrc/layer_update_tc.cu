// Tensor-core form of the affected-row layer update for sm_100a: tcgen05.mma (kind::tf32) with
// the accumulator tile in tensor memory.
//
// One CTA owns tiles of 128 affected rows x all (<= 256) output columns.  Per 32-float K chunk the
// CTA's threads gather the A rows by vertex id (applying the sink normalisation or the GIN self
// factor on the way), split every fp32 value x into hi = x with the 13 low mantissa bits cleared
// (exactly representable in tf32) and lo = x - hi, and store both into shared memory in the
// K-major 128-byte-swizzle layout the tensor core reads; the transposed weights arrive pre-split
// the same way.  One elected thread then issues hi*hi + lo*hi + hi*lo (three MMAs per 8-float K
// step), which reproduces the fp32 product to about 2^-21 relative, and commits to an mbarrier
// so that the next-but-one chunk can reuse the stage.  With tc_mode = TC_TF32 only hi*hi is
// issued (plain TF32, 2^-11).  The epilogue reads the accumulators back with tcgen05.ld, one row
// per thread, and runs the same fused bias / activation / delta / commit code as the SIMT form.
//
// Every wait is bounded: if an mbarrier does not complete within the spin limit the CTA records
// RIPPLE_ERR_TIMEOUT in the control block, frees its tensor memory and returns.
#include "layer_update.cuh"

#include <algorithm>
#include <cstring>
#include <vector>

namespace rp {

constexpr int TC_M = 128;        // rows per tile (= TMEM lanes)
constexpr int TC_KC = 32;        // floats per K chunk: one 128-byte swizzle row
constexpr int TC_THREADS = 256;
constexpr int TC_A_BYTES = TC_M * 128;
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// true once the phase with the given parity has completed; gives up after TC_SPIN_LIMIT polls
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < TC_SPIN_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;             // leading byte offset (not used by swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;             // descriptor version
    d |= (uint64_t)2 << 61;             // SWIZZLE_128B
    return d;
}

__device__ __forceinline__ void tc_mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}

// byte offset of 16-byte chunk c (0..7) of row r inside a K-major SWIZZLE_128B tile
__device__ __forceinline__ uint32_t tc_swz(int r, int c) {
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + (((c ^ r) & 7) << 4));
}

__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const float* gptr) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gptr) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// barrier among the loader warps only (the MMA warp never joins it)
__device__ __forceinline__ void loaders_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TC_THREADS) : "memory"); }

// Warp roles: warps 0..7 ("loaders") stage the operands of every K chunk and run the epilogue;
// warp 8 issues the MMAs.  Two mbarriers per stage hand the stage back and forth:
//   full[s]   8 arrivals (one per loader warp, after its stores and proxy fence) -> MMA warp may read
//   empty[s]  1 arrival (tcgen05.commit of the MMAs that read the stage)         -> loaders may refill
// so the single-thread MMA issue (a microsecond per chunk) overlaps the loads of the next chunk.
template <bool X3>
__global__ void __launch_bounds__(TC_THREADS + 32, 1)
k_update_rows_tc(Ctl* ctl, UpdParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[2], empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int row_id[TC_M];
    __shared__ float row_scale[TC_M];
    __shared__ volatile int s_fail;

    if (ctl->abort) return;
    const int n = upd_rows(p);
    if (!upd_use_tc(p, n)) return;
    const int row_tiles = (n + TC_M - 1) / TC_M;
    if ((int)blockIdx.x >= row_tiles) return;   // before any allocation

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_mma_warp = warp == TC_THREADS / 32;
    const int n_pad = p.n_pad;
    const uint32_t b_bytes = (uint32_t)n_pad * 128u;
    const uint32_t stage_bytes = (X3 ? 2u : 1u) * (TC_A_BYTES + b_bytes);
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < n_pad) tmem_cols <<= 1;

    if (tid == 0) {
        mbar_init(&full[0], TC_THREADS / 32);
        mbar_init(&full[1], TC_THREADS / 32);
        mbar_init(&empty[0], 1);
        mbar_init(&empty[1], 1);
        s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    // instruction descriptor: fp32 accumulate, tf32 x tf32, both K-major, N = n_pad, M = 128
    const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n_pad >> 3) << 17) |
                           ((uint32_t)(TC_M >> 4) << 24);
    const int nchunks = p.k_pad / TC_KC;
    uint32_t uses[2] = {0u, 0u};   // how often each stage has been handed over so far (same in every thread)

    if (is_mma_warp) {
        // ---------------- MMA issue ----------------
        for (int tile = blockIdx.x; tile < row_tiles && !s_fail; tile += gridDim.x) {
            for (int kc = 0; kc < nchunks; ++kc) {
                const int s = kc & 1;
                uint8_t* a_hi = smem + (size_t)s * stage_bytes;
                uint8_t* a_lo = a_hi + TC_A_BYTES;
                uint8_t* b_hi = a_hi + (X3 ? 2 : 1) * TC_A_BYTES;
                uint8_t* b_lo = b_hi + b_bytes;
                if (lane == 0) {
                    if (!mbar_wait_bounded(&full[s], uses[s] & 1)) s_fail = 1;
                    if (!s_fail) {
                        tc_fence_after();
                        const uint64_t da_hi = tc_smem_desc(smem_u32(a_hi)), db_hi = tc_smem_desc(smem_u32(b_hi));
                        const uint64_t da_lo = tc_smem_desc(smem_u32(a_lo)), db_lo = tc_smem_desc(smem_u32(b_lo));
#pragma unroll
                        for (int j = 0; j < TC_KC / 8; ++j) {     // one MMA K step = 8 floats = 32 bytes
                            const uint64_t adv = (uint64_t)((j * 32) >> 4);
                            tc_mma_tf32(tmem_base, da_hi + adv, db_hi + adv, idesc, (kc | j) != 0);
                            if (X3) {
                                tc_mma_tf32(tmem_base, da_lo + adv, db_hi + adv, idesc, 1u);
                                tc_mma_tf32(tmem_base, da_hi + adv, db_lo + adv, idesc, 1u);
                            }
                        }
                        tc_commit(&empty[s]);
                    }
                }
                __syncwarp();
                uses[s]++;
                if (s_fail) break;
            }
        }
    } else {
        // ---------------- loaders + epilogue ----------------
        for (int tile = blockIdx.x; tile < row_tiles && !s_fail; tile += gridDim.x) {
            const int r0 = tile * TC_M;
            if (tid < TC_M) {
                int i = r0 + tid, v = -1;
                float sc = 0.f;
                if (i < n) {
                    v = p.list ? p.list[i] : i;
                    sc = upd_row_scale(p, v);
                }
                row_id[tid] = v;
                row_scale[tid] = sc;
            }
            loaders_sync();

            // The gathered A rows come from DRAM, the weights from L2: A is therefore loaded one chunk
            // further ahead (registers), so that two chunks of row gathers are in flight.
            constexpr int A_ITERS = (TC_M * 8) / TC_THREADS;
            constexpr int B_ITERS = (256 * 8) / TC_THREADS;   // n_pad <= 256
            float4 ax[A_ITERS], ax_next[A_ITERS];
            auto load_a = [&](int kc, float4 (&dst)[A_ITERS]) {
#pragma unroll
                for (int it = 0; it < A_ITERS; ++it) {   // 128 rows x 8 chunks of 16 bytes, by vertex id
                    const int idx = tid + it * TC_THREADS, r = idx >> 3, c = idx & 7;
                    const int v = row_id[r], k = kc * TC_KC + c * 4;
                    dst[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (v >= 0 && k < p.K) dst[it] = upd_load_a(p, v, r0 + r, k, row_scale[r]);
                }
            };
            // asynchronous copy of chunk kc's pre-split transposed weights (n_pad output columns x 8
            // pieces of 16 bytes, hi and lo) from L2 straight into their swizzled places in stage kc & 1;
            // the MMAs that last read that stage must have finished
            auto copy_b = [&](int kc) {
                const int s = kc & 1;
                uint8_t* b_hi = smem + (size_t)s * stage_bytes + (X3 ? 2 : 1) * TC_A_BYTES;
                uint8_t* b_lo = b_hi + b_bytes;
                if (uses[s] > 0 && !mbar_wait_bounded(&empty[s], (uses[s] - 1) & 1)) s_fail = 1;
#pragma unroll
                for (int it = 0; it < B_ITERS; ++it) {
                    const int idx = tid + it * TC_THREADS;
                    if (idx < n_pad * 8) {
                        const size_t g = (size_t)(idx >> 3) * p.k_pad + kc * TC_KC + (idx & 7) * 4;
                        const uint32_t off = tc_swz(idx >> 3, idx & 7);
                        cp_async16(smem_u32(b_hi + off), p.Wt_hi + g);
                        if (X3) cp_async16(smem_u32(b_lo + off), p.Wt_lo + g);
                    }
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            };
            load_a(0, ax);
            copy_b(0);
            for (int kc = 0; kc < nchunks; ++kc) {
                const int s = kc & 1;
                uint8_t* a_hi = smem + (size_t)s * stage_bytes;
                uint8_t* a_lo = a_hi + TC_A_BYTES;                              // only if X3
                // next chunk's row gathers first (registers), so that they have a whole iteration to land
                if (kc + 1 < nchunks) load_a(kc + 1, ax_next);
#pragma unroll
                for (int it = 0; it < A_ITERS; ++it) {
                    const int idx = tid + it * TC_THREADS;
                    const uint32_t off = tc_swz(idx >> 3, idx & 7);
                    const float4 x = ax[it];
                    const float4 h = make_float4(tf32_hi(x.x), tf32_hi(x.y), tf32_hi(x.z), tf32_hi(x.w));
                    *reinterpret_cast<float4*>(a_hi + off) = h;
                    if (X3) *reinterpret_cast<float4*>(a_lo + off) = make_float4(x.x - h.x, x.y - h.y, x.z - h.z, x.w - h.w);
                }
                asm volatile("cp.async.wait_group 0;" ::: "memory");   // this chunk's weights have landed
                fence_async_smem();   // generic-proxy stores -> visible to the tensor core's async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[s]);
                uses[s]++;
                // the next chunk's weights travel while its rows are split and stored
                if (kc + 1 < nchunks) copy_b(kc + 1);
#pragma unroll
                for (int it = 0; it < A_ITERS; ++it) ax[it] = ax_next[it];
                if (s_fail) break;
            }
            if (s_fail) break;
            // the last commit covers every MMA of the tile
            {
                const int s = (nchunks - 1) & 1;
                if (!mbar_wait_bounded(&empty[s], (uses[s] - 1) & 1)) s_fail = 1;
            }
            if (s_fail) break;
            tc_fence_after();

            // Epilogue in two steps.  (1) Every thread copies its accumulator row (warp w: tensor-memory
            // lanes 32 (w % 4).., warps 0-3 the first half of the 16-column blocks, warps 4-7 the rest)
            // into a row-major tile in shared memory; the operand stages are free now.  (2) Each warp
            // then takes whole rows, 32 lanes x 16 bytes per pass, so that the previous row, the cached
            // projection, the delta row and the new row all move in coalesced 512-byte pieces, four
            // rows in flight.
            float* tile_s = reinterpret_cast<float*>(smem);
            const int tstride = n_pad + 4;   // = 4 mod 32: conflict-free 16-byte stores down a column
            {
                const int g = warp & 3, half = warp >> 2;
                const int nblk = n_pad >> 4, split = (nblk + 1) >> 1;
                const int b0 = half ? split : 0, b1 = half ? nblk : split;
                const int r = 32 * g + lane;
                for (int blk = b0; blk < b1; ++blk) {
                    uint32_t x[16];
                    const uint32_t taddr = tmem_base + ((uint32_t)(32 * g) << 16) + (uint32_t)(blk * 16);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                        : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]),
                          "=r"(x[7]), "=r"(x[8]), "=r"(x[9]), "=r"(x[10]), "=r"(x[11]), "=r"(x[12]), "=r"(x[13]),
                          "=r"(x[14]), "=r"(x[15])
                        : "r"(taddr) : "memory");
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    float4* dst = reinterpret_cast<float4*>(tile_s + (size_t)r * tstride + blk * 16);
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dst[q] = make_float4(__uint_as_float(x[4 * q]), __uint_as_float(x[4 * q + 1]),
                                             __uint_as_float(x[4 * q + 2]), __uint_as_float(x[4 * q + 3]));
                }
            }
            tc_fence_before();   // accumulators consumed: the MMA warp may overwrite them after our next arrival
            loaders_sync();
            {
                constexpr int RUN = 4;                       // rows in flight per warp
                const bool need_old = upd_needs_old(p);
                const bool need_z = p.addend2 != nullptr;
                const int npass = (p.n_cols + 127) >> 7;     // <= 2
                for (int rb = warp; rb < TC_M; rb += (TC_THREADS / 32) * RUN) {
                    int vv[RUN];
                    float4 oldv[RUN][2], zv[RUN][2];
#pragma unroll
                    for (int t = 0; t < RUN; ++t) {
                        const int r = rb + t * (TC_THREADS / 32);
                        vv[t] = r < TC_M ? row_id[r] : -1;
#pragma unroll
                        for (int ps = 0; ps < 2; ++ps) {
                            const int col = 4 * lane + 128 * ps;
                            if (vv[t] >= 0 && ps < npass && col < p.n_cols) {
                                if (need_old) oldv[t][ps] = upd_load_old(p, vv[t], col);
                                if (need_z) zv[t][ps] = *reinterpret_cast<const float4*>(p.addend2 + (size_t)vv[t] * p.ld_add + col);
                            }
                        }
                    }
#pragma unroll
                    for (int t = 0; t < RUN; ++t) {
                        const int r = rb + t * (TC_THREADS / 32);
                        if (vv[t] < 0) continue;
#pragma unroll
                        for (int ps = 0; ps < 2; ++ps) {
                            const int col = 4 * lane + 128 * ps;
                            if (ps < npass && col < p.n_cols) {
                                const float4 acc = *reinterpret_cast<const float4*>(tile_s + (size_t)r * tstride + col);
                                upd_epilogue4(p, vv[t], r0 + r, col, acc, row_scale[r], need_old, oldv[t][ps], need_z, zv[t][ps]);
                            }
                        }
                    }
                }
            }
            // the tile buffer (= the operand stages) and row_id are free before the next tile's staging
            loaders_sync();
        }
    }

    if (s_fail && lane == 0) {
        atomicCAS(&ctl->err, 0, (int)RIPPLE_ERR_TIMEOUT);
        ctl->abort = 1;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

void launch_update_tc(Ctx* c, const UpdParams& p) {
    const bool x3 = p.tc_mode == TC_TF32X3;
    const size_t stage = (size_t)(x3 ? 2 : 1) * (TC_A_BYTES + (size_t)p.n_pad * 128);
    // two operand stages, reused by the epilogue as a 128 x (n_pad + 4) fp32 tile
    const size_t tile = (size_t)TC_M * (p.n_pad + 4) * sizeof(float);
    const size_t smem = std::max(2 * stage, tile) + 1024;
    const int per_sm = std::max<size_t>(1, std::min<size_t>(4, (size_t)(220 * 1024) / (smem + 2048)));
    const int grid = c->n_sm * per_sm;
    if (x3) {
        RP_LAUNCH(c, k_update_rows_tc<true>, grid, TC_THREADS + 32, smem, c->ctl, p);
    } else {
        RP_LAUNCH(c, k_update_rows_tc<false>, grid, TC_THREADS + 32, smem, c->ctl, p);
    }
}

void tc_prepare() {
    const int max_smem = 2 * 2 * (TC_A_BYTES + 256 * 128) + 1024;
    cudaFuncSetAttribute(k_update_rows_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    cudaFuncSetAttribute(k_update_rows_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

// Transposed, K-contiguous, tf32-split copy of a row-major K x ldw weight block.
cudaError_t tc_weights_build(TcW* out, const float* W, int K, int ldw) {
    out->k_pad = (K + TC_KC - 1) / TC_KC * TC_KC;
    out->n_pad = (ldw + 15) / 16 * 16;
    if (K <= 0 || out->n_pad > 256) { out->hi = out->lo = nullptr; return cudaSuccess; }
    const size_t cnt = (size_t)out->k_pad * out->n_pad;
    std::vector<float> hi(cnt, 0.f), lo(cnt, 0.f);
    for (int k = 0; k < K; ++k)
        for (int j = 0; j < ldw; ++j) {
            float x = W[(size_t)k * ldw + j];
            uint32_t bits;
            memcpy(&bits, &x, 4);
            bits &= 0xffffe000u;
            float h;
            memcpy(&h, &bits, 4);
            hi[(size_t)j * out->k_pad + k] = h;
            lo[(size_t)j * out->k_pad + k] = x - h;
        }
    cudaError_t e = cudaMalloc(&out->hi, sizeof(float) * cnt);
    if (!e) e = cudaMalloc(&out->lo, sizeof(float) * cnt);
    if (!e) e = cudaMemcpy(out->hi, hi.data(), sizeof(float) * cnt, cudaMemcpyHostToDevice);
    if (!e) e = cudaMemcpy(out->lo, lo.data(), sizeof(float) * cnt, cudaMemcpyHostToDevice);
    return e;
}

}  // namespace rp
