// Tensor-core form of the affected-row layer update for sm_100a: tcgen05.mma (kind::tf32) with
// the accumulator tile in tensor memory.
//
// One persistent CTA per SM takes tiles of 128 affected rows x all (<= 256) output columns, in
// passes of at most 128 columns.  Per 32-float K chunk the loader warps gather the A rows by vertex
// id (applying the sink normalisation or the GIN self factor on the way), split every fp32 value x
// into hi = x with the 13 low mantissa bits cleared (exactly representable in tf32) and lo = x - hi,
// and store both into shared memory in the K-major 128-byte-swizzle layout the tensor core reads;
// the transposed weights arrive pre-split the same way (cp.async from L2, two steps ahead).  One
// elected thread issues hi*hi + lo*hi + hi*lo (three MMAs per 8-float K step), which reproduces
// the fp32 product to about 2^-21 relative, and commits to an mbarrier so that the stage can be
// refilled.  With tc_mode = TC_TF32 only hi*hi is issued (plain TF32, 2^-11).  Accumulators are
// double-buffered in tensor memory; eight epilogue warps read a finished tile back with tcgen05.ld
// and run the same fused bias / activation / delta / commit code as the SIMT form while the next
// tile's main loop is already running.
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

// true once the phase with the given parity has completed; gives up after `limit` polls
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < limit; ++it) {
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

// barrier among the loader warps only (the other roles never join it)
__device__ __forceinline__ void loaders_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TC_THREADS) : "memory"); }

// the same barrier, returning whether any loader thread passed a non-zero flag: a decision every
// loader thread takes alike (a thread that left the loop alone would strand the others here)
__device__ __forceinline__ bool loaders_sync_any(int flag) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out) : "r"(flag), "n"(TC_THREADS) : "memory");
    return out != 0;
}

// warp-uniform view of the failure flag
__device__ __forceinline__ bool warp_failed(volatile int* flag) { return __any_sync(0xffffffffu, *flag != 0); }

constexpr int TC_STAGES = 2;
constexpr int TC_NH = 256;                 // output columns per MMA pass (all of them: n_pad <= 256)
constexpr int TC_EPI_WARPS = 8;             // two per tensor-memory lane quarter, alternating column slabs
constexpr int TC_ALL_THREADS = TC_THREADS + 32 + 32 * TC_EPI_WARPS;
constexpr int TC_SLAB = 16;                // columns per epilogue step
constexpr int TC_SLAB_LD = TC_SLAB + 4;    // 20 floats: 16-byte stores of 8 consecutive rows fall on distinct banks

// Warp roles.  Warps 0..7 ("loaders") stage the operands, warp 8 issues the MMAs, warps 9..16 run
// the epilogue.  Every K chunk of a tile (128 rows x all output columns) is one step and takes one
// of two operand stages; the step counter runs on across tiles, so the loads of the next tile
// start while the last MMAs of this one are still in flight.
// Accumulators are double-buffered in tensor memory: the epilogue of tile t overlaps the main
// loop of tile t + 1.  Barriers (all waits bounded):
//   full[s]        8 arrivals (one per loader warp, after its stores and proxy fence) -> MMA warp may read
//   empty[s]       tcgen05.commit of the MMAs that read stage s                      -> loaders may refill
//   acc_full[b]    tcgen05.commit after the last MMA of a tile into buffer b         -> epilogue may read
//   acc_empty[b]   8 arrivals (one per epilogue warp, accumulators read)             -> MMA warp may overwrite
// Weights of step g + 1 are requested (cp.async from L2) as soon as step g has been handed over;
// the gathered A rows are prefetched one step ahead in registers.
template <bool X3>
__global__ void __launch_bounds__(TC_ALL_THREADS, 1)
k_update_rows_tc(Ctl* ctl, UpdParams p) {
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[TC_STAGES], empty[TC_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int row_id[2][TC_M];
    __shared__ float row_scale[2][TC_M];
    __shared__ volatile int s_fail;

    if (ctl->abort) return;
    const int n = upd_rows(p);
    if (!upd_use_tc(p, n)) return;
    const int row_tiles = (n + TC_M - 1) / TC_M;
    if ((int)blockIdx.x >= row_tiles) return;   // before any allocation

    // the diagnostic that withholds a completion also shortens the waits, so that they run out in milliseconds
    const uint32_t spin_limit = p.tc_withhold ? (1u << 16) : TC_SPIN_LIMIT;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_loader = warp < TC_THREADS / 32;
    const bool is_mma_warp = warp == TC_THREADS / 32;
    const int n_pad = p.n_pad;
    const int n_pass = (n_pad + TC_NH - 1) / TC_NH;
    constexpr uint32_t B_BYTES = TC_NH * 128u;
    constexpr uint32_t STAGE_BYTES = (X3 ? 2u : 1u) * (TC_A_BYTES + B_BYTES);
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* slabs = reinterpret_cast<float*>(smem + TC_STAGES * STAGE_BYTES);   // one 32-row slab per epilogue warp
    uint32_t buf_cols = 32;
    while ((int)buf_cols < n_pad) buf_cols <<= 1;
    const uint32_t tmem_cols = 2 * buf_cols;

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(&full[s], TC_THREADS / 32); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], TC_EPI_WARPS); }
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

    const int nchunks = p.k_pad / TC_KC;
    const int steps_per_tile = n_pass * nchunks;
    const int my_tiles = (row_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int total_steps = my_tiles * steps_per_tile;

    if (is_mma_warp) {
        // ---------------- MMA issue ----------------
        int g = 0;
        bool failed = false;
        for (int lt = 0; lt < my_tiles && !failed; ++lt) {
            const int b = lt & 1, ub = lt >> 1;
            // the epilogue must have drained this accumulator buffer (tile lt - 2)
            if (lane == 0 && ub > 0 && !mbar_wait_bounded(&acc_empty[b], (ub - 1) & 1, spin_limit)) s_fail = 1;
            __syncwarp();
            if ((failed = warp_failed(&s_fail))) break;
            tc_fence_after();
            for (int ps = 0; ps < n_pass && !failed; ++ps) {
                const int ncol = min(TC_NH, n_pad - ps * TC_NH);
                // instruction descriptor: fp32 accumulate, tf32 x tf32, both K-major, N = ncol, M = 128
                const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ncol >> 3) << 17) |
                                       ((uint32_t)(TC_M >> 4) << 24);
                const uint32_t d_addr = tmem_base + (uint32_t)b * buf_cols + (uint32_t)(ps * TC_NH);
                for (int kc = 0; kc < nchunks; ++kc, ++g) {
                    const int s = g % TC_STAGES;
                    const uint32_t u = (uint32_t)(g / TC_STAGES);
                    uint8_t* a_hi = smem + (size_t)s * STAGE_BYTES;
                    uint8_t* a_lo = a_hi + TC_A_BYTES;
                    uint8_t* b_hi = a_hi + (X3 ? 2 : 1) * TC_A_BYTES;
                    uint8_t* b_lo = b_hi + B_BYTES;
                    if (lane == 0) {
                        if (!mbar_wait_bounded(&full[s], u & 1, spin_limit)) s_fail = 1;
                        if (!s_fail) {
                            tc_fence_after();
                            const uint64_t da_hi = tc_smem_desc(smem_u32(a_hi)), db_hi = tc_smem_desc(smem_u32(b_hi));
                            const uint64_t da_lo = tc_smem_desc(smem_u32(a_lo)), db_lo = tc_smem_desc(smem_u32(b_lo));
#pragma unroll
                            for (int j = 0; j < TC_KC / 8; ++j) {     // one MMA K step = 8 floats = 32 bytes
                                const uint64_t adv = (uint64_t)((j * 32) >> 4);
                                tc_mma_tf32(d_addr, da_hi + adv, db_hi + adv, idesc, (kc | j) != 0);
                                if (X3) {
                                    tc_mma_tf32(d_addr, da_lo + adv, db_hi + adv, idesc, 1u);
                                    tc_mma_tf32(d_addr, da_hi + adv, db_lo + adv, idesc, 1u);
                                }
                            }
                            tc_commit(&empty[s]);
                            // (diagnostic: with tc_withhold the first tile is never reported finished, so that
                            // the epilogue's bounded wait runs out and the status path can be exercised)
                            if (ps == n_pass - 1 && kc == nchunks - 1 && !(p.tc_withhold && lt == 0)) tc_commit(&acc_full[b]);
                        }
                    }
                    __syncwarp();
                    if ((failed = warp_failed(&s_fail))) break;
                }
            }
        }
    } else if (is_loader) {
        // ---------------- operand staging ----------------
        constexpr int A_ITERS = (TC_M * 8) / TC_THREADS;
        constexpr int B_ITERS = (TC_NH * 8) / TC_THREADS;
        auto write_ids = [&](int lt) {   // vertex ids and sink scales of local tile lt, buffer lt & 1
            if (tid < TC_M) {
                const int i = ((int)blockIdx.x + lt * (int)gridDim.x) * TC_M + tid;
                int v = -1;
                float sc = 0.f;
                if (lt < my_tiles && i < n) {
                    v = p.list ? p.list[i] : i;
                    sc = upd_row_scale(p, v);
                }
                row_id[lt & 1][tid] = v;
                row_scale[lt & 1][tid] = sc;
            }
        };
        float4 ax[A_ITERS], ax_next[A_ITERS];
        auto load_a = [&](int g, float4 (&dst)[A_ITERS]) {   // 128 rows x 8 pieces of 16 bytes, by vertex id
            const int lt = g / steps_per_tile, kc = (g - lt * steps_per_tile) % nchunks, b = lt & 1;
            const int r0 = ((int)blockIdx.x + lt * (int)gridDim.x) * TC_M;
#pragma unroll
            for (int it = 0; it < A_ITERS; ++it) {
                const int idx = tid + it * TC_THREADS, r = idx >> 3, c = idx & 7;
                const int v = row_id[b][r], k = kc * TC_KC + c * 4;
                dst[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (v >= 0 && k < p.K) dst[it] = upd_load_a(p, v, r0 + r, k, row_scale[b][r]);
            }
        };
        // asynchronous copy of step g's pre-split transposed weights (<= 128 output columns x 8 pieces
        // of 16 bytes, hi and lo) from L2 straight into their swizzled places in stage g % TC_STAGES; the MMAs
        // that last read that stage must have finished.  Always closes one copy group.
        auto copy_b = [&](int g) {
            if (g < total_steps) {
                const int s = g % TC_STAGES;
                const uint32_t u = (uint32_t)(g / TC_STAGES);
                if (u > 0 && !s_fail && !mbar_wait_bounded(&empty[s], (u - 1) & 1, spin_limit)) s_fail = 1;
                const int r = g % steps_per_tile, ps = r / nchunks, kc = r - ps * nchunks;
                const int ncol = min(TC_NH, n_pad - ps * TC_NH);
                uint8_t* b_hi = smem + (size_t)s * STAGE_BYTES + (X3 ? 2 : 1) * TC_A_BYTES;
                uint8_t* b_lo = b_hi + B_BYTES;
#pragma unroll
                for (int it = 0; it < B_ITERS; ++it) {
                    const int idx = tid + it * TC_THREADS;
                    if (idx < ncol * 8) {
                        const size_t go = (size_t)(ps * TC_NH + (idx >> 3)) * p.k_pad + kc * TC_KC + (idx & 7) * 4;
                        const uint32_t off = tc_swz(idx >> 3, idx & 7);
                        cp_async16(smem_u32(b_hi + off), p.Wt_hi + go);
                        if (X3) cp_async16(smem_u32(b_lo + off), p.Wt_lo + go);
                    }
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        write_ids(0);
        write_ids(1);
        loaders_sync();
        load_a(0, ax);
        copy_b(0);
        for (int g = 0; g < total_steps; ++g) {
            const int s = g % TC_STAGES;
            const int lt = g / steps_per_tile;
            if (lt >= 1 && g == lt * steps_per_tile) {
                // ids of the tile after this one; their buffer last served tile lt - 1, fully staged by now
                write_ids(lt + 1);
                if (loaders_sync_any(s_fail)) break;   // the only place the loaders leave early, all together
            }
            uint8_t* a_hi = smem + (size_t)s * STAGE_BYTES;
            uint8_t* a_lo = a_hi + TC_A_BYTES;                              // only if X3
            // next step's row gathers first (registers), so that they have a whole step to land
            if (g + 1 < total_steps) load_a(g + 1, ax_next);
#pragma unroll
            for (int it = 0; it < A_ITERS; ++it) {
                const int idx = tid + it * TC_THREADS;
                const uint32_t off = tc_swz(idx >> 3, idx & 7);
                const float4 x = ax[it];
                const float4 h = make_float4(tf32_hi(x.x), tf32_hi(x.y), tf32_hi(x.z), tf32_hi(x.w));
                *reinterpret_cast<float4*>(a_hi + off) = h;
                if (X3) *reinterpret_cast<float4*>(a_lo + off) = make_float4(x.x - h.x, x.y - h.y, x.z - h.z, x.w - h.w);
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");   // this step's weights have landed
            fence_async_smem();   // generic-proxy stores -> visible to the tensor core's async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&full[s]);
            copy_b(g + 1);   // travels while the next step's rows are split and stored
#pragma unroll
            for (int it = 0; it < A_ITERS; ++it) ax[it] = ax_next[it];
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else {
        // ---------------- epilogue ----------------
        // A warp's index modulo 4 fixes the tensor-memory lanes it may read: rows 32 q .. 32 q + 31 of the
        // tile, shared by two warps that take alternate 16-column slabs.  Per slab every lane pulls
        // its own row's 16 accumulators, the warp turns them through a small shared-memory slab, and
        // then each pass handles 8 rows x 64 bytes, so that the previous row, the cached projection,
        // the delta row and the new row move in whole sectors; the loads of all 4 passes are issued
        // before the first is used.
        const int q = warp & 3;
        const int ew = warp - (TC_THREADS / 32 + 1);     // 0..7
        const int parity = ew >> 2;                      // which of the quarter's two warps: even or odd slabs
        float* slab = slabs + (size_t)ew * 32 * TC_SLAB_LD;
        const bool need_old = upd_needs_old(p);
        const bool need_z = p.addend2 != nullptr;
        const int sub_r = lane >> 2, sub_c = 4 * (lane & 3);   // 8 rows x 64 bytes per pass
        for (int lt = 0; lt < my_tiles; ++lt) {
            const int b = lt & 1, ub = lt >> 1;
            const int r0 = ((int)blockIdx.x + lt * (int)gridDim.x) * TC_M + 32 * q;
            int v_own = -1;
            float sc_own = 0.f;
            if (r0 + lane < n) {
                v_own = p.list ? p.list[r0 + lane] : r0 + lane;
                sc_own = upd_row_scale(p, v_own);
            }
            if (lane == 0 && !mbar_wait_bounded(&acc_full[b], ub & 1, spin_limit)) s_fail = 1;
            __syncwarp();
            if (warp_failed(&s_fail)) break;
            tc_fence_after();
            for (int c0 = parity * TC_SLAB; c0 < p.n_cols; c0 += 2 * TC_SLAB) {
                uint32_t x[16];
                const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)b * buf_cols + (uint32_t)c0;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                    : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]),
                      "=r"(x[7]), "=r"(x[8]), "=r"(x[9]), "=r"(x[10]), "=r"(x[11]), "=r"(x[12]), "=r"(x[13]),
                      "=r"(x[14]), "=r"(x[15])
                    : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                float4* mine = reinterpret_cast<float4*>(slab + (size_t)lane * TC_SLAB_LD);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    mine[j] = make_float4(__uint_as_float(x[4 * j]), __uint_as_float(x[4 * j + 1]),
                                          __uint_as_float(x[4 * j + 2]), __uint_as_float(x[4 * j + 3]));
                __syncwarp();
                const int col = c0 + sub_c;
                int vv[4];
                float ss[4];
                float4 oldv[4], zv[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int rr = 8 * t + sub_r;
                    vv[t] = __shfl_sync(FULL, v_own, rr);
                    ss[t] = __shfl_sync(FULL, sc_own, rr);
                    if (vv[t] >= 0 && col < p.n_cols) {
                        if (need_old) oldv[t] = upd_load_old(p, vv[t], col);
                        if (need_z) zv[t] = *reinterpret_cast<const float4*>(p.addend2 + (size_t)vv[t] * p.ld_add + col);
                    }
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int rr = 8 * t + sub_r;
                    if (vv[t] >= 0 && col < p.n_cols) {
                        const float4 acc = *reinterpret_cast<const float4*>(slab + (size_t)rr * TC_SLAB_LD + sub_c);
                        upd_epilogue4(p, vv[t], r0 + rr, col, acc, ss[t], need_old, oldv[t], need_z, zv[t]);
                    }
                }
                __syncwarp();   // the slab is rewritten by the next step
            }
            tc_fence_before();   // accumulators consumed: the MMA warp may overwrite them after this arrival
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[b]);
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

static size_t tc_smem_bytes(bool x3) {
    const size_t stage = (size_t)(x3 ? 2 : 1) * (TC_A_BYTES + (size_t)TC_NH * 128);
    return TC_STAGES * stage + (size_t)TC_EPI_WARPS * 32 * TC_SLAB_LD * sizeof(float) + 1024;
}

void launch_update_tc(Ctx* c, const UpdParams& p) {
    const bool x3 = p.tc_mode == TC_TF32X3;
    // one persistent CTA per SM: the operand stages and the epilogue slabs fill its shared memory
    const int grid = c->n_sm;
    if (x3) {
        RP_LAUNCH(c, k_update_rows_tc<true>, grid, TC_ALL_THREADS, tc_smem_bytes(true), c->ctl, p);
    } else {
        RP_LAUNCH(c, k_update_rows_tc<false>, grid, TC_ALL_THREADS, tc_smem_bytes(false), c->ctl, p);
    }
}

void tc_prepare() {
    cudaFuncSetAttribute(k_update_rows_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(true));
    cudaFuncSetAttribute(k_update_rows_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(false));
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
