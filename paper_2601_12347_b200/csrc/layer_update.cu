// Affected-row layer update (Compute + Prepare of Sec. 3.3.1): gather the inputs of Update^l for the
// rows of A_l, multiply by the layer weights, add bias, apply the activation, write h^l_v in
// place and emit the delta row D_v = c_new h_new - c_old h_old for the next hop (Sec. 3.3.3).
//
// Two forms of the same contraction, chosen on the device from the row count:
//   SIMT fp32    register-tiled GEMM whose A operand is gathered by row id (this file); used
//                while the affected set is too small to be a real dense contraction;
//   tensor core  tcgen05 TF32 with a 3-term split that keeps fp32 accuracy (layer_update_tc.cu).
#include "layer_update.cuh"

#include <algorithm>

namespace rp {

// K is walked in chunks of 64: every thread has eight independent 16-byte loads in flight per chunk
// (four pieces of a gathered A row, four of the weights).  With chunks of 16 a small frontier -- a
// handful of tiles, so nothing to overlap with -- paid one trip to L2 per 16 columns of K: 20 to 27 us
// for a few dozen rows, half of the latency of a batch of one update.
constexpr int BM = 64, BN = 64, BK = 64, TM = 4, TN = 4;

// A frontier of a few rows (a batch of a few updates at the first hops) is nothing but latency: the tiled form
// walks K in chunks, each a round trip to L2 behind the last.  For up to FEW_MAX rows and K up to FEW_K the same
// kernel takes another route: a block owns FEW_ROWS rows and 32 output columns, stages its A rows in shared
// memory once, its eight warps each take an eighth of K with every weight load independent of the others (one
// round trip in all), the partial sums meet in shared memory and the ordinary epilogue finishes the rows.
constexpr int FEW_ROWS = 16, FEW_K = 256, FEW_COLS = 32, FEW_MAX = 256;

__device__ __forceinline__ bool upd_few(const UpdParams& p, int n) {
    return n > 0 && n <= FEW_MAX && p.K > 0 && p.K <= FEW_K;
}

__device__ __forceinline__ void update_few_rows(const UpdParams& p, int n_all, float* A_s, float* red, int* row_id,
                                                float* row_scale) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kq = p.K >> 2;
    const int groups = (p.n_cols + FEW_COLS - 1) / FEW_COLS, row_groups = (n_all + FEW_ROWS - 1) / FEW_ROWS;
    for (int item = blockIdx.x; item < groups * row_groups; item += gridDim.x) {
        const int g = item % groups, r0 = (item / groups) * FEW_ROWS;
        const int n = min(FEW_ROWS, n_all - r0);   // rows of this block: compact indices r0 .. r0 + n - 1
        __syncthreads();
        if (tid < n) {
            const int v = p.list ? p.list[r0 + tid] : r0 + tid;
            row_id[tid] = v;
            row_scale[tid] = upd_row_scale(p, v);
        }
        __syncthreads();
        for (int it = tid; it < n * kq; it += blockDim.x) {
            const int r = it / kq, k = 4 * (it - r * kq);
            *reinterpret_cast<float4*>(A_s + r * FEW_K + k) = upd_load_a(p, row_id[r], r0 + r, k, row_scale[r]);
        }
        __syncthreads();
        const int c = g * FEW_COLS + lane;
        const int kper = (p.K + 7) >> 3, k_begin = warp * kper, k_end = min(p.K, k_begin + kper);
        float acc[FEW_ROWS];
#pragma unroll
        for (int r = 0; r < FEW_ROWS; ++r) acc[r] = 0.f;
#pragma unroll 8
        for (int k = k_begin; k < k_end; ++k) {
            const float wv = c < p.n_cols ? __ldg(p.W + (size_t)k * p.ldw + c) : 0.f;
#pragma unroll
            for (int r = 0; r < FEW_ROWS; ++r)
                if (r < n) acc[r] = fmaf(A_s[r * FEW_K + k], wv, acc[r]);
        }
#pragma unroll
        for (int r = 0; r < FEW_ROWS; ++r) red[(warp * FEW_ROWS + r) * FEW_COLS + lane] = acc[r];
        __syncthreads();
        if (tid < n * (FEW_COLS / 4)) {
            const int r = tid / (FEW_COLS / 4), q = tid - r * (FEW_COLS / 4), col = g * FEW_COLS + 4 * q;
            if (col < p.n_cols) {
                float4 h = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int w = 0; w < 8; ++w) {
                    const float4 x = *reinterpret_cast<const float4*>(red + (w * FEW_ROWS + r) * FEW_COLS + 4 * q);
                    h.x += x.x; h.y += x.y; h.z += x.z; h.w += x.w;
                }
                upd_epilogue4(p, row_id[r], r0 + r, col, h, row_scale[r]);
            }
        }
    }
}

// FEW: the instantiation that small batches launch also holds the few-row form.  Large batches launch the one
// without it: with the few-row code inlined beside it the tiled form, unchanged in registers and shared memory,
// made a batch of 1000 updates on the dense graph 0.3 ms slower (1.65 -> 2.0 ms) once the kernels of the chain
// overlap their launches, and calling the few-row form out of line cost the small batches 10 us of the 30 it saves.
template <bool FEW>
__global__ void __launch_bounds__(256)
k_update_rows(const Ctl* ctl, UpdParams p) {
    pdl_enter();
    if (ctl->abort) return;
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN];
    __shared__ int row_id[BM];
    __shared__ float row_scale[BM];
    const int n = upd_rows(p);
    if (upd_use_tc(p, n) || upd_use_narrow(p, n)) return;
    if (FEW && upd_few(p, n)) {
        static_assert(sizeof(As) >= sizeof(float) * FEW_ROWS * FEW_K && sizeof(Bs) >= sizeof(float) * 8 * FEW_ROWS * FEW_COLS,
                      "the few-row form borrows the tiles' shared memory");
        update_few_rows(p, n, &As[0][0], &Bs[0][0], row_id, row_scale);
        return;
    }
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
                sc = upd_row_scale(p, v);
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

        const int ar = tid >> 2, ak = (tid & 3) * 4;   // A tile: row ar, k offsets ak + 16 j .. + 3, j = 0..3
        const int bk = tid >> 4, bn = (tid & 15) * 4;  // B tile: k rows bk + 16 j, cols bn..bn+3
        for (int k0 = 0; k0 < p.K; k0 += BK) {
            float4 a[4], b[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int v = row_id[ar], k = k0 + ak + 16 * j;
                if (v >= 0 && k < p.K) a[j] = upd_load_a(p, v, r0 + ar, k, row_scale[ar]);
                b[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int kb = k0 + bk + 16 * j;
                if (kb < p.K && c0 + bn < p.n_cols)
                    b[j] = __ldg(reinterpret_cast<const float4*>(p.W + (size_t)kb * p.ldw + c0 + bn));
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                As[ak + 16 * j + 0][ar] = a[j].x; As[ak + 16 * j + 1][ar] = a[j].y;
                As[ak + 16 * j + 2][ar] = a[j].z; As[ak + 16 * j + 3][ar] = a[j].w;
                *reinterpret_cast<float4*>(&Bs[bk + 16 * j][bn]) = b[j];
            }
            __syncthreads();
            const int kmax = min(BK, p.K - k0);
#pragma unroll 16
            for (int k = 0; k < kmax; ++k) {
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
        const int col = c0 + tx * TN;
        if (col < p.n_cols) {
#pragma unroll
            for (int a2 = 0; a2 < TM; ++a2) {
                const int lr = ty * TM + a2, v = row_id[lr];
                if (v < 0) continue;
                upd_epilogue4(p, v, r0 + lr, col, make_float4(acc[a2][0], acc[a2][1], acc[a2][2], acc[a2][3]),
                              row_scale[lr]);
            }
        }
    }
}

// Outputs of at most 48 columns over many rows (the last layers of the configurations: 47 and 40 classes, as the
// neighbour and the self projection of a million senders): the 64 x 64 tile above leaves a quarter of its threads
// multiplying zero columns, and it waits for every chunk of K before it multiplies it.  Here a tile is 256 rows x 48
// columns.  The gathered rows arrive through a ring of NST stages filled by cp.async, 16 entries of K per stage and
// row, NST - 1 chunks ahead of the one being multiplied and without passing through registers.  A warp owns six
// columns (its loads of the weights are uniform: one broadcast), a lane the eight rows ty, ty + 32, ...; it reads
// four entries of K per row with one 16-byte load (rows are 20 floats apart in a stage, so the loads of eight
// consecutive lanes fall into eight different 16-byte bank groups).  The factor on the A operand is per row: it is
// applied to the finished sums.  The finished tile goes through shared memory once more so that the epilogue sees
// 16-byte pieces of rows.  One source per A entry: the operand alpha h + scale S of GIN layers stays with the tiled form.
constexpr int NBM = 256, NBN = 48, NBK = 16, NTM = 8, NTN = 6, NST = 4, NARROW_MIN_ROWS = 65536;
constexpr int NAS_LD = NBK + 4, NCS_LD = NBN + 4;
constexpr size_t NARROW_SMEM = sizeof(float) * ((size_t)NST * NBM * NAS_LD + 2 * NBK * NBN + 2 * NBM) + sizeof(int) * NBM;
static_assert(NST * NBM * NAS_LD >= (NBM / 2) * NCS_LD, "the finished half tile is staged in the ring");

__device__ __forceinline__ void cp_async16_zfill(float* smem_dst, const float* gptr, bool valid) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int bytes = valid ? 16 : 0;      // (0: sixteen zero bytes are written, nothing is read)
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gptr), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(256, 2)
k_update_rows_narrow(const Ctl* ctl, UpdParams p) {
    pdl_enter();
    if (ctl->abort) return;
    extern __shared__ __align__(16) float nsm[];
    float* ring = nsm;                                   // [NST][NBM][NAS_LD], later the finished tile, half at a time
    float* Bs = ring + (size_t)NST * NBM * NAS_LD;       // [2][NBK][NBN]
    float* row_scale = Bs + 2 * NBK * NBN;               // [NBM]
    float* row_fac = row_scale + NBM;                    // [NBM]
    int* row_id = reinterpret_cast<int*>(row_fac + NBM); // [NBM]
    const int n = upd_rows(p);
    if (!upd_use_narrow(p, n)) return;
    const int row_tiles = (n + NBM - 1) / NBM, chunks = (p.K + NBK - 1) / NBK;
    const int tid = threadIdx.x, tx = tid >> 5, ty = tid & 31;
    for (int rt = blockIdx.x; rt < row_tiles; rt += gridDim.x) {
        const int r0 = rt * NBM;
        __syncthreads();
        {
            const int i = r0 + tid;
            int v = -1;
            float sc = 0.f;
            if (i < n) {
                v = p.list ? p.list[i] : i;
                sc = upd_row_scale(p, v);
            }
            row_id[tid] = v;
            row_scale[tid] = sc;
            row_fac[tid] = p.a_mode == A_DENSE ? 1.0f : p.a_mode == A_SELF ? p.alpha : sc;
        }
        __syncthreads();
        float acc[NTM][NTN];
#pragma unroll
        for (int a2 = 0; a2 < NTM; ++a2)
#pragma unroll
            for (int b2 = 0; b2 < NTN; ++b2) acc[a2][b2] = 0.f;
        // this thread's part of a chunk of A: rows ar + 64 s, entries ak .. ak + 3 of the chunk
        const int ar = tid >> 2, ak = (tid & 3) * 4;
        const float* src[4];
#pragma unroll
        for (int s2 = 0; s2 < 4; ++s2) {
            const int r = ar + 64 * s2, v = row_id[r];
            src[s2] = nullptr;
            if (v >= 0) {
                if (p.a_mode == A_DENSE) src[s2] = p.Hprev + (size_t)(r0 + r) * p.ld_h;
                else if (p.a_mode == A_SELF) src[s2] = p.Hprev + (size_t)v * p.ld_h;
                else src[s2] = p.S + (size_t)v * p.ld_s;
            }
        }
        auto request = [&](int c) {      // chunk c of A into its stage (beyond K: an empty group keeps the count)
            if (c < chunks) {
                float* stage = ring + (size_t)(c % NST) * NBM * NAS_LD;
                const int k = c * NBK + ak;
#pragma unroll
                for (int s2 = 0; s2 < 4; ++s2) {
                    const bool ok = src[s2] && k < p.K;
                    cp_async16_zfill(stage + (ar + 64 * s2) * NAS_LD + ak, ok ? src[s2] + k : p.W, ok);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        // this thread's piece of a chunk of the weights (192 threads): row bk of the chunk, columns 4 bq .. 4 bq + 3
        const int bk = tid / (NBN / 4), bq = tid - bk * (NBN / 4);
        auto load_b = [&](int c) {
            float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
            if (bk < NBK && c * NBK + bk < p.K && 4 * bq < p.n_cols)
                b = __ldg(reinterpret_cast<const float4*>(p.W + (size_t)(c * NBK + bk) * p.ldw + 4 * bq));
            return b;
        };
#pragma unroll
        for (int c = 0; c < NST - 1; ++c) request(c);
        float4 b = load_b(0);
        for (int c = 0; c < chunks; ++c) {
            float* Bc = Bs + (c & 1) * NBK * NBN;
            if (bk < NBK) *reinterpret_cast<float4*>(Bc + bk * NBN + 4 * bq) = b;
            asm volatile("cp.async.wait_group %0;" ::"n"(NST - 2) : "memory");   // this thread's pieces of chunk c are in
            __syncthreads();                  // everyone's are, the weights too; and chunk c - 1 has been multiplied
            request(c + NST - 1);             // into the stage that chunk c - 1 has left
            b = load_b(c + 1);
            const float* stage = ring + (size_t)(c % NST) * NBM * NAS_LD;
            const int kmax = min(NBK, p.K - c * NBK);      // a multiple of four
            for (int k = 0; k < kmax; k += 4) {
                float4 av[NTM];
#pragma unroll
                for (int a2 = 0; a2 < NTM; ++a2)
                    av[a2] = *reinterpret_cast<const float4*>(stage + (a2 * 32 + ty) * NAS_LD + k);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const float2 w0 = *reinterpret_cast<const float2*>(Bc + (k + kk) * NBN + tx * NTN);
                    const float2 w1 = *reinterpret_cast<const float2*>(Bc + (k + kk) * NBN + tx * NTN + 2);
                    const float2 w2 = *reinterpret_cast<const float2*>(Bc + (k + kk) * NBN + tx * NTN + 4);
                    const float bv[NTN] = {w0.x, w0.y, w1.x, w1.y, w2.x, w2.y};
#pragma unroll
                    for (int a2 = 0; a2 < NTM; ++a2) {
                        const float x = kk == 0 ? av[a2].x : kk == 1 ? av[a2].y : kk == 2 ? av[a2].z : av[a2].w;
#pragma unroll
                        for (int b2 = 0; b2 < NTN; ++b2) acc[a2][b2] = fmaf(x, bv[b2], acc[a2][b2]);
                    }
                }
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        // the finished tile, 128 rows at a time, through shared memory to the epilogue
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            __syncthreads();
#pragma unroll
            for (int a2 = 0; a2 < NTM / 2; ++a2) {
                const int r = (half * (NTM / 2) + a2) * 32 + ty;
                const float f = row_fac[r];
#pragma unroll
                for (int b2 = 0; b2 < NTN; ++b2)
                    ring[(a2 * 32 + ty) * NCS_LD + tx * NTN + b2] = f * acc[half * (NTM / 2) + a2][b2];
            }
            __syncthreads();
            for (int it = tid; it < (NBM / 2) * (NBN / 4); it += 256) {
                const int lr = it / (NBN / 4), q = it - lr * (NBN / 4);
                const int r = half * (NBM / 2) + lr, v = row_id[r];
                if (v < 0 || 4 * q >= p.n_cols) continue;
                const float4 h = *reinterpret_cast<const float4*>(&ring[lr * NCS_LD + 4 * q]);
                upd_epilogue4(p, v, r0 + r, 4 * q, h, row_scale[r]);
            }
        }
    }
}

void narrow_prepare() {
    cudaFuncSetAttribute(k_update_rows_narrow, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)NARROW_SMEM);
}

// K = 0: the layer's self projection and transformed aggregate are both cached, so the update is
// elementwise (bias + cached terms + activation); one thread per 16-byte piece of a row
__global__ void __launch_bounds__(256)
k_update_rows_elementwise(const Ctl* ctl, UpdParams p) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = upd_rows(p), nq = p.n_cols >> 2;
    const long long total = (long long)n * nq;
    for (long long it = blockIdx.x * (long long)blockDim.x + threadIdx.x; it < total;
         it += (long long)gridDim.x * blockDim.x) {
        const int i = (int)(it / nq), q = (int)(it - (long long)i * nq);
        const int v = p.list ? p.list[i] : i;
        upd_epilogue4(p, v, i, 4 * q, make_float4(0.f, 0.f, 0.f, 0.f), upd_row_scale(p, v));
    }
}

// launches both forms; exactly one of them does the work (decided on the device)
static void launch_update(Ctx* c, UpdParams& p, const TcW& tw) {
    p.tc_mode = TC_OFF;
    // measured on the dense graph: the tensor-core form wins for wide outputs (256 columns: 5.5 ms
    // against 9.8 ms SIMT) and loses for narrow ones, where staging latency dominates
    // The tensor-core twin is only put into the chain when the last batch's frontiers (or a whole-graph pass)
    // were large enough for it; without it the SIMT form takes whatever comes.
    if (tw.hi && c->gemm_mode != RIPPLE_GEMM_FP32 && p.K > 0 && tw.n_pad >= 128 && (c->tc_armed || !p.list)) {
        p.tc_mode = c->gemm_mode == RIPPLE_GEMM_TF32 ? TC_TF32 : TC_TF32X3;
        p.tc_min_rows = 1024;
        p.tc_withhold = c->debug_tc_withhold;
        p.Wt_hi = tw.hi; p.Wt_lo = tw.lo; p.k_pad = tw.k_pad; p.n_pad = tw.n_pad;
    }
    if (p.K == 0) {
        RP_LAUNCH(c, k_update_rows_elementwise, c->n_sm * 8, 256, 0, c->ctl, p);
        return;
    }
    // narrow outputs over many rows have a form of their own; in the chain under the same condition as the
    // tensor-core form (the last batch's frontiers, or a whole-graph pass, were large)
    p.narrow_min_rows = (p.n_cols <= NBN && p.a_mode != A_SUM && p.tc_mode == TC_OFF && (c->tc_armed || !p.list)) ? NARROW_MIN_ROWS : 0;
    if (c->few_rows_form && p.list) RP_LAUNCH(c, k_update_rows<true>, c->n_sm * 4, 256, 0, c->ctl, p);
    else RP_LAUNCH(c, k_update_rows<false>, c->n_sm * 4, 256, 0, c->ctl, p);
    if (p.narrow_min_rows) RP_LAUNCH(c, k_update_rows_narrow, c->n_sm * 2, 256, NARROW_SMEM, c->ctl, p);
    if (p.tc_mode != TC_OFF) launch_update_tc(c, p);
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
    launch_update(c, p, ly.tc_nbr);
}

// Layers that transform before the scatter keep P^l_u = W_n^T h^{l-1}_u for every vertex.  For the
// senders of hop l (rows whose h^{l-1}, or whose source coefficient, changed) this recomputes the
// row, commits it and emits the transformed delta message c_new P_new - c_old P_old as a compact
// row.  Because the next batch subtracts exactly the value cached here, the deltas of successive
// batches telescope: the aggregate tracks the cached rows without a rounding drift of its own.
void sender_transform(Ctx* c, int l) {
    const LayerDev& ly = c->layer[l];
    UpdParams p{};
    p.list = c->Clist[(l - 1) & 1]; p.n_dev = &c->ctl->nC[l - 1]; p.n_host = 0;
    p.a_mode = A_SELF; p.epi_mode = EPI_COMMIT; p.alpha = 1.0f;
    p.Hprev = c->H[l - 1]; p.ld_h = c->ld[l - 1];
    p.K = ly.ld_in;
    p.W = ly.kind == RIPPLE_LAYER_SAGE ? ly.W1 + (size_t)ly.ld_in * ly.ld_out : ly.W1;
    p.ldw = c->ws[l]; p.bias = nullptr; p.n_cols = c->ws[l];
    p.act = RIPPLE_ACT_IDENTITY; p.Hout = c->P[l]; p.ld_o = c->ws[l]; p.Dout = c->Dt;
    p.src_norm = c->src_norm; p.deg_out = c->side[0].deg; p.deg_out_old = c->deg_out_old;
    launch_update(c, p, ly.tc_nbr);
}

// Z^l_v = W_self^T h^{l-1}_v for the rows whose h^{l-1} changed (all rows at bootstrap).  SAGE
// layers keep this self projection cached: it is recomputed where the layer's input changed
// (A_{l-1}), not where its output is needed (A_l, usually far larger).  The affected-row update
// then contracts over the aggregate only (half the K of [h || x]); for a layer that also
// transforms before the scatter nothing is left to contract.
void self_project(Ctx* c, int l, bool full) {
    if (!c->Z[l]) return;
    const LayerDev& ly = c->layer[l];
    UpdParams p{};
    p.list = full ? nullptr : c->A[l - 1];
    p.n_dev = full ? nullptr : &c->ctl->nA[l - 1];
    p.n_host = c->N;
    p.a_mode = A_SELF; p.epi_mode = EPI_COMMIT; p.alpha = 1.0f;
    p.Hprev = c->H[l - 1]; p.ld_h = c->ld[l - 1];
    p.K = ly.ld_in; p.W = ly.W1; p.ldw = ly.ld_out; p.n_cols = ly.ld_out;
    p.act = RIPPLE_ACT_IDENTITY; p.Hout = c->Z[l]; p.ld_o = ly.ld_out;
    launch_update(c, p, ly.tc_self);
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
    if (pre) {
        p.addend = c->S[l]; p.ld_add = c->ws[l];
        if (!full && c->fused_fold[l]) { p.addend_rw = c->S[l]; p.addend_delta = c->dS[l]; }   // fold_deltas is skipped for these layers
    }
    float* dout = (full || l == c->L) ? nullptr : c->D[l & 1];  // the last hop sends nothing
    p.dout_old = rp_monotonic(c->agg);
    if (ly.kind == RIPPLE_LAYER_GIN) {
        // hidden = relu(W1^T ((1 + eps) h + x) + b1), kept as compact rows
        p.a_mode = pre ? A_SELF : A_SUM; p.epi_mode = EPI_TEMP; p.alpha = 1.0f + ly.eps;
        p.K = ly.ld_in; p.W = ly.W1; p.ldw = ly.ld_hid; p.bias = ly.b1; p.n_cols = ly.ld_hid;
        p.act = RIPPLE_ACT_RELU; p.Hout = c->T; p.ld_o = ly.ld_hid; p.Dout = nullptr;
        launch_update(c, p, ly.tc_main);
        p.a_mode = A_DENSE; p.epi_mode = EPI_COMMIT; p.addend = nullptr; p.addend_rw = nullptr; p.addend_delta = nullptr;
        p.Hprev = c->T; p.ld_h = ly.ld_hid;
        p.K = ly.ld_hid; p.W = ly.W2; p.ldw = ly.ld_out; p.bias = ly.b2; p.n_cols = ly.ld_out;
        p.act = ly.act; p.Hout = c->H[l]; p.ld_o = ly.ld_out; p.Dout = dout;
        launch_update(c, p, ly.tc_2);
        return;
    }
    p.epi_mode = EPI_COMMIT;
    if (ly.kind == RIPPLE_LAYER_SAGE) {
        p.a_mode = A_AGG;
        p.K = pre ? 0 : ly.ld_in;       // transformed aggregate: nothing left to multiply
        p.addend2 = c->Z[l];            // cached W_self^T h_v
    } else {
        p.a_mode = A_AGG;
        p.K = pre ? 0 : ly.ld_in;   // transformed inbox: nothing left to multiply
    }
    p.W = ly.kind == RIPPLE_LAYER_SAGE ? ly.W1 + (size_t)ly.ld_in * ly.ld_out : ly.W1;   // neighbour matrix
    p.ldw = ly.ld_out; p.bias = ly.b1; p.n_cols = ly.ld_out;
    p.act = ly.act; p.Hout = c->H[l]; p.ld_o = ly.ld_out; p.Dout = dout;
    if (!pre) p.ld_add = ly.ld_out;   // leading dimension of the cached projection
    launch_update(c, p, ly.tc_main);
}

// ---------------------------------------------------------------------------------------------
// hop 0: feature replacement rows and their deltas; one warp per vertex of A_0
// ---------------------------------------------------------------------------------------------
__global__ void k_feature_rows(Ctl* ctl, const ripple_update* __restrict__ ups, const float* __restrict__ feat,
                               int d0, const int32_t* __restrict__ A0, const int32_t* __restrict__ feat_last,
                               int src_norm, const int32_t* __restrict__ deg_out,
                               const int32_t* __restrict__ deg_out_old, float* H0, int ld, float* D, int keep_old) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->nA[0];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int i = warp; i < n; i += nwarps) {
        const int v = A0[i];
        const ripple_update last = ups[feat_last[v]];
        // the last word on the row is either a payload row or the vertex's deletion (zeros)
        const float* src = last.op == RIPPLE_OP_SET_FEATURE ? feat + (size_t)last.v * d0 : nullptr;
        float cn = 1.f, co = 1.f;
        if (src_norm) {
            cn = coef_deg(deg_out[v]);
            co = deg_out_old[v] >= 0 ? coef_deg(deg_out_old[v]) : cn;
        }
        for (int k = lane_id(); k < ld; k += 32) {
            float x = (src && k < d0) ? src[k] : 0.f;
            float o = H0[(size_t)v * ld + k];
            D[(size_t)i * ld + k] = keep_old ? o : cn * x - co * o;
            H0[(size_t)v * ld + k] = x;
        }
    }
}

void feature_rows(Ctx* c, int n) {
    if (n <= 0) return;
    RP_LAUNCH(c, k_feature_rows, std::min(div_up(n, 8), c->n_sm * 8), 256, 0, c->ctl, c->ups_dev, c->feat_dev,
              c->d[0], c->A[0], c->feat_last, (int)c->src_norm, c->side[0].deg, c->deg_out_old, c->H[0],
              c->ld[0], c->D[0], (int)(rp_monotonic(c->agg) || c->attention));
}

// ---------------------------------------------------------------------------------------------
// senders whose row did not change but whose source coefficient did: D_u = (c_new - c_old) h_u
// ---------------------------------------------------------------------------------------------
__global__ void k_extra_senders(Ctl* ctl, int l, const Rec* __restrict__ rec, int32_t* senders,
                                int32_t* posmap, const int32_t* __restrict__ deg_out,
                                const float* __restrict__ H, int ld, float* D) {
    pdl_enter();
    if (ctl->abort) return;
    const int n = ctl->n_rec;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int r = warp; r < n; r += nwarps) {
        const Rec x = rec[r];
        if (!x.rep[0] || x.silent) continue;   // one record per distinct source (a no-compute copy names a remote one)
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
