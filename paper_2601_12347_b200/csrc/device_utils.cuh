// Small device-side building blocks: warp/block scans, bit tricks, vector reductions to global.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace rp {

constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

// First statement of every kernel.  The kernels of a batch are launched with programmatic stream
// serialisation: a kernel may be scheduled while its predecessor is still running, so that launch
// latency overlaps execution (a batch is a chain of some fifty short kernels).  The wait returns
// once every prerequisite grid has completed and its memory operations are visible, so nothing a
// kernel reads can be stale; the trigger then lets the successor be scheduled in turn.  Without a
// programmatic dependency both instructions are no-ops.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// inclusive warp scan
template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T x) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T y = __shfl_up_sync(FULL, x, o);
        if (lane_id() >= o) x += y;
    }
    return x;
}

template <typename T>
__device__ __forceinline__ T warp_sum(T x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(FULL, x, o);
    return x;
}

// Exclusive block scan for blocks of up to 1024 threads; `total` receives the block sum.
// scratch: 33 entries of T in shared memory.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T x, T* scratch, T& total) {
    const int lane = lane_id(), warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    T inc = warp_inclusive_scan(x);
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        T s = lane < nwarp ? scratch[lane] : T(0);
        T si = warp_inclusive_scan(s);
        scratch[lane] = si - s;
        if (lane == 31) scratch[32] = si;
    }
    __syncthreads();
    T base = scratch[warp];
    total = scratch[32];
    __syncthreads();
    return base + inc - x;
}

// 16-byte vector reduction into global memory (sm_90+): four fp32 adds in one request.
__device__ __forceinline__ void red_add_v4(float* addr, float4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y),
                 "f"(v.z), "f"(v.w)
                 : "memory");
}

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// largest i in [0, n) with a[i] <= x, for ascending a with a[0] <= x
__device__ __forceinline__ int upper_row(const int64_t* a, int n, int64_t x) {
    int lo = 0, hi = n;  // invariant: a[lo] <= x, (hi == n or a[hi] > x)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (a[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

}  // namespace rp
