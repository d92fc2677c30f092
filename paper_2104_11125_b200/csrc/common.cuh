// Shared device helpers of the CLT-k kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sc {

// Device-side status codes (mirrors of the negative C-ABI errors, stored positive).
constexpr uint32_t DEV_OK = 0;
constexpr uint32_t DEV_TIMEOUT = 5;
constexpr uint32_t DEV_INTERNAL = 7;

// Coordinates per tile of the learner pass; one tile owns 32 words of the selection bitmap.
constexpr uint32_t TILE = 1024;

constexpr unsigned FULL = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ uint32_t warp_id() { return threadIdx.x >> 5; }

// Magnitude key of Eq. 2: the bit pattern of |x|; unsigned order == magnitude order.
__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// Total order "larger magnitude first, then lower index first" as one 62-bit
// number: larger composite == earlier in that order; all composites are distinct.
__device__ __forceinline__ uint64_t composite(uint32_t key, uint32_t idx) {
    return (uint64_t(key) << 31) | uint64_t(0x7FFFFFFFu - idx);
}

// ---- streaming loads / stores ---------------------------------------------------------------
// Plain ld.global / st.global on purpose: on B200 the default cache policy streamed measurably
// faster than the .cs / .cg / no-allocate variants (0.380 ms vs 0.403 ms for the learner pass of
// the ResNet-50-shaped workload).
// Four consecutive coordinates starting at p.  VEC: one 128-bit load when the
// quad is fully inside [0, d); otherwise (ragged tail, or unaligned vectors)
// guarded scalar loads that return 0 beyond d.
template <bool VEC>
__device__ __forceinline__ void load_quad_stream(const float* __restrict__ a, uint32_t p, uint32_t d, float (&v)[4]) {
    if (VEC && p + 4u <= d) {
        const float4 t = *reinterpret_cast<const float4*>(a + p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = (p + c < d) ? a[p + c] : 0.0f;
    }
}

// 128-bit load with an L2 cache-hint policy (createpolicy); p is 16-byte aligned
__device__ __forceinline__ float4 ld_quad_policy(const float* p, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(__cvta_generic_to_global(p)), "l"(policy));
    return v;
}

template <bool VEC>
__device__ __forceinline__ void store_quad_stream(float* __restrict__ a, uint32_t p, uint32_t d, const float (&v)[4]) {
    if (VEC && p + 4u <= d) {
        *reinterpret_cast<float4*>(a + p) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (p + c < d) a[p + c] = v[c];
    }
}

// ---- warp scans -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(FULL, v, o);
        if (lane_id() >= (uint32_t)o) v += t;
    }
    return v;
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t v) { return __reduce_add_sync(FULL, v); }

// ---- in-kernel time spans ------------------------------------------------------------------------
// A kernel given a non-null `sp` accumulates {~(earliest block start), latest block end} on the
// nanosecond global timer into sp[0], sp[1] (both with atomicMax on zero-initialised words), which
// separates kernel time from launch gaps and event overhead.  One atomic per block at each end.
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void span_begin(unsigned long long* sp) {
    if (sp && threadIdx.x == 0) atomicMax(&sp[0], ~global_timer_ns());
}
__device__ __forceinline__ void span_end(unsigned long long* sp) {
    if (sp) {
        __syncthreads();
        if (threadIdx.x == 0) atomicMax(&sp[1], global_timer_ns());
    }
}

// ---- bounded grid barrier -----------------------------------------------------------------------
// All blocks of a cooperative launch call this the same number of times.  The
// 64-bit arrival counter only ever grows; each arrival derives its own release
// value from it, so nothing needs resetting between barriers or launches as long
// as every launch completes (the host zeroes the counter after a device error).
// The wait is bounded: on expiry the status word becomes DEV_TIMEOUT, every
// waiter sees it and the function returns false; callers then return at once.
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// system scope: the word may live in another GPU's memory, or be written from there
__device__ __forceinline__ uint32_t ld_acquire_sys_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys_u32(uint32_t* p, uint32_t v) {
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

struct GridBarrier {
    unsigned long long* arrive;
    uint32_t nblocks;
    uint32_t* status;
    uint32_t spin_limit;       // 0: every wait expires at once
};

__device__ __forceinline__ bool grid_barrier(const GridBarrier& gb, int* smem_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 0;
        __threadfence();
        const unsigned long long old = atomicAdd(gb.arrive, 1ULL);
        const unsigned long long target = (old / gb.nblocks + 1ULL) * gb.nblocks;
        for (uint32_t it = 0; it < gb.spin_limit; ++it) {
            if (ld_acquire_u64(gb.arrive) >= target) { ok = 1; break; }
            if (ld_relaxed_u32(gb.status) != DEV_OK) break;
            if (it > 64) __nanosleep(it > 4096 ? 256 : 32);
        }
        if (!ok) atomicCAS(gb.status, DEV_OK, DEV_TIMEOUT);
        __threadfence();
        *smem_flag = ok;
    }
    __syncthreads();
    return *smem_flag != 0;
}

}  // namespace sc
