// Diagnostics of Sections 2-3: they read the state and change nothing.
//   mean_acc_kernel      the all-reduced error-feedback gradient (1/n) sum_i (m_i + g_i), whose top-k set
//                        the paper calls the "true top-k"
//   overlap_kernel       |I1 and I2| of two selection bitmaps; Eq. 5's d is k minus that
//   dot3_kernel          x.y, x.x, y.y in double for the cosine distance of two memories
#pragma once
#include "common.cuh"
#include "learner_pass.cuh"

namespace sc {

// Same arithmetic as the reduction of Algorithm 1 line 10, for every coordinate: learner order, one division.
template <int N, bool VEC>
__global__ void __launch_bounds__(256) mean_acc_kernel(const __grid_constant__ PtrTable<N> tab, int n, uint32_t d, float nf,
                                                       float* __restrict__ mean) {
    const uint32_t quads = (d + 3u) / 4u;
    for (uint32_t qd = blockIdx.x * blockDim.x + threadIdx.x; qd < quads; qd += gridDim.x * blockDim.x) {
        const uint32_t p = qd * 4u;
        float s[4];
        for (int i = 0; i < n; ++i) {
            float gv[4], mv[4];
            load_quad_stream<VEC>(tab.g[i], p, d, gv);
            load_quad_stream<VEC>(tab.m[i], p, d, mv);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float acc = __fadd_rn(mv[c], gv[c]);
                s[c] = i == 0 ? acc : __fadd_rn(s[c], acc);
            }
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (p + c < d) mean[p + c] = __fdiv_rn(s[c], nf);
    }
}

__global__ void __launch_bounds__(256) overlap_kernel(const uint32_t* __restrict__ a, const uint32_t* __restrict__ b,
                                                      size_t nwords, unsigned long long* out) {
    unsigned long long local = 0;
    for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < nwords; i += size_t(gridDim.x) * blockDim.x)
        local += uint32_t(__popc(a[i] & b[i]));
    uint32_t w = __reduce_add_sync(FULL, uint32_t(local));             // < 2^32 per thread: nwords / threads * 32
    if (lane_id() == 0 && w) atomicAdd(out, (unsigned long long)w);
}

__global__ void __launch_bounds__(256) dot3_kernel(const float* __restrict__ x, const float* __restrict__ y, uint32_t d,
                                                   double* out3) {
    double xy = 0.0, xx = 0.0, yy = 0.0;
    for (uint32_t p = blockIdx.x * blockDim.x + threadIdx.x; p < d; p += gridDim.x * blockDim.x) {
        const double a = double(x[p]), b = double(y[p]);
        xy += a * b; xx += a * a; yy += b * b;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xy += __shfl_xor_sync(FULL, xy, o);
        xx += __shfl_xor_sync(FULL, xx, o);
        yy += __shfl_xor_sync(FULL, yy, o);
    }
    if (lane_id() == 0) { atomicAdd(&out3[0], xy); atomicAdd(&out3[1], xx); atomicAdd(&out3[2], yy); }
}

}  // namespace sc
