// Pieces of the learner-per-GPU deployment (Section 4 / Appendix E: the leader's indices are broadcast,
// every worker compresses its own error-feedback gradient with them, the kept values are reduced).
//   indices_to_bitmap_kernel   a received ascending index list -> selection bitmap + per-tile prefix counts,
//                              the form the learner pass consumes
//   reduce_rows_kernel         Algorithm 1 line 10 on gathered rows: learner (rank) order, one division
#pragma once
#include "common.cuh"

namespace sc {

// bitmap must be zero on entry.  Entries must be strictly ascending and < d; a violation sets the
// status word (DEV_INTERNAL) instead of writing out of bounds.
__global__ void __launch_bounds__(256) indices_to_bitmap_kernel(const int32_t* __restrict__ idx, uint32_t k, uint32_t d,
                                                                uint32_t ntiles, uint32_t* bitmap, uint32_t* tile_prefix,
                                                                uint32_t* status) {
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, gsize = gridDim.x * blockDim.x;
    for (uint32_t j = gtid; j < k; j += gsize) {
        const uint32_t p = uint32_t(idx[j]);
        const bool ok = p < d && (j == 0 || uint32_t(idx[j - 1]) < p);
        if (ok) atomicOr(&bitmap[p >> 5], 1u << (p & 31u));
        else atomicCAS(status, DEV_OK, DEV_INTERNAL);
    }
    // selected coordinates before a tile = entries below its first coordinate: a lower bound in the list,
    // one warp per tile probing 32 positions per round (4-5 dependent rounds instead of log2 k)
    const uint32_t lane = threadIdx.x & 31u, nwarps = gsize >> 5;
    for (uint32_t tile = gtid >> 5; tile <= ntiles; tile += nwarps) {
        const uint64_t p0 = uint64_t(tile) * TILE;
        uint32_t lo = 0, hi = k;
        while (lo < hi) {                                    // the answer stays in [lo, hi]; the interval shrinks each round
            const uint32_t step = (hi - lo + 31u) >> 5;
            const uint64_t pos = uint64_t(lo) + uint64_t(lane) * step;
            const bool below = pos < hi && uint64_t(uint32_t(idx[pos])) < p0;
            const uint32_t c = __popc(__ballot_sync(FULL, below));
            if (c == 0) { hi = lo; break; }
            const uint64_t top = uint64_t(lo) + uint64_t(c) * step;
            lo = lo + (c - 1) * step + 1;
            hi = top < hi ? uint32_t(top) : hi;
        }
        if (lane == 0) tile_prefix[tile] = lo;
    }
}

// val[j] = (rows[0][j] + rows[1][j] + ... + rows[n-1][j]) / n, summed in row order; with weights given,
// Algorithm 1 line 12 follows in the same thread: theta[idx[j]] -= lr * val[j] (an index >= d sets the status
// word instead).
__global__ void __launch_bounds__(256) reduce_rows_kernel(const float* __restrict__ rows, int n, uint32_t k, float nf,
                                                          float* __restrict__ val, const int32_t* __restrict__ idx,
                                                          float* __restrict__ weights, uint32_t d, float lr,
                                                          uint32_t* status) {
    for (uint32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < k; j += gridDim.x * blockDim.x) {
        float s = rows[j];
        for (int i = 1; i < n; ++i) s = __fadd_rn(s, rows[size_t(i) * k + j]);
        const float v = __fdiv_rn(s, nf);
        val[j] = v;
        if (weights) {
            const uint32_t p = uint32_t(idx[j]);
            if (p < d) weights[p] = __fsub_rn(weights[p], __fmul_rn(lr, v));
            else atomicCAS(status, DEV_OK, DEV_INTERNAL);
        }
    }
}

}  // namespace sc
