// Pieces of the learner-per-GPU deployment (Section 4 / Appendix E: the leader's indices are broadcast,
// every worker compresses its own error-feedback gradient with them, the kept values are reduced).
//   indices_to_bitmap_kernel   a received ascending index list -> selection bitmap + per-tile prefix counts,
//                              the form the learner pass consumes
//   reduce_rows_kernel         Algorithm 1 line 10 on gathered rows: learner (rank) order, one division
#pragma once
#include "common.cuh"

namespace sc {

// bitmap must be zero on entry.  Entries must be strictly ascending and < d; a violation sets the
// status word (DEV_INTERNAL) instead of writing out of bounds (tile_prefix may then hold stale entries:
// the consumer checks every rank against k).
// tile_prefix[t] = number of entries below t * TILE.  Entry j is the first one at or past the start of
// every tile t with idx[j-1] / TILE < t <= idx[j] / TILE, so the thread that holds entry j writes j there:
// usually zero or one tile; a long run of empty tiles is filled by the whole warp.
__global__ void __launch_bounds__(256) indices_to_bitmap_kernel(const int32_t* __restrict__ idx, uint32_t k, uint32_t d,
                                                                uint32_t ntiles, uint32_t* bitmap, uint32_t* tile_prefix,
                                                                uint32_t* status) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t gsize = gridDim.x * blockDim.x;
    constexpr uint32_t OWN = 4;                                          // tiles a lane fills by itself
    for (uint32_t j0 = blockIdx.x * blockDim.x + (threadIdx.x & ~31u); j0 < k; j0 += gsize) {   // warp-uniform
        const uint32_t j = j0 + lane;
        uint32_t t_lo = 1, t_hi = 0;                                     // tiles [t_lo, t_hi] get prefix j (empty by default)
        uint32_t tail_lo = 1, tail_hi = 0;                               // the last entry also fills the tiles after it with k
        if (j < k) {
            const uint32_t p = uint32_t(idx[j]);
            const uint32_t prev = j ? uint32_t(idx[j - 1]) : 0u;
            const bool ok = p < d && (j == 0 || prev < p);
            if (ok) {
                atomicOr(&bitmap[p >> 5], 1u << (p & 31u));
                t_lo = j ? prev / TILE + 1u : 0u;
                t_hi = p / TILE;
                if (j == k - 1) { tail_lo = t_hi + 1u; tail_hi = ntiles; }
            } else {
                atomicCAS(status, DEV_OK, DEV_INTERNAL);
            }
        }
#pragma unroll
        for (int round = 0; round < 2; ++round) {
            const uint32_t lo = round ? tail_lo : t_lo, hi = round ? tail_hi : t_hi;
            const uint32_t val = round ? k : j;
            const uint32_t len = hi >= lo ? hi - lo + 1u : 0u;
            for (uint32_t q = 0; q < (len < OWN ? len : OWN); ++q) tile_prefix[lo + q] = val;
            uint32_t longs = __ballot_sync(FULL, len > OWN);
            while (longs) {                                               // warp-uniform
                const int src = __ffs(longs) - 1;
                longs &= longs - 1u;
                const uint32_t s_lo = __shfl_sync(FULL, lo + OWN, src), s_len = __shfl_sync(FULL, len - OWN, src);
                const uint32_t s_val = __shfl_sync(FULL, val, src);
                for (uint32_t q = lane; q < s_len; q += 32u) tile_prefix[s_lo + q] = s_val;
            }
        }
    }
}

// val[j] = (rows[0][j] + rows[1][j] + ... + rows[n-1][j]) / n, summed in row order; with weights given,
// Algorithm 1 line 12 follows in the same thread: theta[idx[j]] -= lr * val[j] (an index >= d sets the status
// word instead).
// wait_flags != nullptr: the rows are being stored by other ranks' kernels; row i may be read once wait_flags[i]
// holds tag (written there by its sender after all its stores).  Every block waits for all n flags, at most
// spin_limit polls each; when a wait runs out the status word becomes DEV_TIMEOUT and nothing is written.
__global__ void __launch_bounds__(256) reduce_rows_kernel(const float* rows, int n, uint32_t k, float nf,
                                                          float* __restrict__ val, const int32_t* __restrict__ idx,
                                                          float* __restrict__ weights, uint32_t d, float lr,
                                                          uint32_t* status, const uint32_t* wait_flags, uint32_t tag,
                                                          uint32_t spin_limit) {
    if (wait_flags) {
        __shared__ int all_there;
        if (threadIdx.x == 0) all_there = 1;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            bool there = false;
            for (uint32_t it = 0; it < spin_limit; ++it) {
                if (ld_acquire_sys_u32(wait_flags + i) == tag) { there = true; break; }
                if (ld_relaxed_u32(status) != DEV_OK) break;
                if (it > 64) __nanosleep(it > 4096 ? 256 : 64);
            }
            if (!there) {
                atomicCAS(status, DEV_OK, DEV_TIMEOUT);
                all_there = 0;
            }
        }
        __syncthreads();
        if (!all_there) return;
    }
    for (uint32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < k; j += gridDim.x * blockDim.x) {
        float s = __ldcg(&rows[j]);                                      // (L2: the rows may have come from other GPUs)
        for (int i = 1; i < n; ++i) s = __fadd_rn(s, __ldcg(&rows[size_t(i) * k + j]));
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
