// Fused learner pass: Algorithm 1 lines 6-7 and 10 (and 12) for all n learners
// in one streaming sweep.  Every g_i and m_i is read once and m_i written once
// (12 bytes per learner-coordinate); acc_i = m_i + g_i is never stored.
//
// Work is cut by coordinate, not by learner: a tile of 1024 coordinates is
// owned by one block, each thread keeps its four coordinates for all learners,
// so the cross-learner sum of Algorithm 1 line 10 is a register accumulation
// in learner order 0..n-1 -- no atomics, no second pass, bitwise reproducible.
// Whether a coordinate is selected comes from the leader's bitmap; its rank in
// the ascending index list (where the gathered and reduced values go) from the
// per-tile prefix counts written by the selection kernel.
#pragma once
#include "common.cuh"

namespace sc {

constexpr int LP_THREADS = 256;            // x 4 coordinates = one tile
constexpr int LP_UNROLL = 8;               // pairs of 128-bit loads in flight per thread (tiles x learners of a burst)
constexpr int LP_BLOCKS_PER_SM = 2;
// burst shapes and blocks per SM by learner count (each measured against its neighbours on d = 25.6 M)
constexpr int LP_ONE_T = 2;                // single-learner form (learner-per-GPU deployment): tiles per burst
constexpr int LP_ONE_BLOCKS_PER_SM = 4;
constexpr int LP_FEW_T = 2;                // one learner in scalecom_step
constexpr int LP_FEW_BLOCKS_PER_SM = 4;
constexpr int LP_FEW2_T = 1;               // 2 or 3 learners: bursts of two learners
constexpr int LP_FEW2_BLOCKS_PER_SM = 5;
constexpr int LP_MID_T = 1;                // 4 to 7 learners: bursts of four learners
constexpr int LP_MID_BLOCKS_PER_SM = 3;
constexpr bool LP_MID_EARLY = true;
constexpr int LP_MANY_BLOCKS_PER_SM = 6;   // 16 learners and more: bursts of one learner

template <int N>
struct PtrTable {
    const float* g[N];
    float* m[N];
};

// Where else the single-learner form stores its kept values: one row per peer (this rank's row of every
// rank's gathered-rows buffer, peers' memory included), written with plain stores as the values are produced.
constexpr int LP_MAX_PEERS = 64;
// With tag != 0 the kernel also signals: once its last block is through, flag[q] (one word per destination, next
// to that destination's rows) receives tag with release semantics at system scope, so that a consumer that has
// read tag there with acquire semantics may read this rank's row.
struct PeerTable {
    float* dst[LP_MAX_PEERS];
    uint32_t* flag[LP_MAX_PEERS];
    uint32_t* done;                        // this handle's count of finished blocks (zero between launches)
    uint32_t tag;
    int32_t n;
};

struct LearnerParams {
    uint32_t d, k, ntiles;
    int32_t n;
    float beta, omb, lr, nf;               // omb = 1 - beta rounded once in fp32; nf = (float)n
    const uint32_t* bitmap;                // [ntiles * 32]
    uint32_t* bitmap_clear;                // single-learner form: the same words, zeroed once read (or nullptr)
    const uint32_t* tile_prefix;           // [ntiles + 1]
    float* out_val;                        // [k]
    int32_t* out_idx;                      // [k]: the ascending index list, written here from the ranks
    float* gathered;                       // [n * k] or nullptr
    float* weights;                        // [d] or nullptr (then Algorithm 1 line 12 is not applied here)
    unsigned long long* spans;             // nullptr, or where to accumulate the kernel's time span
    const uint32_t* status;                // the handle's status word: anything but DEV_OK and the kernel does nothing
};

// One burst of a thread covers LP_T consecutive tiles x LP_L learners (LP_T * LP_L = LP_UNROLL pairs of
// 128-bit loads in flight).  Few learners: more tiles per burst keep the loads in flight; many
// learners: fewer arrays per burst keep each burst inside a few pages.
// ONE: the single-learner form used when every learner has its own device -- n is 1 at compile time, no
// weights are touched (the reduced values do not exist yet), and ranks are checked against k before a value
// is written, because the bitmap and prefix counts then come from an index list received from elsewhere.
// MINB: blocks per SM the kernel is compiled for.  EARLY: the first burst of g and m is requested before
// anything waits on the bitmap.  Few learners per tile want both (occupancy and the early request supply the
// loads in flight that a burst of 8 learners supplies by itself); with 4 or more learners the later order and
// 2 blocks per SM measured faster.
template <int N, bool VEC, int LP_T, int LP_L, bool ONE = false, int MINB = (ONE ? LP_ONE_BLOCKS_PER_SM : LP_BLOCKS_PER_SM),
          bool EARLY = ONE, bool N1 = ONE>
__global__ void __launch_bounds__(LP_THREADS, MINB)
learner_pass_kernel(const __grid_constant__ PtrTable<N> tab, const LearnerParams P, const __grid_constant__ PeerTable peers) {
    static_assert(LP_T * LP_L <= LP_UNROLL, "burst shape");
    constexpr bool GUARD = ONE;
    constexpr bool TAIL_LOOP = LP_L >= 5;
    const uint32_t tid = threadIdx.x, lane = lane_id();
    const uint32_t d = P.d;
    const int n = N1 ? 1 : P.n;                    // N1: one learner, known when compiling
    float* const weights = ONE ? nullptr : P.weights;
    float* const gathered = ONE ? nullptr : P.gathered;
    const uint32_t wi = tid >> 3;                  // this thread's bitmap word inside a tile
    const uint32_t sh = (tid & 7u) * 4u;           // and its first bit inside that word
    // a selection kernel that gave up leaves no valid bitmap or prefix counts behind
    if (ld_relaxed_u32(P.status) != DEV_OK) return;
    span_begin(P.spans);

    const uint32_t nsuper = (P.ntiles + LP_T - 1) / LP_T;
    for (uint32_t sup = blockIdx.x; sup < nsuper; sup += gridDim.x) {
        // EARLY: the first burst of g and m is requested before anything waits on the bitmap, so that one memory
        // latency covers both.
        uint32_t pc[LP_T], bw[LP_T], tp[LP_T];
#pragma unroll
        for (int t = 0; t < LP_T; ++t) {
            const uint32_t tile = sup * LP_T + t;
            const bool have = tile < P.ntiles;                         // uniform across the block
            pc[t] = have ? tile * TILE + tid * 4u : d;                 // d: nothing to do
            bw[t] = !have ? 0u : ONE ? P.bitmap[size_t(tile) * 32 + lane] : __ldg(&P.bitmap[size_t(tile) * 32 + lane]);
            tp[t] = have ? __ldg(&P.tile_prefix[tile]) : 0u;
        }
        float gv[LP_T][LP_L][4], mv[LP_T][LP_L][4];
        auto load_burst = [&](int i0) {
#pragma unroll
            for (int t = 0; t < LP_T; ++t)
#pragma unroll
                for (int u = 0; u < LP_L; ++u)
                    if (i0 + u < n && pc[t] < d) {
                        load_quad_stream<VEC>(tab.g[i0 + u], pc[t], d, gv[t][u]);
                        load_quad_stream<VEC>(tab.m[i0 + u], pc[t], d, mv[t][u]);
                    }
        };
        if (EARLY) load_burst(0);

        // per tile: selection bits of this thread's four coordinates and the rank of the first selected one
        uint32_t nib[LP_T], rank0[LP_T];
#pragma unroll
        for (int t = 0; t < LP_T; ++t) {
            const uint32_t cnt = __popc(bw[t]);
            const uint32_t incl = warp_incl_scan(cnt);
            const uint32_t excl_word = __shfl_sync(FULL, incl - cnt, wi);
            const uint32_t myword = __shfl_sync(FULL, bw[t], wi);
            nib[t] = (myword >> sh) & 15u;
            rank0[t] = tp[t] + excl_word + __popc(myword & ((1u << sh) - 1u));
        }

        if (ONE && P.bitmap_clear) {           // every warp has its copy of the words: leave the bitmap zero for the next list
            __syncthreads();
            if (tid < 32) {
#pragma unroll
                for (int t = 0; t < LP_T; ++t)
                    if (sup * LP_T + t < P.ntiles) P.bitmap_clear[size_t(sup * LP_T + t) * 32 + lane] = 0u;
            }
        }

        // weights at the selected coordinates, fetched now so that their latency hides behind the learner loop
        float wv[LP_T][4];
#pragma unroll
        for (int t = 0; t < LP_T; ++t)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                wv[t][c] = (weights && ((nib[t] >> c) & 1u) && pc[t] + c < d) ? weights[pc[t] + c] : 0.0f;

        float sum[LP_T][4];
        for (int i0 = 0; i0 < n; i0 += LP_L) {
            if (!EARLY || i0 > 0) load_burst(i0);
#pragma unroll
            for (int t = 0; t < LP_T; ++t)
#pragma unroll
                for (int u = 0; u < LP_L; ++u)
                    if (i0 + u < n && pc[t] < d) {
                        const int i = i0 + u;
                        float acc[4], out[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            acc[c] = __fadd_rn(mv[t][u][c], gv[t][u][c]);                    // line 6: m + g
                            sum[t][c] = (i == 0) ? acc[c] : __fadd_rn(sum[t][c], acc[c]);    // line 10, learner order
                            const float r = ((nib[t] >> c) & 1u) ? 0.0f : acc[c];            // acc - CLT-k(acc)
                            out[c] = __fadd_rn(__fmul_rn(P.omb, mv[t][u][c]), __fmul_rn(P.beta, r));   // Eq. 4
                        }
                        store_quad_stream<VEC>(tab.m[i], pc[t], d, out);
                        if (nib[t] && gathered) {                                             // Eq. 3: learner i's kept values
                            uint32_t r = rank0[t];
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                if (((nib[t] >> c) & 1u) && (!GUARD || r < P.k)) gathered[size_t(i) * P.k + r++] = acc[c];
                        }
                    }
        }
#pragma unroll
        for (int t = 0; t < LP_T; ++t)
            if (nib[t] && pc[t] < d) {
                uint32_t r = rank0[t];
                if (!TAIL_LOOP) {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (((nib[t] >> c) & 1u) && (!GUARD || r < P.k)) {
                            const float v = __fdiv_rn(sum[t][c], P.nf);                       // line 10: one division by n
                            P.out_idx[r] = int32_t(pc[t] + c);
                            P.out_val[r] = v;
                            if (ONE)
                                for (int q = 0; q < peers.n; ++q) peers.dst[q][r] = v;    // Eq. 3's values, sent as they are made
                            ++r;
                            if (weights) weights[pc[t] + c] = __fsub_rn(wv[t][c], __fmul_rn(P.lr, v));   // line 12
                        }
                    continue;
                }
                // bursts of five learners and more: one turn per selected coordinate of the lane (usually one), so that
                // the division is not laid out four times (8 learners: -1 us; evenly spread picks, as the chunk-wise
                // selector and a long run leave them: -2 to -4 us; the shapes for fewer learners measured slower with it)
                for (uint32_t left = nib[t]; left; left &= left - 1u) {
                    const uint32_t c = __ffs(left) - 1u;
                    if (GUARD && r >= P.k) break;
                    const float sc = c == 0 ? sum[t][0] : c == 1 ? sum[t][1] : c == 2 ? sum[t][2] : sum[t][3];
                    const float wc = c == 0 ? wv[t][0] : c == 1 ? wv[t][1] : c == 2 ? wv[t][2] : wv[t][3];
                    const float v = __fdiv_rn(sc, P.nf);                                      // line 10: one division by n
                    P.out_idx[r] = int32_t(pc[t] + c);
                    P.out_val[r] = v;
                    if (ONE)
                        for (int q = 0; q < peers.n; ++q) peers.dst[q][r] = v;        // Eq. 3's values, sent as they are made
                    ++r;
                    if (weights) weights[pc[t] + c] = __fsub_rn(wc, __fmul_rn(P.lr, v));      // line 12
                }
            }
    }
    if (ONE && peers.tag != 0u) {
        // every block's stores are ordered before its increment (barrier, then a system-wide fence by the thread
        // that counts); the block that counts last therefore publishes the flags after all of them
        __syncthreads();
        if (tid == 0) {
            __threadfence_system();
            if (atomicAdd(peers.done, 1u) == gridDim.x - 1u) {
                __threadfence_system();
                for (int q = 0; q < peers.n; ++q) st_release_sys_u32(peers.flag[q], peers.tag);
                *peers.done = 0u;
            }
        }
    }
    span_end(P.spans);
}

// Algorithm 1 line 12 as its own kernel: theta[idx[j]] -= lr * val[j].
__global__ void __launch_bounds__(256) apply_update_kernel(float* __restrict__ weights, const int32_t* __restrict__ idx,
                                                           const float* __restrict__ val, uint32_t k, float lr,
                                                           const uint32_t* __restrict__ status) {
    if (ld_relaxed_u32(status) != DEV_OK) return;                      // no valid index list after a device error
    for (uint32_t j = blockIdx.x * blockDim.x + threadIdx.x; j < k; j += gridDim.x * blockDim.x) {
        const int32_t p = idx[j];
        weights[p] = __fsub_rn(weights[p], __fmul_rn(lr, val[j]));
    }
}

}  // namespace sc
