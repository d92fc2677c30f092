// Exact top-k inside every layer: Eq. 2 applied to each layer on its own, with Section 4's per-layer
// compression rates (layer s keeps keep[s] of its size[s] coordinates; ties go to the lower index).
//
// One persistent cooperative kernel.  All layers are searched at once by a most-significant-digit
// radix select over the 31-bit magnitude key, 11 + 10 + 10 bits:
//   stream pass   every block walks a contiguous range of spans (2048 coordinates), counts the digit of
//                 the coordinates that still match their layer's prefix into a shared-memory histogram
//                 and adds it to the layer's row of a global histogram whenever its range moves on to
//                 another layer; a span that holds several (small) layers counts straight into the rows
//   find          layer s is looked at by block s mod grid: the digit where the count from the top
//                 crosses what the layer still has to keep extends its prefix; the row is left zero
// After three rounds the prefix is the layer's threshold key T and r says how many of the coordinates with
// key == T are kept.  Only if some layer has more such coordinates than r (a tie across the boundary) three
// more rounds run, over the offset inside the layer of the coordinates with key == T, from the bottom: they
// end with the largest offset that is still kept.  A last pass marks the bitmap, counts per tile, and a
// scan over tiles gives the prefix counts the learner pass needs.
// HBM traffic: 4 passes (7 with ties) x 8 B per coordinate.
#pragma once
#include "chunk_select.cuh"   // layer_of, CS_MAX_LAYERS
#include "common.cuh"

namespace sc {

#ifndef SC_LT_BLOCKS_PER_SM
#define SC_LT_BLOCKS_PER_SM 2
#endif
#ifndef SC_LT_UNROLL
#define SC_LT_UNROLL 2
#endif

constexpr int LT_THREADS = 512;
constexpr int LT_BLOCKS_PER_SM = SC_LT_BLOCKS_PER_SM;
constexpr int LT_UNROLL = SC_LT_UNROLL;             // spans whose loads a thread has in flight
constexpr uint32_t LT_SPAN = LT_THREADS * 4;        // coordinates a block takes per iteration (two tiles)
constexpr uint32_t LT_BINS = 2048;                  // widest digit: 11 bits
constexpr uint32_t LT_NOSPLIT = 0xFFFFFFFFu;
// Words between two layers' rows of the global histogram: an odd number of 128-byte lines, so that the same
// bin of different layers does not sit a power of two apart.
constexpr uint32_t LT_ROW = LT_BINS + 32;

struct LayerTopkParams {
    const float* g;
    const float* m;
    uint32_t d, k;
    uint32_t spin_limit;
    uint32_t nl;
    const uint32_t* layer_off;          // [nl + 1] first coordinate of each layer
    const uint32_t* layer_k0;           // [nl + 1] prefix sums of keep[]
    uint32_t* ghist;                    // [nl * LT_ROW], zero on entry, left zero
    uint4* lstate;                      // [nl] {prefix or T, still to keep, split flag, offset prefix or last kept offset}
    uint32_t* tie_flag;                 // one word, zero on entry, left zero
    uint32_t* block_tot;                // [grid]
    uint32_t* bitmap;                   // [ntiles * 32]
    uint32_t* tile_prefix;              // [ntiles + 1]
    uint32_t ntiles;
    uint32_t* ctrl;                     // status word at [1], path at [2], count at [3]
    unsigned long long* barrier;        // arrival counter used by this kernel only
    int32_t* out_idx;                   // [k] or nullptr
    unsigned long long* spans;
};

struct LayerTopkShared {
    uint32_t off[CS_MAX_LAYERS + 1];    // layer starts
    uint32_t x[CS_MAX_LAYERS];          // per layer: key prefix, finally T
    uint32_t w[CS_MAX_LAYERS];          // per layer: LT_NOSPLIT, or offset prefix / last kept offset
    uint32_t hist[LT_BINS];
    uint32_t wtot[LT_THREADS / 32];
    uint32_t res[3];
    uint32_t base;
    int flag;
};

// Exclusive scan over the block (one value per thread, thread order); returns this thread's prefix, *total the sum.
__device__ __forceinline__ uint32_t lt_block_excl_scan(uint32_t v, uint32_t* wtot, uint32_t* total) {
    const uint32_t lane = lane_id(), wp = warp_id();
    const uint32_t incl = warp_incl_scan(v);
    __syncthreads();                                   // wtot may still be read from the call before
    if (lane == 31) wtot[wp] = incl;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int i = 0; i < LT_THREADS / 32; ++i) {
        const uint32_t t = wtot[i];
        if (uint32_t(i) < wp) before += t;
        all += t;
    }
    *total = all;
    return before + incl - v;
}

// hist[0 .. nbins) holds counts.  Finds the bin where the running count, taken from the top bin down
// (FROM_TOP) or from bin 0 up, first reaches r (1 <= r <= total): res = {bin, count before it, count in it}.
// res[0] stays LT_NOSPLIT when r is out of range.
template <bool FROM_TOP>
__device__ __forceinline__ void lt_block_find(LayerTopkShared& S, uint32_t nbins, uint32_t r) {
    const uint32_t tid = threadIdx.x;
    uint32_t c[4], tsum = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t q = tid * 4 + j;                                  // position in search order
        c[j] = q < nbins ? S.hist[FROM_TOP ? nbins - 1 - q : q] : 0u;
        tsum += c[j];
    }
    if (tid == 0) S.res[0] = LT_NOSPLIT;
    uint32_t total;
    uint32_t acc = lt_block_excl_scan(tsum, S.wtot, &total);             // (its barriers order the write above)
    if (tsum && acc < r && r <= acc + tsum) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (acc < r && r <= acc + c[j]) {
                const uint32_t q = tid * 4 + j;
                S.res[0] = FROM_TOP ? nbins - 1 - q : q;
                S.res[1] = acc;
                S.res[2] = c[j];
            }
            acc += c[j];
        }
    }
    __syncthreads();
}

// Does coordinate (key, offset o inside its layer) still match in round PS, and which digit does it count?
template <int PS>
__device__ __forceinline__ bool lt_match(uint32_t key, uint32_t o, uint32_t x, uint32_t w, uint32_t* dg) {
    if (PS == 0) { *dg = key >> 20; return true; }
    if (PS == 1) { *dg = (key >> 10) & 1023u; return (key >> 20) == x; }
    if (PS == 2) { *dg = key & 1023u; return (key >> 10) == x; }
    if (PS == 3) { *dg = o >> 20; return key == x && w != LT_NOSPLIT; }
    if (PS == 4) { *dg = (o >> 10) & 1023u; return key == x && w != LT_NOSPLIT && (o >> 20) == w; }
    *dg = o & 1023u;
    return key == x && w != LT_NOSPLIT && (o >> 10) == w;
}

// Adds what the shared histogram holds to layer `layer`'s global row and leaves it zero.
__device__ __forceinline__ void lt_flush(LayerTopkShared& S, uint32_t* ghist, uint32_t layer) {
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < LT_BINS; i += LT_THREADS) {
        const uint32_t v = S.hist[i];
        if (v) {
            atomicAdd(&ghist[size_t(layer) * LT_ROW + i], v);
            S.hist[i] = 0;
        }
    }
    __syncthreads();
}

// This thread's quads of spans sp0 .. sp0 + LT_UNROLL - 1 (those below span_hi and d).  When all of them are
// whole the loads carry no predicate, which is what keeps all of them in flight at once.
template <bool VEC>
__device__ __forceinline__ void lt_load_spans(const LayerTopkParams& P, uint32_t sp0, uint32_t span_hi,
                                              float (&gv)[LT_UNROLL][4], float (&mv)[LT_UNROLL][4]) {
    const uint32_t tid = threadIdx.x, d = P.d;
    const bool whole = VEC && sp0 + LT_UNROLL <= span_hi && uint64_t(sp0 + LT_UNROLL) * LT_SPAN <= d;   // uniform
    if (whole) {
#pragma unroll
        for (int u = 0; u < LT_UNROLL; ++u) {
            const uint32_t p = (sp0 + u) * LT_SPAN + tid * 4u;
            const float4 a = *reinterpret_cast<const float4*>(P.g + p);
            const float4 b = *reinterpret_cast<const float4*>(P.m + p);
            gv[u][0] = a.x; gv[u][1] = a.y; gv[u][2] = a.z; gv[u][3] = a.w;
            mv[u][0] = b.x; mv[u][1] = b.y; mv[u][2] = b.z; mv[u][3] = b.w;
        }
    } else {
#pragma unroll
        for (int u = 0; u < LT_UNROLL; ++u) {
            const uint32_t p = (sp0 + u) * LT_SPAN + tid * 4u;
            if (sp0 + u < span_hi && p < d) {
                load_quad_stream<VEC>(P.g, p, d, gv[u]);
                load_quad_stream<VEC>(P.m, p, d, mv[u]);
            }
        }
    }
}

// One counting pass over this block's spans [span_lo, span_hi).
template <int PS, bool VEC>
__device__ __forceinline__ void lt_stream_pass(const LayerTopkParams& P, LayerTopkShared& S, uint32_t span_lo,
                                               uint32_t span_hi, uint32_t layer_first) {
    const uint32_t tid = threadIdx.x, d = P.d;
    uint32_t cur = layer_first;                 // layer of this thread's quad (moves forward only)
    uint32_t cf = layer_first, cl = layer_first;        // layers of the span's first and last coordinate (uniform)
    uint32_t hist_layer = LT_NOSPLIT;           // layer whose counts the shared histogram holds (uniform)
    constexpr int U = PS < 3 ? LT_UNROLL : 1;   // the tie rounds read only the spans of layers with a tie to split
    for (uint32_t sp0 = span_lo; sp0 < span_hi; sp0 += U) {
        if (PS >= 3) {
            const uint32_t p0 = sp0 * LT_SPAN, pe = min(p0 + LT_SPAN, d) - 1u;
            while (p0 >= S.off[cf + 1]) ++cf;
            while (pe >= S.off[cl + 1]) ++cl;
            bool any = false;
            for (uint32_t s = cf; s <= cl; ++s) any = any || S.w[s] != LT_NOSPLIT;
            if (!any) continue;                                             // uniform
        }
        // all loads of U spans first, then the counting (which may stop for a flush in between)
        float gv[LT_UNROLL][4], mv[LT_UNROLL][4];
        if (PS < 3) {
            lt_load_spans<VEC>(P, sp0, span_hi, gv, mv);
        } else {
            const uint32_t p = sp0 * LT_SPAN + tid * 4u;
            if (p < d) {
                load_quad_stream<VEC>(P.g, p, d, gv[0]);
                load_quad_stream<VEC>(P.m, p, d, mv[0]);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t sp = sp0 + u;
            if (sp >= span_hi) break;                                       // uniform
            const uint32_t p0 = sp * LT_SPAN, pe = min(p0 + LT_SPAN, d) - 1u;
            while (p0 >= S.off[cf + 1]) ++cf;
            while (pe >= S.off[cl + 1]) ++cl;
            const bool uniform = cf == cl;
            if (uniform && hist_layer != cf) {
                if (hist_layer != LT_NOSPLIT) lt_flush(S, P.ghist, hist_layer);
                hist_layer = cf;
            }
            const uint32_t p = p0 + tid * 4u;
            if (p >= d) continue;               // (the uniform decisions above are already taken)
            while (p >= S.off[cur + 1]) ++cur;
            uint32_t s = cur;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t pc = p + c;
                if (pc >= d) break;
                while (pc >= S.off[s + 1]) ++s;
                const uint32_t key = mag_key(__fadd_rn(mv[u][c], gv[u][c]));
                uint32_t dg;
                if (lt_match<PS>(key, pc - S.off[s], S.x[s], S.w[s], &dg)) {
                    // a span where layers meet counts straight into their global rows (taking such a span through
                    // the shared histogram one layer at a time measured 20 % slower per pass)
                    if (uniform) atomicAdd(&S.hist[dg], 1u);
                    else atomicAdd(&P.ghist[size_t(s) * LT_ROW + dg], 1u);
                }
            }
        }
    }
    if (hist_layer != LT_NOSPLIT) lt_flush(S, P.ghist, hist_layer);
}

// Round PS for the layers this block looks after: extend the prefix from the layer's global row.
template <int PS>
__device__ __forceinline__ void lt_find_round(const LayerTopkParams& P, LayerTopkShared& S) {
    const uint32_t tid = threadIdx.x;
    constexpr uint32_t nbins = (PS == 0 || PS == 3) ? 2048u : 1024u;
    for (uint32_t s = blockIdx.x; s < P.nl; s += gridDim.x) {
        uint4 st = make_uint4(0, 0, 0, LT_NOSPLIT);
        if (PS > 0) st = __ldcg(&P.lstate[s]);
        if (PS >= 3 && st.z == 0) continue;                                // uniform: no tie to split in this layer
        // (an exchange, not a load and a store: one trip to L2 per word)
        for (uint32_t i = tid; i < LT_BINS; i += LT_THREADS)
            S.hist[i] = atomicExch(&P.ghist[size_t(s) * LT_ROW + i], 0u);
        __syncthreads();
        const uint32_t r = PS == 0 ? P.layer_k0[s + 1] - P.layer_k0[s] : st.y;
        lt_block_find<(PS < 3)>(S, nbins, r);
        if (tid == 0) {
            const uint32_t bin = S.res[0];
            if (bin == LT_NOSPLIT) {
                atomicCAS(P.ctrl + 1, DEV_OK, DEV_INTERNAL);               // counts and keep[] disagree
            } else {
                if (PS < 3) st.x = PS == 0 ? bin : (st.x << 10) | bin;
                else st.w = PS == 3 ? bin : (st.w << 10) | bin;
                st.y = r - S.res[1];
                if (PS == 2) {
                    st.z = S.res[2] > st.y ? 1u : 0u;                      // more coordinates with key == T than are kept
                    st.w = st.z ? 0u : LT_NOSPLIT;
                    if (st.z) atomicOr(P.tie_flag, 1u);
                }
                P.lstate[s] = st;
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < LT_BINS; i += LT_THREADS) S.hist[i] = 0;
    }
    __syncthreads();
}

// The per-layer state of the layers this block's range touches, into shared memory.
__device__ __forceinline__ void lt_load_state(const LayerTopkParams& P, LayerTopkShared& S, uint32_t lf, uint32_t ll) {
    for (uint32_t s = lf + threadIdx.x; s <= ll; s += LT_THREADS) {
        const uint4 st = __ldcg(&P.lstate[s]);
        S.x[s] = st.x;
        S.w[s] = st.z ? st.w : LT_NOSPLIT;
    }
    __syncthreads();
}

template <bool VEC>
__global__ void __launch_bounds__(LT_THREADS, LT_BLOCKS_PER_SM) layer_topk_kernel(const LayerTopkParams P) {
    extern __shared__ __align__(16) unsigned char lt_smem[];
    LayerTopkShared& S = *reinterpret_cast<LayerTopkShared*>(lt_smem);
    const uint32_t tid = threadIdx.x, lane = lane_id();
    const uint32_t nblocks = gridDim.x, d = P.d;
    GridBarrier gb;
    gb.arrive = P.barrier; gb.nblocks = nblocks; gb.status = P.ctrl + 1; gb.spin_limit = P.spin_limit;
    span_begin(P.spans);

    for (uint32_t i = tid; i <= P.nl; i += LT_THREADS) S.off[i] = P.layer_off[i];
    for (uint32_t i = tid; i < LT_BINS; i += LT_THREADS) S.hist[i] = 0;
    // this block's contiguous range of spans and the layers it touches
    const uint32_t nspans = (d + LT_SPAN - 1) / LT_SPAN;
    const uint32_t span_lo = uint32_t(uint64_t(blockIdx.x) * nspans / nblocks);
    const uint32_t span_hi = uint32_t(uint64_t(blockIdx.x + 1) * nspans / nblocks);
    __syncthreads();
    const bool have = span_lo < span_hi;
    const uint32_t lf = have ? layer_of(S.off, P.nl, span_lo * LT_SPAN) : 0u;
    const uint32_t ll = have ? layer_of(S.off, P.nl, min(span_hi * LT_SPAN, d) - 1u) : 0u;
    // tile counts are accumulated with atomics in the marking pass
    for (size_t i = size_t(blockIdx.x) * LT_THREADS + tid; i <= P.ntiles; i += size_t(nblocks) * LT_THREADS)
        P.tile_prefix[i] = 0;

    // phase time stamps of block 0 (low word of the nanosecond global timer), for profiling only
#define LT_STAMP(i) do { if (blockIdx.x == 0 && tid == 0) { uint32_t ts_; asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(ts_)); \
                                                            P.ctrl[8 + (i)] = ts_; } } while (0)
    LT_STAMP(0);
    // ---------------- three rounds over the magnitude key ---------------------------------------------
    lt_stream_pass<0, VEC>(P, S, span_lo, span_hi, lf);
    LT_STAMP(1);
    if (!grid_barrier(gb, &S.flag)) return;
    LT_STAMP(2);
    lt_find_round<0>(P, S);
    LT_STAMP(3);
    if (!grid_barrier(gb, &S.flag)) return;
    if (have) lt_load_state(P, S, lf, ll);
    LT_STAMP(4);
    lt_stream_pass<1, VEC>(P, S, span_lo, span_hi, lf);
    LT_STAMP(5);
    if (!grid_barrier(gb, &S.flag)) return;
    lt_find_round<1>(P, S);
    if (!grid_barrier(gb, &S.flag)) return;
    if (have) lt_load_state(P, S, lf, ll);
    LT_STAMP(6);
    lt_stream_pass<2, VEC>(P, S, span_lo, span_hi, lf);
    LT_STAMP(7);
    if (!grid_barrier(gb, &S.flag)) return;
    lt_find_round<2>(P, S);
    if (!grid_barrier(gb, &S.flag)) return;
    if (have) lt_load_state(P, S, lf, ll);
    LT_STAMP(8);

    // ---------------- ties across a layer's boundary: three rounds over the offset ---------------------
    if (__ldcg(P.tie_flag) != 0u) {                                          // the same answer in every block
        lt_stream_pass<3, VEC>(P, S, span_lo, span_hi, lf);
        if (!grid_barrier(gb, &S.flag)) return;
        lt_find_round<3>(P, S);
        if (!grid_barrier(gb, &S.flag)) return;
        if (have) lt_load_state(P, S, lf, ll);
        lt_stream_pass<4, VEC>(P, S, span_lo, span_hi, lf);
        if (!grid_barrier(gb, &S.flag)) return;
        lt_find_round<4>(P, S);
        if (!grid_barrier(gb, &S.flag)) return;
        if (have) lt_load_state(P, S, lf, ll);
        lt_stream_pass<5, VEC>(P, S, span_lo, span_hi, lf);
        if (!grid_barrier(gb, &S.flag)) return;
        lt_find_round<5>(P, S);
        if (!grid_barrier(gb, &S.flag)) return;
        if (have) lt_load_state(P, S, lf, ll);
    }

    // ---------------- mark: bitmap words and per-tile counts --------------------------------------------
    uint32_t mine = 0;                                                       // coordinates this thread selected
    {
        uint32_t cur = lf;
        for (uint32_t sp0 = span_lo; sp0 < span_hi; sp0 += LT_UNROLL) {
            float gv[LT_UNROLL][4], mv[LT_UNROLL][4];
            lt_load_spans<VEC>(P, sp0, span_hi, gv, mv);
#pragma unroll
            for (int u = 0; u < LT_UNROLL; ++u) {
                const uint32_t sp = sp0 + u;
                if (sp >= span_hi) break;                                    // uniform
                const uint32_t p = sp * LT_SPAN + tid * 4u;
                uint32_t nib = 0;
                if (p < d) {
                    while (p >= S.off[cur + 1]) ++cur;
                    uint32_t s = cur;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t pc = p + c;
                        if (pc >= d) break;
                        while (pc >= S.off[s + 1]) ++s;
                        const uint32_t key = mag_key(__fadd_rn(mv[u][c], gv[u][c]));
                        const uint32_t T = S.x[s], w = S.w[s];
                        if (key > T || (key == T && (w == LT_NOSPLIT || pc - S.off[s] <= w))) nib |= 1u << c;
                    }
                }
                // eight neighbouring threads make one bitmap word
                uint32_t word = nib << ((lane & 7u) * 4u);
                word |= __shfl_xor_sync(FULL, word, 1);
                word |= __shfl_xor_sync(FULL, word, 2);
                word |= __shfl_xor_sync(FULL, word, 4);
                const uint32_t widx = sp * (LT_SPAN / 32u) + (tid >> 3);
                if ((lane & 7u) == 0u && widx < P.ntiles * 32u) P.bitmap[widx] = word;
                const uint32_t wcnt = warp_sum(__popc(nib));                 // a warp lies inside one tile
                const uint32_t tile = sp * 2u + (tid >> 8);
                if (lane == 0 && wcnt && tile < P.ntiles) atomicAdd(&P.tile_prefix[tile], wcnt);
                mine += __popc(nib);
            }
        }
    }
    {
        uint32_t total;
        lt_block_excl_scan(mine, S.wtot, &total);
        if (tid == 0) P.block_tot[blockIdx.x] = total;
    }
    LT_STAMP(9);
    if (!grid_barrier(gb, &S.flag)) return;
    LT_STAMP(10);

    // ---------------- per-tile counts -> prefix counts (each block its own tiles) -------------------------
    if (tid < 32) {
        uint32_t b = 0;
        for (uint32_t i = lane; i < blockIdx.x; i += 32) b += __ldcg(&P.block_tot[i]);
        b = warp_sum(b);
        if (lane == 0) S.base = b;
    }
    __syncthreads();
    uint32_t running = S.base;
    const uint32_t t_lo = min(span_lo * 2u, P.ntiles), t_hi = min(span_hi * 2u, P.ntiles);
    for (uint32_t t0 = t_lo; t0 < t_hi; t0 += LT_THREADS) {
        const uint32_t tile = t0 + tid;
        const uint32_t cnt = tile < t_hi ? __ldcg(&P.tile_prefix[tile]) : 0u;
        uint32_t total;
        const uint32_t excl = lt_block_excl_scan(cnt, S.wtot, &total);
        if (tile < t_hi) P.tile_prefix[tile] = running + excl;
        running += total;
    }
    if (blockIdx.x == nblocks - 1 && tid == 0) {
        P.tile_prefix[P.ntiles] = P.k;
        if (running != P.k) atomicCAS(P.ctrl + 1, DEV_OK, DEV_INTERNAL);     // the layers did not add up to k
        P.ctrl[2] = 4u;                                                      // path 4: exact top-k per layer
        P.ctrl[3] = P.k;
        *P.tie_flag = 0u;                                                    // every block read it before the last barrier
    }
    // ---------------- the ascending index list, if asked for -----------------------------------------------
    if (P.out_idx) {
        __syncthreads();                                                     // this block's prefix counts and bitmap words
        for (uint32_t tile = t_lo + (tid >> 5); tile < t_hi; tile += LT_THREADS / 32) {
            uint32_t word = P.bitmap[size_t(tile) * 32 + lane];
            const uint32_t cnt = __popc(word);
            uint32_t r = P.tile_prefix[tile] + warp_incl_scan(cnt) - cnt;
            while (word) {
                const uint32_t b = __ffs(word) - 1u;
                if (r < P.k) P.out_idx[r] = int32_t(tile * TILE + lane * 32u + b);
                ++r;
                word &= word - 1u;
            }
        }
    }
    LT_STAMP(11);
#undef LT_STAMP
    span_end(P.spans);
}

}  // namespace sc
