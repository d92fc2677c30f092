// Exact top-k inside every layer: Eq. 2 applied to each layer on its own, with Section 4's per-layer
// compression rates (layer s keeps keep[s] of its size[s] coordinates; ties go to the lower index).
//
// One persistent cooperative kernel.  All layers are searched at once by a most-significant-digit
// radix select over the 31-bit magnitude key, 11 + 10 + 10 bits.  A round is
//   count   the digit of every coordinate that still matches its layer's prefix goes into the layer's
//           row of a global histogram
//   find    layer s is looked at by block s mod grid: the digit where the count from the top reaches
//           what the layer still has to keep extends its prefix; the row is left zero.  When the digit's
//           own count is exactly what is left to keep, the layer is done: every key >= T is kept
// After three rounds a layer is done, or it has more coordinates with key == T than it may keep (a tie
// across the boundary); for those, three more rounds over the offset inside the layer, from the bottom,
// end with the largest offset that is still kept.
//
// Two routes share these rounds:
//   collecting (the usual one)  the first count streams g and m (blocks own contiguous ranges of 2048-coordinate
//           spans and count in shared memory); a second streaming pass classifies every coordinate against
//           its layer's first digit: above it -> selected (bitmap word written), equal -> undecided, kept as
//           (key, index) in a segment owned by the warp; all later rounds run over these few per cent only.
//           2 passes x 8 B per coordinate.
//   streaming (a warp's segment overflowed: many equal or near-equal magnitudes)  every round and the final
//           marking stream g and m again: 4 passes (7 with ties) x 8 B per coordinate.
#pragma once
#include "chunk_select.cuh"   // layer_of, CS_MAX_LAYERS
#include "common.cuh"

namespace sc {

constexpr int LT_THREADS = 512;
constexpr int LT_WARPS = LT_THREADS / 32;
constexpr int LT_BLOCKS_PER_SM = 2;
constexpr int LT_UNROLL = 2;             // spans whose loads a thread has in flight
constexpr uint32_t LT_SPAN = LT_THREADS * 4;        // coordinates a block takes per iteration (two tiles)
constexpr uint32_t LT_BINS = 2048;                  // widest digit: 11 bits
// Per-layer marker in shared memory (S.w): the key rounds are still running / the layer is done (keep every
// key >= T) / anything below 2^31: prefix of, and finally, the last kept offset among the keys equal to T.
constexpr uint32_t LT_NOSPLIT = 0xFFFFFFFFu;
constexpr uint32_t LT_DONE = 0xFFFFFFFEu;
// Words between two layers' rows of the global histogram: an odd number of 128-byte lines, so that the same
// bin of different layers does not sit a power of two apart.
constexpr uint32_t LT_ROW = LT_BINS + 32;
// Selection paths reported in ctrl[2]
constexpr uint32_t LT_PATH_COLLECT = 4, LT_PATH_STREAM = 5;

struct LayerTopkParams {
    const float* g;
    const float* m;
    uint32_t d, k;
    uint32_t spin_limit;
    uint32_t force_stream;              // 1: take the streaming route from the start (testing)
    uint32_t nl;
    const uint32_t* layer_off;          // [nl + 1] first coordinate of each layer
    const uint32_t* layer_k0;           // [nl + 1] prefix sums of keep[]
    uint32_t* ghist;                    // [nl * LT_ROW], zero on entry, left zero
    uint4* lstate;                      // [nl] {prefix or T, still to keep, flags (1 tie to split, 2 done), offset prefix}
    uint32_t* ctl;                      // [0] some layer has a tie to split, [1] a segment overflowed; zero on entry, left zero
    uint32_t* block_tot;                // [grid]
    uint2* cand;                        // [grid * LT_WARPS * seg_cap] undecided (key, index), one segment per warp
    uint32_t seg_cap;
    uint32_t* bitmap;                   // [ntiles * 32]
    uint32_t* tile_prefix;              // [ntiles + 1]
    uint32_t ntiles;
    uint32_t* ctrl;                     // status word at [1], path at [2], count at [3], phase stamps from [8]
    unsigned long long* barrier;        // arrival counter used by this kernel only
    int32_t* out_idx;                   // [k] or nullptr
    unsigned long long* spans;
};

struct LayerTopkShared {
    uint32_t off[CS_MAX_LAYERS + 1];    // layer starts
    uint32_t x[CS_MAX_LAYERS];          // per layer: key prefix, finally T
    uint32_t w[CS_MAX_LAYERS];          // per layer: LT_NOSPLIT, LT_DONE, or offset prefix / last kept offset
    uint32_t hist[LT_BINS];
    uint32_t wtot[LT_WARPS];
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
    for (int i = 0; i < LT_WARPS; ++i) {
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
// x, w: the layer's S.x and S.w.
template <int PS>
__device__ __forceinline__ bool lt_match(uint32_t key, uint32_t o, uint32_t x, uint32_t w, uint32_t* dg) {
    if (PS == 0) { *dg = key >> 20; return true; }
    if (PS == 1) { *dg = (key >> 10) & 1023u; return w == LT_NOSPLIT && (key >> 20) == x; }
    if (PS == 2) { *dg = key & 1023u; return w == LT_NOSPLIT && (key >> 10) == x; }
    if (PS == 3) { *dg = o >> 20; return w < LT_DONE && key == x; }
    if (PS == 4) { *dg = (o >> 10) & 1023u; return w < LT_DONE && key == x && (o >> 20) == w; }
    *dg = o & 1023u;
    return w < LT_DONE && key == x && (o >> 10) == w;
}

// Once all rounds are over: is the coordinate kept?
__device__ __forceinline__ bool lt_selected(uint32_t key, uint32_t o, uint32_t T, uint32_t w) {
    return w == LT_DONE ? key >= T : (key > T || (key == T && o <= w));
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
            for (uint32_t s = cf; s <= cl; ++s) any = any || S.w[s] < LT_DONE;
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

// Eight neighbouring threads' nibbles make one bitmap word; complete in the lane with (lane & 7) == 0.
__device__ __forceinline__ uint32_t lt_word_of(uint32_t nib) {
    uint32_t word = nib << ((lane_id() & 7u) * 4u);
    word |= __shfl_xor_sync(FULL, word, 1);
    word |= __shfl_xor_sync(FULL, word, 2);
    word |= __shfl_xor_sync(FULL, word, 4);
    return word;
}

// The second streaming pass of the collecting route: every coordinate against its layer's first digit.
// Above -> selected, equal -> this warp's segment, below -> dropped; in a layer that is already done the key
// is compared with T.  Returns the number of entries in the warp's segment (warp-uniform); an overflow sets
// ctl[1] and stops the appending (the count then no longer matters).
template <bool VEC>
__device__ __forceinline__ uint32_t lt_classify_pass(const LayerTopkParams& P, LayerTopkShared& S, uint32_t span_lo,
                                                     uint32_t span_hi, uint32_t layer_first, uint2* seg) {
    const uint32_t tid = threadIdx.x, lane = lane_id(), d = P.d;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t cur = layer_first, nseg = 0;
    bool full = false;                                                      // warp-uniform
    for (uint32_t sp0 = span_lo; sp0 < span_hi; sp0 += LT_UNROLL) {
        float gv[LT_UNROLL][4], mv[LT_UNROLL][4];
        lt_load_spans<VEC>(P, sp0, span_hi, gv, mv);
#pragma unroll
        for (int u = 0; u < LT_UNROLL; ++u) {
            const uint32_t sp = sp0 + u;
            if (sp >= span_hi) break;                                       // uniform
            const uint32_t p = sp * LT_SPAN + tid * 4u;
            uint32_t nib = 0, und = 0, keys[4] = {0u, 0u, 0u, 0u};
            if (p < d) {
                while (p >= S.off[cur + 1]) ++cur;
                uint32_t s = cur;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t pc = p + c;
                    if (pc >= d) break;
                    while (pc >= S.off[s + 1]) ++s;
                    const uint32_t key = mag_key(__fadd_rn(mv[u][c], gv[u][c]));
                    const uint32_t x = S.x[s];
                    keys[c] = key;
                    if (S.w[s] == LT_DONE) {
                        if (key >= x) nib |= 1u << c;
                    } else if ((key >> 20) > x) {
                        nib |= 1u << c;
                    } else if ((key >> 20) == x) {
                        und |= 1u << c;
                    }
                }
            }
            const uint32_t word = lt_word_of(nib);
            const uint32_t widx = sp * (LT_SPAN / 32u) + (tid >> 3);
            if ((lane & 7u) == 0u && widx < P.ntiles * 32u) P.bitmap[widx] = word;
            // the undecided ones go to the warp's segment (most quad rows of a strongly compressed layer have none)
            if (__ballot_sync(FULL, und != 0u) == 0u) continue;             // warp-uniform
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t bal = __ballot_sync(FULL, (und >> c) & 1u);
                if (bal == 0u || full) continue;                            // warp-uniform
                const uint32_t add = __popc(bal);
                if (nseg + add > P.seg_cap) {
                    full = true;
                    if (lane == 0) atomicOr(&P.ctl[1], 1u);
                    continue;
                }
                if ((und >> c) & 1u) seg[nseg + __popc(bal & lt_mask)] = make_uint2(keys[c], p + c);
                nseg += add;
            }
        }
    }
    return nseg;
}

// Round PS of the collecting route: this warp's undecided coordinates into the rows.  A block whose range
// lies inside one layer (the usual case for large layers) counts in shared memory and adds the sums once.
template <int PS>
__device__ __forceinline__ void lt_cand_round(const LayerTopkParams& P, LayerTopkShared& S, const uint2* seg,
                                              uint32_t nseg, uint32_t lf, uint32_t ll) {
    const bool one = lf == ll;                                              // uniform
    for (uint32_t i = lane_id(); i < nseg; i += 32u) {
        const uint2 e = seg[i];
        const uint32_t s = one ? lf : lf + layer_of(S.off + lf, ll - lf + 1u, e.y);
        uint32_t dg;
        if (lt_match<PS>(e.x, e.y - S.off[s], S.x[s], S.w[s], &dg)) {
            if (one) atomicAdd(&S.hist[dg], 1u);
            else atomicAdd(&P.ghist[size_t(s) * LT_ROW + dg], 1u);
        }
    }
    if (one) lt_flush(S, P.ghist, lf);
}

// Round PS for the layers this block looks after: extend the prefix from the layer's global row.
template <int PS>
__device__ __forceinline__ void lt_find_round(const LayerTopkParams& P, LayerTopkShared& S) {
    const uint32_t tid = threadIdx.x;
    constexpr uint32_t nbins = (PS == 0 || PS == 3) ? 2048u : 1024u;
    for (uint32_t s = blockIdx.x; s < P.nl; s += gridDim.x) {
        uint4 st = make_uint4(0, 0, 0, 0);
        if (PS > 0) st = __ldcg(&P.lstate[s]);
        if (PS > 0 && PS < 3 && (st.z & 2u)) continue;                     // uniform: the layer is done
        if (PS >= 3 && !(st.z & 1u)) continue;                             // uniform: no tie to split in this layer
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
            } else if (PS < 3) {
                const uint32_t prefix = PS == 0 ? bin : (st.x << 10) | bin;
                st.y = r - S.res[1];                                       // to keep among the keys with this prefix
                if (S.res[2] == st.y) {                                    // all of them: every key >= the lowest such key
                    st.x = prefix << (PS == 0 ? 20 : PS == 1 ? 10 : 0);
                    st.z = 2u;
                } else if (PS == 2) {                                      // more keys equal to T than may be kept
                    st.x = prefix;
                    st.z = 1u;
                    st.w = 0u;
                    atomicOr(&P.ctl[0], 1u);
                } else {
                    st.x = prefix;
                    st.z = 0u;
                }
                P.lstate[s] = st;
            } else {
                st.w = PS == 3 ? bin : (st.w << 10) | bin;
                st.y = r - S.res[1];
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
        S.w[s] = (st.z & 2u) ? LT_DONE : (st.z & 1u) ? st.w : LT_NOSPLIT;
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
    const uint32_t t_lo = min(span_lo * 2u, P.ntiles), t_hi = min(span_hi * 2u, P.ntiles);   // and of tiles
    __syncthreads();
    const bool have = span_lo < span_hi;
    const uint32_t lf = have ? layer_of(S.off, P.nl, span_lo * LT_SPAN) : 0u;
    const uint32_t ll = have ? layer_of(S.off, P.nl, min(span_hi * LT_SPAN, d) - 1u) : 0u;
    // (the streaming route accumulates tile counts with atomics)
    for (size_t i = size_t(blockIdx.x) * LT_THREADS + tid; i <= P.ntiles; i += size_t(nblocks) * LT_THREADS)
        P.tile_prefix[i] = 0;
    uint2* const seg = P.cand + (size_t(blockIdx.x) * LT_WARPS + (tid >> 5)) * P.seg_cap;

    // phase time stamps of block 0 (low word of the nanosecond global timer), for profiling only
#define LT_STAMP(i) do { if (blockIdx.x == 0 && tid == 0) { uint32_t ts_; asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(ts_)); \
                                                            P.ctrl[8 + (i)] = ts_; } } while (0)
#define LT_BARRIER() do { if (!grid_barrier(gb, &S.flag)) return; } while (0)
#define LT_LOAD() do { if (have) lt_load_state(P, S, lf, ll); } while (0)
    LT_STAMP(0);
    // ---------------- first digit of every layer --------------------------------------------------------------
    lt_stream_pass<0, VEC>(P, S, span_lo, span_hi, lf);
    LT_STAMP(1);
    LT_BARRIER();
    lt_find_round<0>(P, S);
    LT_BARRIER();
    LT_LOAD();
    LT_STAMP(2);

    uint32_t mine = 0;                                                       // coordinates this thread counted as selected
    bool stream = P.force_stream != 0u;
    if (!stream) {
        // ---------------- collecting route ---------------------------------------------------------------------
        const uint32_t nseg = lt_classify_pass<VEC>(P, S, span_lo, span_hi, lf, seg);
        LT_STAMP(3);
        __syncwarp();
        lt_cand_round<1>(P, S, seg, nseg, lf, ll);
        LT_BARRIER();
        stream = __ldcg(&P.ctl[1]) != 0u;                                    // the same answer in every block
        if (!stream) {
            lt_find_round<1>(P, S);
            LT_BARRIER();
            LT_LOAD();
            lt_cand_round<2>(P, S, seg, nseg, lf, ll);
            LT_BARRIER();
            lt_find_round<2>(P, S);
            LT_BARRIER();
            LT_LOAD();
            LT_STAMP(4);
            if (__ldcg(&P.ctl[0]) != 0u) {                                   // the same answer in every block
                lt_cand_round<3>(P, S, seg, nseg, lf, ll);
                LT_BARRIER();
                lt_find_round<3>(P, S);
                LT_BARRIER();
                LT_LOAD();
                lt_cand_round<4>(P, S, seg, nseg, lf, ll);
                LT_BARRIER();
                lt_find_round<4>(P, S);
                LT_BARRIER();
                LT_LOAD();
                lt_cand_round<5>(P, S, seg, nseg, lf, ll);
                LT_BARRIER();
                lt_find_round<5>(P, S);
                LT_BARRIER();
                LT_LOAD();
            }
            LT_STAMP(5);
            // the undecided ones that are kept after all, then the count of every tile of this block's range
            for (uint32_t i = lane; i < nseg; i += 32u) {
                const uint2 e = seg[i];
                const uint32_t s = lf + layer_of(S.off + lf, ll - lf + 1u, e.y);
                if (lt_selected(e.x, e.y - S.off[s], S.x[s], S.w[s])) atomicOr(&P.bitmap[e.y >> 5], 1u << (e.y & 31u));
            }
            __syncthreads();
            for (uint32_t tile = t_lo + (tid >> 5); tile < t_hi; tile += LT_WARPS) {
                const uint32_t cnt = warp_sum(__popc(__ldcg(&P.bitmap[size_t(tile) * 32 + lane])));
                if (lane == 0) {
                    P.tile_prefix[tile] = cnt;
                    mine += cnt;
                }
            }
        } else {
            // a segment overflowed: the rows hold part of the second count and are cleared before the streaming route starts
            for (uint32_t s = blockIdx.x; s < P.nl; s += nblocks)
                for (uint32_t i = tid; i < LT_BINS; i += LT_THREADS) P.ghist[size_t(s) * LT_ROW + i] = 0u;
            LT_BARRIER();
        }
    }
    if (stream) {
        // ---------------- streaming route ------------------------------------------------------------------------
        lt_stream_pass<1, VEC>(P, S, span_lo, span_hi, lf);
        LT_BARRIER();
        lt_find_round<1>(P, S);
        LT_BARRIER();
        LT_LOAD();
        lt_stream_pass<2, VEC>(P, S, span_lo, span_hi, lf);
        LT_BARRIER();
        lt_find_round<2>(P, S);
        LT_BARRIER();
        LT_LOAD();
        LT_STAMP(4);
        if (__ldcg(&P.ctl[0]) != 0u) {                                       // the same answer in every block
            lt_stream_pass<3, VEC>(P, S, span_lo, span_hi, lf);
            LT_BARRIER();
            lt_find_round<3>(P, S);
            LT_BARRIER();
            LT_LOAD();
            lt_stream_pass<4, VEC>(P, S, span_lo, span_hi, lf);
            LT_BARRIER();
            lt_find_round<4>(P, S);
            LT_BARRIER();
            LT_LOAD();
            lt_stream_pass<5, VEC>(P, S, span_lo, span_hi, lf);
            LT_BARRIER();
            lt_find_round<5>(P, S);
            LT_BARRIER();
            LT_LOAD();
        }
        LT_STAMP(5);
        // mark: bitmap words and per-tile counts
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
                        if (lt_selected(key, pc - S.off[s], S.x[s], S.w[s])) nib |= 1u << c;
                    }
                }
                const uint32_t word = lt_word_of(nib);
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
    LT_STAMP(6);
    LT_BARRIER();
    LT_STAMP(7);

    // ---------------- per-tile counts -> prefix counts (each block its own tiles) -------------------------
    if (tid < 32) {
        uint32_t b = 0;
        for (uint32_t i = lane; i < blockIdx.x; i += 32) b += __ldcg(&P.block_tot[i]);
        b = warp_sum(b);
        if (lane == 0) S.base = b;
    }
    __syncthreads();
    uint32_t running = S.base;
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
        P.ctrl[2] = stream ? LT_PATH_STREAM : LT_PATH_COLLECT;
        P.ctrl[3] = P.k;
        P.ctl[0] = 0u;                                                       // every block read both before the last barrier
        P.ctl[1] = 0u;
    }
    // ---------------- the ascending index list, if asked for -----------------------------------------------
    if (P.out_idx) {
        __syncthreads();                                                     // this block's prefix counts and bitmap words
        for (uint32_t tile = t_lo + (tid >> 5); tile < t_hi; tile += LT_WARPS) {
            uint32_t word = __ldcg(&P.bitmap[size_t(tile) * 32 + lane]);
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
    LT_STAMP(8);
#undef LT_STAMP
#undef LT_BARRIER
#undef LT_LOAD
    span_end(P.spans);
}

}  // namespace sc
