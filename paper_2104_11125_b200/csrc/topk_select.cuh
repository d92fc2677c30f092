// Leader top-k (Eq. 2): one persistent cooperative kernel.
//
// Selects the k coordinates of acc = m + g (computed on the fly, never stored)
// that come first in the order "larger |acc| first, lower index first", and
// leaves the result in three forms: a d-bit bitmap, the per-tile prefix counts
// of that bitmap, and the ascending index list.
//
// Fast path (one streaming read of g and m):
//   P0  histogram a strided sample of the keys (top 13 bits)
//   P1  every block derives from the sample a conservative lower bound on the
//       k-th key (bin b_lo), aiming at slightly more than k survivors.
//       P0/P1 are skipped when earlier launches of the same handle left a
//       hint: the bin of this leader's k-th key the last time it led, moved by what the
//       previous step's leader saw change over the same interval (else the previous
//       step's bin), minus a margin.  A hint that turns out useless
//       costs one wasted pass; the step then runs P0/P1 as if there had been none,
//       and later hints of the handle keep one more bin of distance
//   P2  stream g, m once.  A survivor (key bin >= b_lo) is appended as (key, idx)
//       to a candidate segment owned by the warp that found it -- no atomics, no
//       staging; slots come from a warp ballot.  Survivor keys also pass through a
//       small per-warp ring in shared memory from which, 32 at a time and with all
//       lanes busy, they are added to two histograms (13-bit bins in a 64-bin
//       window above b_lo, per block in shared memory; 22-bit prefixes, global)
//   P3  the two histograms fix the first 22 bits of the k-th key: candidates
//       above that prefix are winners, the few hundred sharing it form the
//       boundary group
//   P4  every warp marks the winners of its own segment in the bitmap and appends
//       boundary members to a short global list
//   P5  every block ranks the boundary list exactly (by key, then lower index),
//       takes the winners that fall in its own span, and prefix-scans its span of
//       the bitmap: tile prefixes + ascending indices.  The scratch arrays are
//       cleared here for the next launch
// A boundary group too large for the short list (heavy ties) is resolved by a
// radix select over the candidate segments instead (one pass per digit).
// Exact path (taken when a candidate segment overflowed, too few survived, or
// the k-th key left the histogram window; also on request): the same radix
// select with every pass streaming g and m again (up to six passes) and a mark
// pass.  Correctness never depends on the sample or on the hint.
#pragma once
#include "common.cuh"

namespace sc {

constexpr int TK_THREADS = 512;
constexpr int TK_BLOCKS_PER_SM = 2;
constexpr int TK_WARPS = TK_THREADS / 32;
static_assert(TK_WARPS >= 16 && TK_WARPS <= 32, "the block-wide bin search needs 16..32 warps per block");
constexpr int TK_UNROLL = 4;                        // quads of g and of m in flight per thread
constexpr uint32_t TK_CHUNK = TK_THREADS * 4 * TK_UNROLL;      // coordinates per block iteration (8192)
constexpr uint32_t TK_UNIT = TK_THREADS * 4;                   // coordinates one block covers with one quad per thread

constexpr int COARSE_SHIFT = 18;                               // key >> 18: 13-bit coarse bin
constexpr uint32_t NCOARSE = 1u << 13;
constexpr int FINE_SHIFT = 9;                                  // key >> 9: 22-bit fine prefix
constexpr uint32_t WIN = 64;                                   // coarse bins covered above b_lo
constexpr uint32_t NFINE = WIN * 512;
constexpr uint32_t LOCAL_CB = NCOARSE / 512;                   // coarse bins above the bound whose fine bins a block counts in shared memory
constexpr uint32_t DH_BINS = 2048;                             // digit histogram of one radix pass
constexpr uint32_t DH_PASSES = 8;
constexpr uint32_t SAMPLE_GRANULE = 128;                       // coordinates one warp samples at a time
constexpr uint32_t BCAP = 1024;                                // boundary list entries
constexpr double KEEP_SHARE = 0.25;                            // largest share of the leader's lines held in L2 for the learner pass
constexpr double KEEP_SHARE_MIN = 0.05;                        // and the smallest worth marking the stream for

// ctrl words
constexpr int CT_CAND = 0, CT_STATUS = 1, CT_PATH = 2, CT_M = 3, CT_BCOUNT = 4, CT_OVERFLOW = 5, CT_HINT = 6, CT_MARGIN = 7;
constexpr int CT_DRIFT = 21;                                   // (words 8 .. 20 are the phase stamps)
constexpr int CT_PEER_DONE = 22;                               // finished blocks of a signalling single-learner pass
constexpr int CT_STAMP = 8, CT_NSTAMPS = 13, CT_WORDS = 32;
// selection paths reported in ctrl[CT_PATH]
constexpr uint32_t PATH_FAST = 0, PATH_EXACT = 1, PATH_FAST_HINT = 2;

struct TopkParams {
    const float* g;            // leader's gradient, fp32[d]
    const float* m;            // leader's memory, fp32[d]
    uint32_t d, k;
    uint32_t samp_stride;      // sample one granule out of this many
    uint32_t samp_target;      // wanted number of sampled keys at or above the bound
    uint32_t force_exact;
    uint32_t use_hint;         // 1: start from the bound earlier launches left behind
    uint32_t* leader_hint;     // this leader's own entry (bin + 1 of its last threshold, 0 = none), or nullptr
    uint32_t* all_hints;       // every leader's entry [n_hints] (or nullptr): forgotten when a hint turns out useless
    uint32_t n_hints;
    uint32_t spin_limit;
    float keep_frac;           // share of the leader's lines asked to stay in L2 for the kernel that reads them next (0: none)
    // the four histograms are all zero on entry and all zero again on exit
    uint32_t* samp_hist;       // [NCOARSE]
    uint32_t* coarse_win;      // [WIN + 1]
    uint32_t* fine_hist;       // [NFINE]
    uint32_t* fine_hist_next;  // [NFINE] the copy the next launch will use, cleared here behind the stream (or nullptr:
                               //         this launch clears its own copy at the end)
    uint32_t* digit_hist;      // [DH_PASSES * DH_BINS]
    uint32_t* block_tot;       // [gridDim.x] winners per block span
    uint32_t* ctrl;            // [CT_WORDS]
    unsigned long long* barrier;   // arrival counter of the grid barrier
    uint2* cand;               // [seg_cap * warps in the grid] (key, idx), one segment per warp
    uint32_t seg_cap;          // entries per warp segment
    uint2* blist;              // [BCAP] boundary group
    uint32_t* bitmap;          // [ntiles * 32]
    uint32_t* tile_prefix;     // [ntiles + 1]
    uint32_t ntiles;
    uint32_t tiles_per_block;  // span of the final scan
    int32_t* out_idx;          // [k], or nullptr when the caller derives the index list itself
    unsigned long long* spans;     // nullptr, or where to accumulate the kernel's time span
};

struct TopkShared {
    uint32_t hist[NCOARSE];            // sample histogram / span counters / digit histogram / boundary list
    uint32_t ring[TK_WARPS][64];       // survivor keys waiting for a lane-dense histogram update
    uint32_t cw[WIN + 1];              // this block's share of the coarse window histogram
    uint32_t scan[32];
    uint32_t res[4];
    uint32_t mcount;                   // survivors found by this block
    uint32_t own_n;                    // boundary winners inside this block's span
    int flag;
};

// Block-wide search from the top of a histogram of nb <= TK_THREADS bins held one bin per thread: thread r holds
// v = h[nb - 1 - r] (0 for r >= nb).  Finds the bin holding the `need`-th element counted from the top:
// s.res = {bin, count strictly above bin, count in bin}, bin = 0xFFFFFFFF when the histogram holds fewer.
// (Shared: any shared-memory struct with scan[32] and res[4].)
template <class Shared>
__device__ inline void find_in_regs(uint32_t v, uint32_t nb, uint32_t need, Shared& s) {
    const uint32_t lane = lane_id(), warp = warp_id(), r = threadIdx.x;
    if (threadIdx.x == 0) s.res[0] = 0xFFFFFFFFu;
    const uint32_t incl = warp_incl_scan(v);
    if (lane == 31) s.scan[warp] = incl;
    __syncthreads();
    uint32_t before = incl - v;
#pragma unroll
    for (int w = 0; w < TK_WARPS; ++w)
        if (w < (int)warp) before += s.scan[w];
    if (v && r < nb && before < need && need <= before + v) { s.res[0] = nb - 1 - r; s.res[1] = before; s.res[2] = v; }
    __syncthreads();
}

// The same for a histogram in global memory (written by other blocks before the last grid barrier) of up to 8192
// bins: TK_WARPS warp-sized segments first, then one bin per thread inside the segment that holds the answer.
template <class Shared>
__device__ inline void find_from_top(const uint32_t* h, uint32_t nb, uint32_t need, Shared& s) {
    const uint32_t lane = lane_id(), warp = warp_id();
    if (nb <= uint32_t(TK_THREADS)) {
        const uint32_t r = threadIdx.x;
        find_in_regs(r < nb ? __ldcg(h + (nb - 1 - r)) : 0u, nb, need, s);
        return;
    }
    if (threadIdx.x == 0) s.res[0] = 0xFFFFFFFFu;
    const uint32_t seglen = (nb + TK_WARPS - 1) / TK_WARPS;
    {
        const uint32_t r0 = warp * seglen, r1 = min(nb, r0 + seglen);
        uint32_t sum = 0;
        for (uint32_t r = r0 + lane; r < r1; r += 32) sum += __ldcg(h + (nb - 1 - r));
        sum = warp_sum(sum);
        if (lane == 0) s.scan[warp] = sum;
    }
    __syncthreads();
    uint32_t seg = TK_WARPS, excl = 0;
    {
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < TK_WARPS; ++w) {
            const uint32_t v = s.scan[w];
            if (seg == TK_WARPS && need <= run + v) { seg = w; excl = run; }
            run += v;
        }
    }
    __syncthreads();
    if (seg == TK_WARPS) return;                       // fewer than `need` elements (uniform across the block)
    const uint32_t s0 = seg * seglen, s1 = min(nb, s0 + seglen);
    const uint32_t sublen = (seglen + TK_WARPS - 1) / TK_WARPS;
    const uint32_t r = s0 + warp * sublen + lane;
    const bool live = lane < sublen && r < s1;
    const uint32_t v = live ? __ldcg(h + (nb - 1 - r)) : 0u;
    const uint32_t incl = warp_incl_scan(v);
    if (lane == 31) s.scan[warp] = incl;
    __syncthreads();
    uint32_t sub = TK_WARPS, excl2 = excl;
    {
        uint32_t run = excl;
#pragma unroll
        for (int w = 0; w < TK_WARPS; ++w) {
            const uint32_t t = s.scan[w];
            if (sub == TK_WARPS && need <= run + t) { sub = w; excl2 = run; }
            run += t;
        }
    }
    if (warp == sub && live) {
        const uint32_t before = excl2 + incl - v;
        if (before < need && need <= before + v) { s.res[0] = nb - 1 - r; s.res[1] = before; s.res[2] = v; }
    }
    __syncthreads();
}

// First coordinate of this block's it-th unit, or d (nothing to do) past its last unit.
__device__ __forceinline__ uint32_t unit_coord(uint32_t it, uint32_t my_units, uint32_t nblocks, uint32_t d) {
    return it < my_units ? (it * nblocks + blockIdx.x) * TK_UNIT : d;
}

__device__ inline void zero_words(uint32_t* p, size_t nwords, size_t gtid, size_t gsize) {
    // p is 16-byte aligned and nwords a multiple of 4 for the large arrays; the generic loop handles the rest
    const size_t nv = nwords / 4;
    uint4* pv = reinterpret_cast<uint4*>(p);
    for (size_t i = gtid; i < nv; i += gsize) pv[i] = make_uint4(0, 0, 0, 0);
    for (size_t i = nv * 4 + gtid; i < nwords; i += gsize) p[i] = 0;
}

// Running state of the radix select over composites (62 bits, most significant first).
struct SelState {
    uint64_t prefix;   // the nbits leading bits fixed so far
    int nbits;
    uint32_t need;     // how many more to take from the group matching prefix
    uint32_t group;    // size of that group
};

__device__ __forceinline__ bool sel_done(const SelState& st) { return st.group == st.need || st.nbits >= 62; }

template <bool VEC>
__global__ void __launch_bounds__(TK_THREADS, TK_BLOCKS_PER_SM) topk_select_kernel(const TopkParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TopkShared& s = *reinterpret_cast<TopkShared*>(smem_raw);

    const uint32_t tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    const uint32_t nblocks = gridDim.x;
    const size_t gtid = size_t(blockIdx.x) * TK_THREADS + tid;
    const size_t gsize = size_t(nblocks) * TK_THREADS;
    const uint32_t d = P.d, k = P.k;
    uint32_t* status = P.ctrl + CT_STATUS;
    GridBarrier gb;
    gb.arrive = P.barrier; gb.nblocks = nblocks; gb.status = status; gb.spin_limit = P.spin_limit;
    // this warp's candidate segment
    uint2* const seg = P.cand + size_t(blockIdx.x * TK_WARPS + warp) * P.seg_cap;
    uint32_t seg_cnt = 0;                                              // survivors this warp found (warp-uniform)
    const uint32_t lt_mask = (1u << lane) - 1u;

    // streaming phases: the vector is cut into units of TK_UNIT coordinates dealt round-robin to the
    // blocks (unit j belongs to block j mod nblocks), TK_UNROLL units per block iteration: block loads differ
    // by at most one unit, and every block sees every region of the vector (survivors cluster by layer)
    const uint32_t nunits = (d + TK_UNIT - 1) / TK_UNIT;
    const uint32_t my_units = nunits > blockIdx.x ? (nunits - blockIdx.x + nblocks - 1) / nblocks : 0u;
    const uint32_t full_units = d / TK_UNIT;                           // units 0 .. full_units-1 need no bounds checks
    const uint32_t span_coords = P.tiles_per_block * TILE;             // coordinates per block span of the final scan

    // phase time stamps of block 0 (low word of the nanosecond global timer), for profiling only
#define SC_STAMP(i) do { if (gtid == 0) { uint32_t ts_; asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(ts_)); \
                                          P.ctrl[CT_STAMP + (i)] = ts_; } } while (0)
#define SC_BARRIER() do { if (!grid_barrier(gb, &s.flag)) return; } while (0)

    span_begin(P.spans);
    SC_STAMP(0);
    SC_STAMP(1); SC_STAMP(2); SC_STAMP(3);                             // overwritten when the sample phases run

    // what must be zero before winners are marked; marking starts at least one grid barrier later
    auto clear_outputs = [&] {
        zero_words(P.bitmap, size_t(P.ntiles) * 32, gtid, gsize);
        for (size_t i = gtid; i < nblocks; i += gsize) P.block_tot[i] = 0;
        if (gtid == 0) P.ctrl[CT_BCOUNT] = 0;
        if (P.fine_hist_next) zero_words(P.fine_hist_next, NFINE, gtid, gsize);
    };

    SelState st;
    st.prefix = 0; st.nbits = 0; st.need = k; st.group = d;
    bool fast = false, used_hint = false, hint_overflowed = false;
    uint32_t b_lo = 0, M = 0;
    // Bound to start from (bin + 1, 0 = none).  The bin of the k-th key is predicted as what this leader's own
    // vector gave the last time it led (learners may differ in scale) plus the change the previous step's
    // leader saw over the same interval (the memories grow together while training warms up: without this
    // term every leader's own value is stale by n steps and the survivors overflow, again and again); a leader
    // without a value of its own starts from the previous step's.  The bound lies `margin` bins below.
    uint32_t hint = 0, hint_margin = 1;
    const uint32_t own_prev = (P.use_hint && P.leader_hint) ? __ldcg(P.leader_hint) : 0u;   // bin + 1, 0 = none
    if (!P.force_exact && P.use_hint) {
        const uint32_t prev = __ldcg(&P.ctrl[CT_HINT]);
        const int32_t margin = 1 + int32_t(__ldcg(&P.ctrl[CT_MARGIN]));
        int32_t pred = own_prev ? int32_t(own_prev - 1u) + int32_t(__ldcg(&P.ctrl[CT_DRIFT]))
                                : int32_t(prev) - 1;
        pred = min(pred, int32_t(NCOARSE) - 1);
        if (pred > margin) { hint = uint32_t(pred - margin) + 1u; hint_margin = uint32_t(margin); }
    }

    for (int attempt = hint ? 0 : 1; attempt < 2 && !P.force_exact; ++attempt) {
        if (attempt == 0) {
            b_lo = hint - 1u;
        } else {
            // ---------------- P0: sample ----------------------------------------------------------
            if (hint) {                                                // the hinted pass failed: undo what it counted
                zero_words(P.fine_hist, NFINE, gtid, gsize);
                for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
                if (gtid == 0) { P.ctrl[CT_CAND] = 0; P.ctrl[CT_OVERFLOW] = 0; }
            }
            for (uint32_t i = tid; i < NCOARSE; i += TK_THREADS) s.hist[i] = 0;
            __syncthreads();
            const uint32_t span = SAMPLE_GRANULE * P.samp_stride;      // coordinates between sampled granules
            const uint32_t ngran = (d + span - 1) / span;
            for (uint32_t gidx = blockIdx.x * TK_WARPS + warp; gidx < ngran; gidx += nblocks * TK_WARPS) {
                const uint32_t p = gidx * span + lane * 4;             // gidx*span < d
                float gv[4], mv[4];
                load_quad_stream<VEC>(P.g, p, d, gv);
                load_quad_stream<VEC>(P.m, p, d, mv);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (p + c < d) atomicAdd(&s.hist[mag_key(__fadd_rn(mv[c], gv[c])) >> COARSE_SHIFT], 1u);
            }
            __syncthreads();
            for (uint32_t i = tid; i < NCOARSE; i += TK_THREADS) {
                const uint32_t h = s.hist[i];
                if (h) atomicAdd(&P.samp_hist[i], h);
            }
            SC_STAMP(1);
            SC_BARRIER();
            SC_STAMP(2);
            // ---------------- P1: bound from the sample ----------------------------------------------
            find_from_top(P.samp_hist, NCOARSE, P.samp_target, s);
            b_lo = (s.res[0] == 0xFFFFFFFFu) ? 0u : s.res[0];
            __syncthreads();
            SC_STAMP(3);
        }
        b_lo = min(b_lo, 0x7F800000u >> COARSE_SHIFT);                 // at most the bin of +inf: the bound stays a number

        // ---------------- P2: filter pass ----------------------------------------------------------
        clear_outputs();                                               // hidden behind the stream
        for (uint32_t i = tid; i <= WIN; i += TK_THREADS) s.cw[i] = 0;
        for (uint32_t i = tid; i < LOCAL_CB * 512u; i += TK_THREADS) s.hist[i] = 0;
        if (tid == 0) s.mcount = 0;
        __syncthreads();
        seg_cnt = 0;
        uint32_t done = 0;                                             // survivors of this warp already histogrammed
        const uint32_t thr_key = b_lo << COARSE_SHIFT;
        const uint32_t fine_base = b_lo << (COARSE_SHIFT - FINE_SHIFT);
        // keys >= thr_key  <=>  !(|acc| < thr_f): one compare per element, true for NaN like the integer order
        const float thr_f = __uint_as_float(thr_key);
        uint32_t* const ring = s.ring[warp];
        // add `cnt` (<= 32) waiting survivor keys to the histograms, one per lane
        auto drain = [&](uint32_t cnt) {
            __syncwarp();
            if (lane < cnt) {
                const uint32_t key = ring[(done + lane) & 63u];
                const uint32_t cb = (key >> COARSE_SHIFT) - b_lo;
                atomicAdd(&s.cw[cb < WIN ? cb : WIN], 1u);
                // the 22-bit prefixes just above the bound -- where error feedback piles the coordinates up, a few hot bins
                // late in a run -- are counted per block in shared memory and added to the global histogram once
                if (cb < LOCAL_CB) atomicAdd(&s.hist[(key >> FINE_SHIFT) - fine_base], 1u);
                else if (cb < WIN) atomicAdd(&P.fine_hist[(key >> FINE_SHIFT) - fine_base], 1u);
            }
            done += cnt;
            __syncwarp();
        };
        // append this lane's survivors (bits of nib) of the quad at p to the warp's segment
        auto append = [&](uint32_t nib, const float (&acc)[4], uint32_t p) {
            uint32_t bal = __ballot_sync(FULL, nib != 0);
            while (bal) {                                              // every round, each lane still holding one appends it
                if (nib) {
                    const uint32_t c = __ffs(nib) - 1;
                    const float a = c == 0 ? acc[0] : c == 1 ? acc[1] : c == 2 ? acc[2] : acc[3];
                    const uint32_t slot = seg_cnt + __popc(bal & lt_mask);
                    const uint32_t key = mag_key(a);
                    if (slot < P.seg_cap) seg[slot] = make_uint2(key, p + c);
                    ring[slot & 63u] = key;
                    nib &= nib - 1;
                }
                seg_cnt += __popc(bal);
                if (seg_cnt - done >= 32u) drain(32u);                 // keeps fewer than 32 waiting: the ring never wraps
                bal = __ballot_sync(FULL, nib != 0);
            }
        };
        // L2 policy of the stream: a share of the lines is marked to be replaced last, so that the learner pass, which
        // reads the leader's g and m once more, finds them in the cache; the rest is marked to be replaced first and
        // recycles itself instead of pushing out what the previous kernel left there.
        uint64_t stream_policy;
        if (P.keep_frac > 0.0f)
            asm volatile("createpolicy.fractional.L2::evict_last.L2::evict_first.b64 %0, %1;" : "=l"(stream_policy) : "f"(P.keep_frac));
        else
            asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(stream_policy));
        for (uint32_t it0 = 0; it0 < my_units; it0 += TK_UNROLL) {
            float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
            const bool whole = VEC && it0 + TK_UNROLL <= my_units &&
                               (it0 + TK_UNROLL - 1) * nblocks + blockIdx.x < full_units;
            if (whole) {
                const uint32_t pbase = (it0 * nblocks + blockIdx.x) * TK_UNIT + tid * 4;
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = pbase + u * (nblocks * TK_UNIT);
                    const float4 a = ld_quad_policy(P.g + p, stream_policy);
                    const float4 b = ld_quad_policy(P.m + p, stream_policy);
                    gv[u][0] = a.x; gv[u][1] = a.y; gv[u][2] = a.z; gv[u][3] = a.w;
                    mv[u][0] = b.x; mv[u][1] = b.y; mv[u][2] = b.z; mv[u][3] = b.w;
                }
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = pbase + u * (nblocks * TK_UNIT);
                    float acc[4];
                    uint32_t nib = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        acc[c] = __fadd_rn(mv[u][c], gv[u][c]);
                        if (!(fabsf(acc[c]) < thr_f)) nib |= 1u << c;
                    }
                    append(nib, acc, p);
                }
            } else {
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
                    if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
                }
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
                    float acc[4];
                    uint32_t nib = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        acc[c] = __fadd_rn(mv[u][c], gv[u][c]);
                        if ((p + c < d) && !(fabsf(acc[c]) < thr_f)) nib |= 1u << c;
                    }
                    append(nib, acc, p);
                }
            }
        }
        if (seg_cnt > done) drain(seg_cnt - done);
        if (lane == 0) {
            atomicAdd(&s.mcount, seg_cnt);
            if (seg_cnt > P.seg_cap) P.ctrl[CT_OVERFLOW] = 1u;
        }
        __syncthreads();
        for (uint32_t i = tid; i <= WIN; i += TK_THREADS) {
            const uint32_t h = s.cw[i];
            if (h) atomicAdd(&P.coarse_win[i], h);
        }
        for (uint32_t i = tid; i < LOCAL_CB * 512u; i += TK_THREADS) {
            const uint32_t h = s.hist[i];
            if (h) atomicAdd(&P.fine_hist[i], h);
        }
        if (tid == 0 && s.mcount) atomicAdd(&P.ctrl[CT_CAND], s.mcount);
        SC_STAMP(4);
        SC_BARRIER();
        SC_STAMP(5);
        if (attempt == 1) zero_words(P.samp_hist, NCOARSE, gtid, gsize);   // all blocks have read it

        // ---------------- P3: locate the k-th composite -------------------------------------------
        // both levels are requested at once: the window (one bin per thread) and, on a guess of the window bin,
        // the 512 fine bins below it (right whenever the prediction behind the hint was; harmless otherwise)
        const uint32_t cb_guess = min(attempt == 0 ? hint_margin : 1u, WIN - 1u);
        const uint32_t vwin = tid <= WIN ? __ldcg(&P.coarse_win[WIN - tid]) : 0u;
        uint32_t vfine = tid < 512u ? __ldcg(&P.fine_hist[cb_guess * 512u + 511u - tid]) : 0u;
        M = __ldcg(&P.ctrl[CT_CAND]);
        const bool overflowed = __ldcg(&P.ctrl[CT_OVERFLOW]) != 0u;
        bool ok = (M >= k) && !overflowed;
        if (attempt == 0) hint_overflowed = overflowed;
        if (ok) {
            find_in_regs(vwin, WIN + 1, k, s);
            const uint32_t cb = s.res[0], above = s.res[1], at = s.res[2];
            __syncthreads();
            ok = cb < WIN;                                             // else the k-th key is above the window (or not found)
            if (ok) {
                st.prefix = b_lo + cb; st.nbits = 13; st.need = k - above; st.group = at;
                if (!sel_done(st)) {
                    if (cb != cb_guess) vfine = tid < 512u ? __ldcg(&P.fine_hist[cb * 512u + 511u - tid]) : 0u;
                    find_in_regs(vfine, 512, st.need, s);
                    const uint32_t fb = s.res[0], fa = s.res[1], fc = s.res[2];
                    __syncthreads();
                    ok = fb != 0xFFFFFFFFu;                            // else the histograms disagree
                    if (ok) { st.prefix = (st.prefix << 9) | fb; st.nbits = 22; st.need -= fa; st.group = fc; }
                }
            }
        }
        if (ok) { fast = true; used_hint = attempt == 0; break; }
        st.prefix = 0; st.nbits = 0; st.need = k; st.group = d;
        if (attempt == 0) SC_BARRIER();                                // every block has checked the pass before it is undone
    }
    if (P.force_exact) {
        clear_outputs();
        SC_BARRIER();                                                  // the exact mark pass may follow with no other barrier
        SC_STAMP(4); SC_STAMP(5);
    }
    if (gtid == 0) {
        P.ctrl[CT_PATH] = fast ? (used_hint ? PATH_FAST_HINT : PATH_FAST) : PATH_EXACT;
        P.ctrl[CT_M] = M;
    }

    // a small boundary group is ranked in P5; anything else goes digit by digit
    const bool boundary = fast && !sel_done(st) && st.nbits == 22 && st.group <= BCAP;
    uint32_t pass = 0;
    while (!boundary && !sel_done(st)) {
        // digit width: the key's 31 bits split 11/10/10 (or the 9 left after the fine prefix), the index's 11/10/10
        int W;
        if (st.nbits == 22) W = 9;
        else if (st.nbits == 0 || st.nbits == 31) W = 11;
        else W = 10;
        const int shift_match = 62 - st.nbits, shift_digit = 62 - st.nbits - W;
        const uint32_t dmask = (1u << W) - 1u;
        uint32_t* gh = P.digit_hist + pass * DH_BINS;
        if (fast) {
            for (uint32_t i = lane; i < seg_cnt; i += 32) {
                const uint2 e = __ldcg(&seg[i]);
                const uint64_t c = composite(e.x, e.y);
                if ((c >> shift_match) == st.prefix) atomicAdd(&gh[uint32_t(c >> shift_digit) & dmask], 1u);
            }
        } else {
            for (uint32_t i = tid; i < DH_BINS; i += TK_THREADS) s.hist[i] = 0;
            __syncthreads();
            for (uint32_t it0 = 0; it0 < my_units; it0 += TK_UNROLL) {
                float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
                    if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
                }
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint64_t cc = composite(mag_key(__fadd_rn(mv[u][c], gv[u][c])), p + c);
                        const bool pr = (p + c < d) && (cc >> shift_match) == st.prefix;
                        const uint32_t act = __ballot_sync(FULL, pr);
                        if (pr) {
                            const uint32_t dg = uint32_t(cc >> shift_digit) & dmask;
                            const uint32_t peers = __match_any_sync(act, dg);
                            if (lane == uint32_t(__ffs(peers) - 1)) atomicAdd(&s.hist[dg], uint32_t(__popc(peers)));
                        }
                    }
                }
            }
            __syncthreads();
            for (uint32_t i = tid; i < DH_BINS; i += TK_THREADS) {
                const uint32_t h = s.hist[i];
                if (h) atomicAdd(&gh[i], h);
            }
        }
        SC_BARRIER();
        find_from_top(gh, 1u << W, st.need, s);
        const uint32_t dg = s.res[0], above = s.res[1], at = s.res[2];
        __syncthreads();
        ++pass;
        if (dg == 0xFFFFFFFFu) {                                       // cannot happen: the group holds >= need
            if (tid == 0) atomicCAS(status, DEV_OK, DEV_INTERNAL);
            st.need = st.group;                                        // terminate consistently on every block
            break;
        }
        st.prefix = (st.prefix << W) | dg; st.nbits += W; st.need -= above; st.group = at;
        if (pass >= DH_PASSES) break;
    }

    // ---------------- P4: mark winners ---------------------------------------------------------
    SC_STAMP(6);
    // winners are the composites >= T; with a boundary group, T covers it and the group is ranked separately
    const uint64_t T = st.nbits >= 62 ? st.prefix : (st.prefix << (62 - st.nbits));
    const uint64_t T_above = boundary ? ((st.prefix + 1) << (62 - st.nbits)) : T;   // strictly above the group
    if (fast) {
        // winners per scan span are counted in shared memory first (nblocks <= NCOARSE spans)
        for (uint32_t i = tid; i < nblocks; i += TK_THREADS) s.hist[i] = 0;
        __syncthreads();
        for (uint32_t i = lane; i < seg_cnt; i += 32) {
            const uint2 e = __ldcg(&seg[i]);
            const uint64_t c = composite(e.x, e.y);
            if (c >= T_above) {
                atomicOr(&P.bitmap[e.y >> 5], 1u << (e.y & 31u));
                atomicAdd(&s.hist[e.y / span_coords], 1u);
            } else if (c >= T) {                                       // only with a boundary group
                const uint32_t slot = atomicAdd(&P.ctrl[CT_BCOUNT], 1u);
                if (slot < BCAP) P.blist[slot] = e;
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < nblocks; i += TK_THREADS) {
            const uint32_t h = s.hist[i];
            if (h) atomicAdd(&P.block_tot[i], h);
        }
    } else {
        // every 128-coordinate group is owned by one warp: whole bitmap words, plain stores
        for (uint32_t it0 = 0; it0 < my_units; it0 += TK_UNROLL) {
            float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
                if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
            }
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = unit_coord(it0 + u, my_units, nblocks, d) + tid * 4;
                uint32_t nib = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint64_t cc = composite(mag_key(__fadd_rn(mv[u][c], gv[u][c])), p + c);
                    if ((p + c < d) && cc >= T) nib |= 1u << c;
                }
                uint32_t word = nib << (4 * (lane & 7u));
                word |= __shfl_xor_sync(FULL, word, 1);
                word |= __shfl_xor_sync(FULL, word, 2);
                word |= __shfl_xor_sync(FULL, word, 4);
                const uint32_t wsum = warp_sum(uint32_t(__popc(nib)));
                const uint32_t p0 = p - lane * 4;                      // first coordinate of the warp's 128
                if (p0 < d) {
                    if ((lane & 7u) == 0) P.bitmap[(p0 >> 5) + (lane >> 3)] = word;
                    if (lane == 0 && wsum) atomicAdd(&P.block_tot[p0 / span_coords], wsum);
                }
            }
        }
    }
    SC_STAMP(7);
    SC_BARRIER();
    SC_STAMP(8);

    // ---------------- P5: boundary group, scan of the bitmap, clean-up ----------------------------------
    {
        // each warp owns a contiguous run of the span's tiles; all loads of this phase are issued up front
        const uint32_t t0 = blockIdx.x * P.tiles_per_block;
        const uint32_t t1 = min(P.ntiles, t0 + P.tiles_per_block);
        const uint32_t nt = t1 > t0 ? t1 - t0 : 0u;
        const uint32_t per_warp = (nt + TK_WARPS - 1) / TK_WARPS;
        const uint32_t w0 = min(t1, t0 + warp * per_warp), w1 = min(t1, w0 + per_warp);
        constexpr int RW = 8;                                          // tiles per warp kept in registers
        uint32_t wreg[RW];
#pragma unroll
        for (int j = 0; j < RW; ++j) wreg[j] = (w0 + j < w1) ? __ldcg(&P.bitmap[size_t(w0 + j) * 32 + lane]) : 0u;
        uint32_t part = 0;                                             // winners before this block's span
        for (uint32_t b = tid; b < blockIdx.x; b += TK_THREADS) part += __ldcg(&P.block_tot[b]);

        // shared-memory scratch carved from the (idle) histogram array
        uint32_t* own = s.hist;                                        // [BCAP] boundary winners inside this block's span
        uint32_t* kh = own + BCAP;                                     // [512]  histogram of the members' last 9 key bits
        uint32_t* ties = kh + 512;                                     // [BCAP] members sharing the k-th key
        if (tid == 0) { s.own_n = 0; s.res[3] = 0; }
        if (boundary) {
            // Every block ranks the boundary group itself.  The members share 22 key bits; a 512-bin
            // histogram of the remaining 9 finds the k-th key, members above it win, members on it are
            // ranked by index among themselves.  Winners inside this block's span are kept in `own`
            // (and set in the global bitmap for the learner pass), winners before it are counted.
            const uint32_t cnt = st.group;                             // <= BCAP
            if (tid == 0 && __ldcg(&P.ctrl[CT_BCOUNT]) != cnt)         // cannot happen: the histograms counted `group`
                atomicCAS(status, DEV_OK, DEV_INTERNAL);
            for (uint32_t i = tid; i < 512; i += TK_THREADS) kh[i] = 0;
            uint2 mine[BCAP / TK_THREADS];
#pragma unroll
            for (int r = 0; r < int(BCAP / TK_THREADS); ++r) {
                const uint32_t i = tid + r * TK_THREADS;
                mine[r] = i < cnt ? __ldcg(&P.blist[i]) : make_uint2(0u, 0u);
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < int(BCAP / TK_THREADS); ++r)
                if (tid + r * TK_THREADS < cnt) atomicAdd(&kh[mine[r].x & 511u], 1u);
            __syncthreads();
            if (warp == 0) {                                           // k-th key: 16 bins per lane, from the top
                uint32_t sum = 0;
#pragma unroll
                for (int j = 0; j < 16; ++j) sum += kh[511 - (lane * 16 + j)];
                const uint32_t incl = warp_incl_scan(sum);
                uint32_t run = incl - sum;
                if (run < st.need && st.need <= incl) {
                    for (int j = 0; j < 16; ++j) {
                        const uint32_t c = kh[511 - (lane * 16 + j)];
                        if (st.need <= run + c) { s.res[0] = 511 - (lane * 16 + j); s.res[1] = run; s.res[2] = c; break; }
                        run += c;
                    }
                }
            }
            __syncthreads();
            const uint32_t kstar = s.res[0], need_ties = st.need - s.res[1];
            const uint32_t c0 = blockIdx.x * span_coords;
            auto win = [&](uint32_t idx) {
                if (idx < c0) {
                    ++part;
                } else if (idx - c0 < span_coords) {
                    atomicOr(&P.bitmap[idx >> 5], 1u << (idx & 31u));   // for the learner pass; not read back here
                    own[atomicAdd(&s.own_n, 1u)] = idx;
                }
            };
#pragma unroll
            for (int r = 0; r < int(BCAP / TK_THREADS); ++r)
                if (tid + r * TK_THREADS < cnt) {
                    const uint32_t kl = mine[r].x & 511u;
                    if (kl > kstar) win(mine[r].y);
                    else if (kl == kstar) ties[atomicAdd(&s.res[3], 1u)] = mine[r].y;
                }
            __syncthreads();
            const uint32_t nties = s.res[3];
            for (uint32_t i = tid; i < nties; i += TK_THREADS) {       // lower index first among equal keys
                const uint32_t idx = ties[i];
                uint32_t before = 0;
                for (uint32_t j = 0; j < nties; ++j) before += ties[j] < idx ? 1u : 0u;
                if (before < need_ties) win(idx);
            }
        }
        __syncthreads();
        SC_STAMP(10);
        const uint32_t own_n = s.own_n;
        // bitmap word (tile, lane) with this block's boundary winners merged in
        auto merge_own = [&](uint32_t tile, uint32_t word) {
            for (uint32_t o = 0; o < own_n; ++o) {
                const uint32_t idx = own[o];
                if ((idx >> 5) == tile * 32 + lane) word |= 1u << (idx & 31u);
            }
            return word;
        };
        uint32_t ttot[RW];                                             // winners per cached tile
        uint32_t wtot = 0;
#pragma unroll
        for (int j = 0; j < RW; ++j) {
            if (own_n && w0 + j < w1) wreg[j] = merge_own(w0 + j, wreg[j]);
            ttot[j] = __reduce_add_sync(FULL, uint32_t(__popc(wreg[j])));
            wtot += ttot[j];
        }
        for (uint32_t tile = w0 + RW; tile < w1; ++tile)
            wtot += __reduce_add_sync(FULL, uint32_t(__popc(merge_own(tile, __ldcg(&P.bitmap[size_t(tile) * 32 + lane])))));
        part = __reduce_add_sync(FULL, part);
        if (lane == 0) { s.scan[warp] = wtot; s.cw[warp] = part; }
        __syncthreads();
        SC_STAMP(11);
        uint32_t running = 0;                                          // winners before this warp's run
#pragma unroll
        for (int w = 0; w < TK_WARPS; ++w) {
            running += s.cw[w];
            if (w < (int)warp) running += s.scan[w];
        }
        // per tile: its prefix count, and (when asked for) its indices in ascending order
        auto emit = [&](uint32_t tile, uint32_t word, uint32_t total) {
            if (lane == 0) P.tile_prefix[tile] = running;
            if (P.out_idx) {
                const uint32_t cnt = __popc(word);
                uint32_t off = running + warp_incl_scan(cnt) - cnt;
                const uint32_t cbase = tile * TILE + lane * 32;
                while (word) {
                    const uint32_t b = __ffs(word) - 1;
                    word &= word - 1;
                    if (off < k) P.out_idx[off] = int32_t(cbase + b);
                    ++off;
                }
            }
            running += total;
        };
#pragma unroll
        for (int j = 0; j < RW; ++j)
            if (w0 + j < w1) emit(w0 + j, wreg[j], ttot[j]);
        for (uint32_t tile = w0 + RW; tile < w1; ++tile) {
            const uint32_t word = merge_own(tile, __ldcg(&P.bitmap[size_t(tile) * 32 + lane]));
            emit(tile, word, __reduce_add_sync(FULL, uint32_t(__popc(word))));
        }
        if (blockIdx.x == nblocks - 1 && tid == TK_THREADS - 1) {
            // the last warp of the last block ends on the grand total: the winners must number exactly k
            P.tile_prefix[P.ntiles] = running;
            if (running != k) atomicCAS(status, DEV_OK, DEV_INTERNAL);
        }

        SC_STAMP(12);
        // leave the histograms and counters zero for the next launch, and the hint for its bound
        if (!P.fine_hist_next) zero_words(P.fine_hist, NFINE, gtid, gsize);
        for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
        if (pass) zero_words(P.digit_hist, size_t(pass) * DH_BINS, gtid, gsize);
        if (gtid == 0) {
            P.ctrl[CT_CAND] = 0; P.ctrl[CT_OVERFLOW] = 0;
        }
        if (gtid == 0 && P.use_hint) {
            // the 13-bit bin (about 3 % in magnitude) of the k-th key just found, for this leader and for the next
            // step.  Later bounds keep one bin of distance; two after a hint that left too few survivors, one again
            // after one that left too many or came close to it (error feedback piles coordinates up just below
            // the threshold: late in a run one bin holds about k of them)
            if (hint && !used_hint) P.ctrl[CT_MARGIN] = hint_overflowed ? 0u : 1u;
            else if (used_hint && M > 3u * k) P.ctrl[CT_MARGIN] = 0u;
            // a useless hint that came from this leader's own earlier value means the scale moved under the learners:
            // what the other leaders remember (and the change this one is about to record against its stale value)
            // would mislead the next steps, which start from this step's bin instead until each leader has led
            // again.  (A useless hint borrowed from the previous step's leader only says that learners differ.)
            const bool forget = hint && !used_hint && own_prev && P.all_hints;
            if (forget)
                for (uint32_t i = 0; i < P.n_hints; ++i) P.all_hints[i] = 0u;
            const uint32_t cbk = st.nbits >= 13 ? uint32_t(st.prefix >> (st.nbits - 13)) : 0u;
            if (forget) P.ctrl[CT_DRIFT] = 0u;
            else if (cbk && own_prev) P.ctrl[CT_DRIFT] = uint32_t(int32_t(cbk) - int32_t(own_prev - 1u));
            P.ctrl[CT_HINT] = cbk ? cbk + 1u : 0u;
            if (P.leader_hint) *P.leader_hint = cbk ? cbk + 1u : 0u;
        }
    }
    SC_STAMP(9);
    span_end(P.spans);
#undef SC_BARRIER
#undef SC_STAMP
}

}  // namespace sc
