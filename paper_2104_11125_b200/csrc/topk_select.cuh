// Leader top-k (Eq. 2): one persistent cooperative kernel.
//
// Selects the k coordinates of acc = m + g (computed on the fly, never stored)
// that come first in the order "larger |acc| first, lower index first", and
// leaves the result in three forms: a d-bit bitmap, the per-tile prefix counts
// of that bitmap, and the ascending index list.
//
// Fast path (one streaming read of g and m):
//   P0  clear scratch; histogram a strided sample of the keys (top 13 bits)
//   P1  every block derives from the sample a conservative lower bound on the
//       k-th key (bin b_lo), aiming at slightly more than k survivors
//   P2  stream g, m once: survivors (key bin >= b_lo) go to a compact candidate
//       list (warp-staged, one atomic per ~100 survivors) and into two small
//       histograms (13-bit bins in a 64-bin window above b_lo; 22-bit prefixes)
//   P3  radix-select the k-th composite among the candidates: the two histograms
//       fix 22 key bits, one pass over the (L2-resident) list fixes the last 9,
//       up to three more fix the index when equal keys straddle rank k
//   P4  mark the winners in the bitmap, count them per block span
//   P5  prefix-scan the bitmap: tile prefixes + ascending indices
// Exact path (taken when the candidate list overflowed, came up short, or the
// k-th key left the histogram window; also on request): the same radix select
// with every pass streaming g and m again (up to six passes) and a mark pass.
// Correctness never depends on the sample.
#pragma once
#include "common.cuh"

namespace sc {

#ifndef SC_TK_THREADS
#define SC_TK_THREADS 512
#endif
#ifndef SC_TK_BLOCKS_PER_SM
#define SC_TK_BLOCKS_PER_SM 2
#endif
constexpr int TK_THREADS = SC_TK_THREADS;
constexpr int TK_BLOCKS_PER_SM = SC_TK_BLOCKS_PER_SM;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int TK_UNROLL = 4;                                   // quads of g and of m in flight per thread
constexpr uint32_t TK_CHUNK = TK_THREADS * 4 * TK_UNROLL;      // coordinates per block iteration (8192)

constexpr int COARSE_SHIFT = 18;                               // key >> 18: 13-bit coarse bin
constexpr uint32_t NCOARSE = 1u << 13;
constexpr int FINE_SHIFT = 9;                                  // key >> 9: 22-bit fine prefix
constexpr uint32_t WIN = 64;                                   // coarse bins covered above b_lo
constexpr uint32_t NFINE = WIN * 512;
constexpr uint32_t DH_BINS = 2048;                             // digit histogram of one radix pass
constexpr uint32_t DH_PASSES = 8;
constexpr uint32_t WCAP = 192;                                 // candidate staging entries per warp
constexpr uint32_t SAMPLE_GRANULE = 128;                       // coordinates one warp samples at a time

// ctrl words
constexpr int CT_CAND = 0, CT_STATUS = 1, CT_PATH = 2, CT_M = 3, CT_STAMP = 8, CT_NSTAMPS = 10, CT_WORDS = 32;

struct TopkParams {
    const float* g;            // leader's gradient, fp32[d]
    const float* m;            // leader's memory, fp32[d]
    uint32_t d, k;
    uint32_t samp_stride;      // sample one granule out of this many
    uint32_t samp_target;      // wanted number of sampled keys at or above the bound
    uint32_t force_exact;
    uint32_t spin_limit;
    uint32_t* samp_hist;       // [NCOARSE], zero on entry, zero on exit
    uint32_t* coarse_win;      // [WIN + 1]
    uint32_t* fine_hist;       // [NFINE]
    uint32_t* digit_hist;      // [DH_PASSES * DH_BINS]
    uint32_t* block_tot;       // [gridDim.x] winners per block span
    uint32_t* ctrl;            // [CT_WORDS]
    unsigned long long* barrier;
    uint2* cand;               // [cand_cap] (key, idx)
    uint32_t cand_cap;
    uint32_t* bitmap;          // [ntiles * 32]
    uint32_t* tile_prefix;     // [ntiles + 1]
    uint32_t ntiles;
    uint32_t tiles_per_block;  // span of the final scan
    int32_t* out_idx;          // [k]
};

struct TopkShared {
    uint32_t hist[NCOARSE];            // sample histogram / staging for bin searches / digit histogram
    uint2 stage[TK_WARPS][WCAP];       // per-warp candidate staging
    uint32_t cw[WIN + 1];              // this block's share of the coarse window histogram
    uint32_t scan[32];
    uint32_t res[4];
    int flag;
};

// Search a histogram (global memory, written by other blocks before the last
// grid barrier) from its top bin downwards for the bin holding the `need`-th
// element: res = {bin, count strictly above bin, count in bin}, or bin =
// 0xFFFFFFFF when the histogram holds fewer than `need` elements.  nb <= 8192.
// Two levels, both with one bin per lane per load (coalesced, no bank
// conflicts): 16 warp-sized segments, then 16 sub-segments of <= 32 bins.
__device__ inline void find_from_top(const uint32_t* h, uint32_t nb, uint32_t need, TopkShared& s) {
    const uint32_t lane = lane_id(), warp = warp_id();
    if (threadIdx.x == 0) s.res[0] = 0xFFFFFFFFu;
    // level 1: warp w sums reversed positions [w*seglen, (w+1)*seglen)
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
    // level 2: inside segment `seg`, warp w owns reversed positions [w*sublen, (w+1)*sublen), sublen <= 32
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
    const uint32_t nchunks = (d + TK_CHUNK - 1) / TK_CHUNK;

    // phase time stamps of block 0 (low word of the nanosecond global timer), for profiling only
#define SC_STAMP(i) do { if (gtid == 0) { uint32_t ts_; asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(ts_)); \
                                          P.ctrl[CT_STAMP + (i)] = ts_; } } while (0)
#define SC_BARRIER() do { if (!grid_barrier(P.barrier, nblocks, status, P.spin_limit, &s.flag)) return; } while (0)

    // ---------------- P0: clear scratch, sample ----------------------------------------------
    SC_STAMP(0);
    zero_words(P.bitmap, size_t(P.ntiles) * 32, gtid, gsize);
    zero_words(P.fine_hist, NFINE, gtid, gsize);
    zero_words(P.digit_hist, DH_PASSES * DH_BINS, gtid, gsize);
    for (size_t i = gtid; i < nblocks; i += gsize) P.block_tot[i] = 0;
    for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
    if (gtid == 0) { P.ctrl[CT_CAND] = 0; P.ctrl[CT_PATH] = 0; P.ctrl[CT_M] = 0; }

    uint32_t b_lo = 0;
    if (!P.force_exact) {
        for (uint32_t i = tid; i < NCOARSE; i += TK_THREADS) s.hist[i] = 0;
        __syncthreads();
        const uint32_t span = SAMPLE_GRANULE * P.samp_stride;          // coordinates between sampled granules
        const uint32_t ngran = (d + span - 1) / span;
        for (uint32_t gidx = blockIdx.x * TK_WARPS + warp; gidx < ngran; gidx += nblocks * TK_WARPS) {
            const uint32_t p = gidx * span + lane * 4;                 // gidx*span < d
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
    }
    SC_STAMP(1);
    SC_BARRIER();
    SC_STAMP(2);

    // ---------------- P1 + P2: bound from the sample, filter pass ----------------------------------
    bool fast = !P.force_exact;
    if (fast) {
        find_from_top(P.samp_hist, NCOARSE, P.samp_target, s);
        b_lo = (s.res[0] == 0xFFFFFFFFu) ? 0u : s.res[0];
        __syncthreads();
        SC_STAMP(3);

        for (uint32_t i = tid; i <= WIN; i += TK_THREADS) s.cw[i] = 0;
        __syncthreads();
        const uint32_t thr_key = b_lo << COARSE_SHIFT;
        const uint32_t fine_base = b_lo << (COARSE_SHIFT - FINE_SHIFT);
        uint2* stage = s.stage[warp];
        uint32_t wcnt = 0;                                             // warp-uniform
        for (uint32_t ch = blockIdx.x; ch < nchunks; ch += nblocks) {
            const uint32_t base = ch * TK_CHUNK + tid * 4;
            float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = base + u * (TK_THREADS * 4);
                if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
            }
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = base + u * (TK_THREADS * 4);
                uint32_t key[4];
                bool pred[4];
                bool any = false;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    key[c] = mag_key(__fadd_rn(mv[u][c], gv[u][c]));
                    pred[c] = (p < d) && (p + c < d) && key[c] >= thr_key;
                    any |= pred[c];
                }
                if (__any_sync(FULL, any)) {
                    if (wcnt + 128u > WCAP) {                          // make room: flush the warp's staging
                        uint32_t gb = 0;
                        if (lane == 0) gb = atomicAdd(&P.ctrl[CT_CAND], wcnt);
                        gb = __shfl_sync(FULL, gb, 0);
                        for (uint32_t i = lane; i < wcnt; i += 32)
                            if (gb + i < P.cand_cap) P.cand[gb + i] = stage[i];
                        __syncwarp();
                        wcnt = 0;
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t bal = __ballot_sync(FULL, pred[c]);
                        if (pred[c]) {
                            stage[wcnt + __popc(bal & ((1u << lane) - 1u))] = make_uint2(key[c], p + c);
                            const uint32_t cb = (key[c] >> COARSE_SHIFT) - b_lo;
                            atomicAdd(&s.cw[cb < WIN ? cb : WIN], 1u);
                            if (cb < WIN) atomicAdd(&P.fine_hist[(key[c] >> FINE_SHIFT) - fine_base], 1u);
                        }
                        wcnt += __popc(bal);
                    }
                    __syncwarp();
                }
            }
        }
        if (wcnt) {
            uint32_t gb = 0;
            if (lane == 0) gb = atomicAdd(&P.ctrl[CT_CAND], wcnt);
            gb = __shfl_sync(FULL, gb, 0);
            for (uint32_t i = lane; i < wcnt; i += 32)
                if (gb + i < P.cand_cap) P.cand[gb + i] = stage[i];
        }
        __syncthreads();
        for (uint32_t i = tid; i <= WIN; i += TK_THREADS) {
            const uint32_t h = s.cw[i];
            if (h) atomicAdd(&P.coarse_win[i], h);
        }
    }
    SC_STAMP(4);
    SC_BARRIER();
    SC_STAMP(5);

    // the sample histogram must be all zero again when the kernel ends
    if (!P.force_exact) zero_words(P.samp_hist, NCOARSE, gtid, gsize);

    // ---------------- P3: radix select ------------------------------------------------------------
    SelState st;
    st.prefix = 0; st.nbits = 0; st.need = k; st.group = d;
    uint32_t M = 0;
    uint32_t pass = 0;
    if (fast) {
        M = __ldcg(&P.ctrl[CT_CAND]);
        fast = (M >= k) && (M <= P.cand_cap);
    }
    if (fast) {
        find_from_top(P.coarse_win, WIN + 1, k, s);
        const uint32_t cb = s.res[0], above = s.res[1], at = s.res[2];
        __syncthreads();
        if (cb >= WIN) {
            fast = false;                                              // k-th key above the window (or not found)
        } else {
            st.prefix = b_lo + cb; st.nbits = 13; st.need = k - above; st.group = at;
            if (!sel_done(st)) {
                find_from_top(P.fine_hist + cb * 512u, 512, st.need, s);
                const uint32_t fb = s.res[0], fa = s.res[1], fc = s.res[2];
                __syncthreads();
                if (fb == 0xFFFFFFFFu) {
                    fast = false;                                      // histograms disagree: take the exact path
                } else {
                    st.prefix = (st.prefix << 9) | fb; st.nbits = 22; st.need -= fa; st.group = fc;
                }
            }
        }
    }
    if (!fast) { st.prefix = 0; st.nbits = 0; st.need = k; st.group = d; }
    if (gtid == 0) { P.ctrl[CT_PATH] = fast ? 0u : 1u; P.ctrl[CT_M] = M; }

    while (!sel_done(st)) {
        // digit width: the key's 31 bits split 11/10/10 (or the 9 left after the fine prefix), the index's 11/10/10
        int W;
        if (st.nbits == 22) W = 9;
        else if (st.nbits == 0 || st.nbits == 31) W = 11;
        else W = 10;
        const int shift_match = 62 - st.nbits, shift_digit = 62 - st.nbits - W;
        const uint32_t dmask = (1u << W) - 1u;
        uint32_t* gh = P.digit_hist + pass * DH_BINS;
        if (fast) {
            for (size_t i = gtid; i < M; i += gsize) {
                const uint2 e = __ldcg(&P.cand[i]);
                const uint64_t c = composite(e.x, e.y);
                if ((c >> shift_match) == st.prefix) atomicAdd(&gh[uint32_t(c >> shift_digit) & dmask], 1u);
            }
        } else {
            for (uint32_t i = tid; i < DH_BINS; i += TK_THREADS) s.hist[i] = 0;
            __syncthreads();
            for (uint32_t ch = blockIdx.x; ch < nchunks; ch += nblocks) {
                const uint32_t base = ch * TK_CHUNK + tid * 4;
                float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = base + u * (TK_THREADS * 4);
                    if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
                }
#pragma unroll
                for (int u = 0; u < TK_UNROLL; ++u) {
                    const uint32_t p = base + u * (TK_THREADS * 4);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint64_t cc = composite(mag_key(__fadd_rn(mv[u][c], gv[u][c])), p + c);
                        const bool pr = (p < d) && (p + c < d) && (cc >> shift_match) == st.prefix;
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
        if (dg == 0xFFFFFFFFu) {                                       // cannot happen: the group holds >= need
            if (tid == 0) atomicCAS(status, DEV_OK, DEV_INTERNAL);
            st.need = st.group;                                        // terminate consistently on every block
            break;
        }
        st.prefix = (st.prefix << W) | dg; st.nbits += W; st.need -= above; st.group = at;
        ++pass;
        if (pass >= DH_PASSES) break;
    }

    // ---------------- P4: mark winners (composite >= T) ---------------------------------------------
    SC_STAMP(6);
    const uint64_t T = st.nbits >= 62 ? st.prefix : (st.prefix << (62 - st.nbits));
    const uint32_t span_coords = P.tiles_per_block * TILE;
    if (fast) {
        // winners per scan span are counted in shared memory first (nblocks <= NCOARSE spans)
        for (uint32_t i = tid; i < nblocks; i += TK_THREADS) s.hist[i] = 0;
        __syncthreads();
        for (size_t i = gtid; i < M; i += gsize) {
            const uint2 e = __ldcg(&P.cand[i]);
            if (composite(e.x, e.y) >= T) {
                atomicOr(&P.bitmap[e.y >> 5], 1u << (e.y & 31u));
                atomicAdd(&s.hist[e.y / span_coords], 1u);
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < nblocks; i += TK_THREADS) {
            const uint32_t h = s.hist[i];
            if (h) atomicAdd(&P.block_tot[i], h);
        }
    } else {
        // every 128-coordinate group is owned by one warp: whole bitmap words, plain stores
        for (uint32_t ch = blockIdx.x; ch < nchunks; ch += nblocks) {
            const uint32_t base = ch * TK_CHUNK + tid * 4;
            float gv[TK_UNROLL][4], mv[TK_UNROLL][4];
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = base + u * (TK_THREADS * 4);
                if (p < d) { load_quad_stream<VEC>(P.g, p, d, gv[u]); load_quad_stream<VEC>(P.m, p, d, mv[u]); }
            }
#pragma unroll
            for (int u = 0; u < TK_UNROLL; ++u) {
                const uint32_t p = base + u * (TK_THREADS * 4);
                uint32_t nib = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint64_t cc = composite(mag_key(__fadd_rn(mv[u][c], gv[u][c])), p + c);
                    if ((p < d) && (p + c < d) && cc >= T) nib |= 1u << c;
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

    // ---------------- P5: scan the bitmap: tile prefixes and ascending indices ---------------------
    {
        uint32_t part = 0;
        for (uint32_t b = tid; b < blockIdx.x; b += TK_THREADS) part += __ldcg(&P.block_tot[b]);
        part = warp_sum(part);
        if (lane == 0) s.scan[warp] = part;
        __syncthreads();
        uint32_t running = 0;
#pragma unroll
        for (int w = 0; w < TK_WARPS; ++w) running += s.scan[w];
        __syncthreads();

        const uint32_t t0 = blockIdx.x * P.tiles_per_block;
        const uint32_t t1 = min(P.ntiles, t0 + P.tiles_per_block);
        for (uint32_t tb = t0; tb < t1; tb += TK_WARPS) {
            const uint32_t tile = tb + warp;
            uint32_t word = 0;
            if (tile < t1) word = __ldcg(&P.bitmap[size_t(tile) * 32 + lane]);
            const uint32_t cnt = __popc(word);
            const uint32_t incl = warp_incl_scan(cnt);
            if (lane == 31) s.scan[warp] = incl;
            __syncthreads();
            uint32_t before = running, all = 0;
#pragma unroll
            for (int w = 0; w < TK_WARPS; ++w) {
                const uint32_t v = s.scan[w];
                if (w < (int)warp) before += v;
                all += v;
            }
            if (tile < t1) {
                if (lane == 0) P.tile_prefix[tile] = before;
                uint32_t off = before + incl - cnt;
                const uint32_t cbase = tile * TILE + lane * 32;
                while (word) {
                    const uint32_t b = __ffs(word) - 1;
                    word &= word - 1;
                    if (off < k) P.out_idx[off] = int32_t(cbase + b);
                    ++off;
                }
            }
            running += all;
            __syncthreads();
        }
        if (blockIdx.x == nblocks - 1 && tid == 0) {
            P.tile_prefix[P.ntiles] = running;
            if (running != k) atomicCAS(status, DEV_OK, DEV_INTERNAL);  // the winners must number exactly k
        }
    }
    SC_STAMP(9);
#undef SC_BARRIER
#undef SC_STAMP
}

}  // namespace sc
