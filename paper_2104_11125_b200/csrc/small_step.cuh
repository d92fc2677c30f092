// One CLT-k step (Algorithm 1 lines 6-12) in ONE cooperative kernel, for vectors small enough that the
// step is bound by launch gaps and grid barriers rather than by memory traffic (all g and m of a step fit
// the L2 cache: a few megabytes per learner, at most 8 learners).
//
// Every block owns a contiguous range of tiles for the whole step, which keeps everything the general
// kernels exchange through global memory inside the block:
//   S1  the block filters ITS OWN range of the leader's acc = m + g against a lower bound on the k-th key
//       (from the handle's threshold hint; without one, or after a useless one, from a histogram of all
//       keys) and keeps the survivors as (key, index) in shared memory; the same two histograms as in the
//       general selection kernel (64-bin window per block in shared memory, 22-bit prefixes in global memory)
//   -- grid barrier --
//   S2  every block locates the k-th key's 22-bit prefix, sets the winners among its own survivors in a
//       bitmap of its own range IN SHARED MEMORY, publishes their number, and appends the survivors sharing
//       the prefix (the boundary group) to a short global list
//   -- grid barrier --
//   S3  every block ranks the boundary list (key, then lower index), takes the winners inside its range,
//       adds up the blocks before it: the rank of its first selected coordinate
//   S4  the learner pass over its own tiles (Eq. 3 gather, line 10 reduction in learner order, Eq. 4
//       memory update, line 12 weight update): same arithmetic, operation by operation, as the general
//       learner pass, with the selection bits read from shared memory
// Two grid barriers, no bitmap in global memory, one launch.  Vectors the pre-filter cannot handle (a
// boundary group beyond the short list, a survivor list that overflows) go through a radix select over the
// 62-bit composites of the block's range, one grid barrier per digit; correctness never depends on the hint.
#pragma once
#include "learner_pass.cuh"
#include "topk_select.cuh"

namespace sc {

constexpr int SS_THREADS = TK_THREADS;                 // the histogram searches of the selection kernel are reused
constexpr int SS_WARPS = SS_THREADS / 32;
constexpr int SS_MAXN = 8;                             // learners
constexpr uint32_t SS_TILES = 16;                      // tiles a block may own
constexpr uint32_t SS_CAND = 4096;                     // survivors a block may keep

struct SmallParams {
    PtrTable<SS_MAXN> tab;     // g_i, m_i of the n learners (16-byte aligned)
    uint32_t d, k, ntiles;
    int32_t n, leader;
    float beta, omb, lr, nf;
    uint32_t force_exact, use_hint, spin_limit;
    uint32_t* leader_hint;     // as in TopkParams
    uint32_t* all_hints;
    uint32_t n_hints;
    // scratch shared with the general selection kernel (all zero on entry and on exit)
    uint32_t* key_hist;        // [NCOARSE] histogram of all keys' coarse bins
    uint32_t* coarse_win;      // [WIN + 1]
    uint32_t* fine_hist;       // [NFINE]
    uint32_t* fine_hist_next;  // [NFINE] or nullptr
    uint32_t* digit_hist;      // [DH_PASSES * DH_BINS]
    uint32_t* block_tot;       // [gridDim.x] winners per block (rewritten by every launch)
    uint32_t* ctrl;            // [CT_WORDS]
    unsigned long long* barrier;
    uint2* blist;              // [BCAP]
    // outputs
    int32_t* out_idx;          // [k]
    float* out_val;            // [k]
    float* gathered;           // [n * k] or nullptr
    float* weights;            // [d] or nullptr
    unsigned long long* spans; // nullptr, or {~start, end} of the kernel
};

struct SmallShared {
    uint32_t hist[NCOARSE];            // key histogram / digit histogram / boundary ranking scratch
    uint2 cand[SS_CAND];               // this block's survivors
    uint32_t bm[SS_TILES * 32];        // selection bits of this block's range
    uint32_t tpre[SS_TILES + 1];       // selected coordinates before each of the block's tiles (block-local)
    uint32_t cw[WIN + 1];
    uint32_t scan[32];
    uint32_t res[4];
    uint32_t ncand;
    uint32_t part;                     // selected coordinates in the blocks before this one
    int flag;
};

// The learner pass over the tiles [t0, t0 + ntl) of one block of the one-kernel step: selection bits from the block's
// shared-memory bitmap, ranks from its prefix counts; the arithmetic is that of learner_pass_kernel, operation by
// operation.  Two tiles at a time (256 threads each).  (Issuing the loads of a half-block's next tile before the
// current one is worked on, with twice the registers, measured no faster.)
template <int NL>
__device__ __forceinline__ void small_learner_tiles(const SmallParams& P, SmallShared& s, uint32_t t0, uint32_t ntl) {
    const uint32_t tid = threadIdx.x, lane = lane_id();
    const uint32_t d = P.d, k = P.k;
    const int n = P.n;
    const uint32_t half = tid >> 8, ht = tid & 255u;                   // which of the two tiles, thread inside it
    const uint32_t wi = ht >> 3, sh = (ht & 7u) * 4u;                  // this thread's bitmap word and first bit in it
    for (uint32_t j = half; j < ntl; j += 2) {
        float gv[NL][4], mv[NL][4];
        const uint32_t pc = (t0 + j) * TILE + ht * 4u;
        const uint32_t bw = s.bm[j * 32 + lane];
#pragma unroll
        for (int i = 0; i < NL; ++i)
            if (i < n && pc < d) {
                load_quad_stream<true>(P.tab.g[i], pc, d, gv[i]);
                load_quad_stream<true>(P.tab.m[i], pc, d, mv[i]);
            }
        const uint32_t cnt = __popc(bw);
        const uint32_t incl = warp_incl_scan(cnt);
        const uint32_t excl_word = __shfl_sync(FULL, incl - cnt, wi);
        const uint32_t myword = __shfl_sync(FULL, bw, wi);
        const uint32_t nib = (myword >> sh) & 15u;
        const uint32_t rank0 = s.part + s.tpre[j] + excl_word + __popc(myword & ((1u << sh) - 1u));
        float wv[4];
#pragma unroll
        for (int c = 0; c < 4; ++c)
            wv[c] = (P.weights && ((nib >> c) & 1u) && pc + c < d) ? P.weights[pc + c] : 0.0f;
        float sum[4];
#pragma unroll
        for (int i = 0; i < NL; ++i)
            if (i < n && pc < d) {
                float acc[4], out[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    acc[c] = __fadd_rn(mv[i][c], gv[i][c]);                              // line 6: m + g
                    sum[c] = (i == 0) ? acc[c] : __fadd_rn(sum[c], acc[c]);                    // line 10, learner order
                    const float r = ((nib >> c) & 1u) ? 0.0f : acc[c];                         // acc - CLT-k(acc)
                    out[c] = __fadd_rn(__fmul_rn(P.omb, mv[i][c]), __fmul_rn(P.beta, r));   // Eq. 4
                }
                store_quad_stream<true>(P.tab.m[i], pc, d, out);
                if (nib && P.gathered) {                                                       // Eq. 3
                    uint32_t r = rank0;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if ((nib >> c) & 1u) P.gathered[size_t(i) * k + r++] = acc[c];
                }
            }
        if (nib && pc < d) {
            uint32_t r = rank0;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if ((nib >> c) & 1u) {
                    const float v = __fdiv_rn(sum[c], P.nf);                                   // line 10: one division by n
                    P.out_idx[r] = int32_t(pc + c);
                    P.out_val[r] = v;
                    ++r;
                    if (P.weights) P.weights[pc + c] = __fsub_rn(wv[c], __fmul_rn(P.lr, v));   // line 12
                }
        }
    }
}

__global__ void __launch_bounds__(SS_THREADS, 1) small_step_kernel(const __grid_constant__ SmallParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmallShared& s = *reinterpret_cast<SmallShared*>(smem_raw);
    const uint32_t tid = threadIdx.x, lane = lane_id(), warp = warp_id();
    const uint32_t nblocks = gridDim.x;
    const size_t gtid = size_t(blockIdx.x) * SS_THREADS + tid;
    const size_t gsize = size_t(nblocks) * SS_THREADS;
    const uint32_t d = P.d, k = P.k;
    uint32_t* status = P.ctrl + CT_STATUS;
    GridBarrier gb;
    gb.arrive = P.barrier; gb.nblocks = nblocks; gb.status = status; gb.spin_limit = P.spin_limit;
#define SS_BARRIER() do { if (!grid_barrier(gb, &s.flag)) return; } while (0)
    // phase time stamps of block 0 (low word of the nanosecond global timer), for profiling only
#define SS_STAMP(i) do { if (gtid == 0) { uint32_t ts_; asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(ts_)); \
                                          P.ctrl[CT_STAMP + (i)] = ts_; } } while (0)

    // this block's range of tiles and coordinates
    const uint32_t t0 = uint32_t(uint64_t(P.ntiles) * blockIdx.x / nblocks);
    const uint32_t t1 = uint32_t(uint64_t(P.ntiles) * (blockIdx.x + 1) / nblocks);
    const uint32_t c0 = t0 * TILE, c1 = min(d, t1 * TILE);
    const float* const gL = P.tab.g[P.leader];
    const float* const mL = P.tab.m[P.leader];

    span_begin(P.spans);
    SS_STAMP(0);
    for (uint32_t i = tid; i < SS_TILES * 32; i += SS_THREADS) s.bm[i] = 0;
    if (gtid == 0) P.ctrl[CT_BCOUNT] = 0;                              // (the list is filled behind a grid barrier)
    if (P.fine_hist_next) zero_words(P.fine_hist_next, NFINE, gtid, gsize);

    SelState st;
    st.prefix = 0; st.nbits = 0; st.need = k; st.group = d;
    bool fast = false, used_hint = false, hint_overflowed = false;
    uint32_t b_lo = 0, M = 0;
    // the bound to start from: exactly as in the general selection kernel (the two share the hint words)
    uint32_t hint = 0, hint_margin = 1;
    const uint32_t own_prev = (P.use_hint && P.leader_hint) ? __ldcg(P.leader_hint) : 0u;
    if (!P.force_exact && P.use_hint) {
        const uint32_t prev = __ldcg(&P.ctrl[CT_HINT]);
        const int32_t margin = 1 + int32_t(__ldcg(&P.ctrl[CT_MARGIN]));
        int32_t pred = own_prev ? int32_t(own_prev - 1u) + int32_t(__ldcg(&P.ctrl[CT_DRIFT])) : int32_t(prev) - 1;
        pred = min(pred, int32_t(NCOARSE) - 1);
        if (pred > margin) { hint = uint32_t(pred - margin) + 1u; hint_margin = uint32_t(margin); }
    }

    // acc of the leader at this thread's quad of the block's it-th row of 2048 coordinates (0 beyond the range)
    auto leader_quad = [&](uint32_t it, float (&acc)[4]) -> uint32_t {
        const uint32_t p = c0 + it * (SS_THREADS * 4u) + tid * 4u;
        float gv[4], mv[4];
        if (p < c1) { load_quad_stream<true>(gL, p, d, gv); load_quad_stream<true>(mL, p, d, mv); }
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[c] = (p + c < c1) ? __fadd_rn(mv[c], gv[c]) : 0.0f;
        return p;
    };
    const uint32_t nrows = (c1 > c0) ? (c1 - c0 + SS_THREADS * 4u - 1u) / (SS_THREADS * 4u) : 0u;

    for (int attempt = hint ? 0 : 1; attempt < 2 && !P.force_exact; ++attempt) {
        if (attempt == 0) {
            b_lo = hint - 1u;
        } else {
            // ---- histogram of all keys (13-bit bins): the exact bin of the k-th key ----
            if (hint) {                                                // the hinted pass failed: undo what it counted
                zero_words(P.fine_hist, NFINE, gtid, gsize);
                for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
                if (gtid == 0) { P.ctrl[CT_CAND] = 0; P.ctrl[CT_OVERFLOW] = 0; }
            }
            for (uint32_t i = tid; i < NCOARSE; i += SS_THREADS) s.hist[i] = 0;
            __syncthreads();
            for (uint32_t it = 0; it < nrows; ++it) {
                float acc[4];
                const uint32_t p = leader_quad(it, acc);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (p + c < c1) atomicAdd(&s.hist[mag_key(acc[c]) >> COARSE_SHIFT], 1u);
            }
            __syncthreads();
            for (uint32_t i = tid; i < NCOARSE; i += SS_THREADS) {
                const uint32_t h = s.hist[i];
                if (h) atomicAdd(&P.key_hist[i], h);
            }
            SS_BARRIER();
            find_from_top(P.key_hist, NCOARSE, k, s);
            b_lo = (s.res[0] == 0xFFFFFFFFu) ? 0u : s.res[0];
            __syncthreads();
        }
        b_lo = min(b_lo, 0x7F800000u >> COARSE_SHIFT);

        // ---- S1: filter the block's own range ----
        for (uint32_t i = tid; i <= WIN; i += SS_THREADS) s.cw[i] = 0;
        if (tid == 0) s.ncand = 0;
        __syncthreads();
        const uint32_t thr_key = b_lo << COARSE_SHIFT;
        const uint32_t fine_base = b_lo << (COARSE_SHIFT - FINE_SHIFT);
        const float thr_f = __uint_as_float(thr_key);
        for (uint32_t it0 = 0; it0 < nrows; it0 += 4) {                 // four rows of loads in flight
            float acc[4][4];
            uint32_t pp[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) pp[u] = leader_quad(it0 + u, acc[u]);
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (pp[u] + c < c1 && !(fabsf(acc[u][c]) < thr_f)) {   // (true for NaN, like the integer order)
                        const uint32_t key = mag_key(acc[u][c]);
                        const uint32_t slot = atomicAdd(&s.ncand, 1u);
                        if (slot < SS_CAND) s.cand[slot] = make_uint2(key, pp[u] + c);
                        const uint32_t cb = (key >> COARSE_SHIFT) - b_lo;
                        atomicAdd(&s.cw[cb < WIN ? cb : WIN], 1u);
                        if (cb < WIN) atomicAdd(&P.fine_hist[(key >> FINE_SHIFT) - fine_base], 1u);
                    }
                }
        }
        __syncthreads();
        for (uint32_t i = tid; i <= WIN; i += SS_THREADS) {
            const uint32_t h = s.cw[i];
            if (h) atomicAdd(&P.coarse_win[i], h);
        }
        if (tid == 0) {
            if (s.ncand) atomicAdd(&P.ctrl[CT_CAND], s.ncand);
            if (s.ncand > SS_CAND) P.ctrl[CT_OVERFLOW] = 1u;
        }
        SS_STAMP(1);
        SS_BARRIER();
        SS_STAMP(2);
        if (attempt == 1) zero_words(P.key_hist, NCOARSE, gtid, gsize);    // all blocks have read it

        // ---- S2a: locate the k-th key (both histogram levels requested at once, as in the general kernel) ----
        const uint32_t cb_guess = min(attempt == 0 ? hint_margin : 0u, WIN - 1u);
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
            ok = cb < WIN;
            if (ok) {
                st.prefix = b_lo + cb; st.nbits = 13; st.need = k - above; st.group = at;
                if (!sel_done(st)) {
                    if (cb != cb_guess) vfine = tid < 512u ? __ldcg(&P.fine_hist[cb * 512u + 511u - tid]) : 0u;
                    find_in_regs(vfine, 512, st.need, s);
                    const uint32_t fb = s.res[0], fa = s.res[1], fc = s.res[2];
                    __syncthreads();
                    ok = fb != 0xFFFFFFFFu;
                    if (ok) { st.prefix = (st.prefix << 9) | fb; st.nbits = 22; st.need -= fa; st.group = fc; }
                }
            }
        }
        // the survivors can settle the selection when the prefix is final or the boundary group fits the short list
        if (ok && (sel_done(st) || (st.nbits == 22 && st.group <= BCAP))) { fast = true; used_hint = attempt == 0; break; }
        st.prefix = 0; st.nbits = 0; st.need = k; st.group = d;
        SS_BARRIER();                                                  // every block has checked the pass before it is undone
        if (attempt == 1) {                                            // nothing follows that would undo it: do it here
            zero_words(P.fine_hist, NFINE, gtid, gsize);
            for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
            if (gtid == 0) { P.ctrl[CT_CAND] = 0; P.ctrl[CT_OVERFLOW] = 0; }
        }
    }
    if (gtid == 0) {
        P.ctrl[CT_PATH] = fast ? (used_hint ? PATH_FAST_HINT : PATH_FAST) : PATH_EXACT;
        P.ctrl[CT_M] = M;
    }
    const bool boundary = fast && !sel_done(st);
    SS_STAMP(3);

    // ---- vectors the pre-filter could not handle: radix select over the composites of the block's range ----
    uint32_t pass = 0;
    while (!fast && !sel_done(st)) {
        int W;                                                         // the key's 31 bits split 11/10/10, the index's 11/10/10
        if (st.nbits == 0 || st.nbits == 31) W = 11; else W = 10;
        const int shift_match = 62 - st.nbits, shift_digit = 62 - st.nbits - W;
        const uint32_t dmask = (1u << W) - 1u;
        uint32_t* gh = P.digit_hist + pass * DH_BINS;
        for (uint32_t i = tid; i < DH_BINS; i += SS_THREADS) s.hist[i] = 0;
        __syncthreads();
        for (uint32_t it = 0; it < nrows; ++it) {
            float acc[4];
            const uint32_t p = leader_quad(it, acc);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint64_t cc = composite(mag_key(acc[c]), p + c);
                if (p + c < c1 && (cc >> shift_match) == st.prefix) atomicAdd(&s.hist[uint32_t(cc >> shift_digit) & dmask], 1u);
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < DH_BINS; i += SS_THREADS) {
            const uint32_t h = s.hist[i];
            if (h) atomicAdd(&gh[i], h);
        }
        SS_BARRIER();
        find_from_top(gh, 1u << W, st.need, s);
        const uint32_t dg = s.res[0], above = s.res[1], at = s.res[2];
        __syncthreads();
        ++pass;
        if (dg == 0xFFFFFFFFu) {                                       // cannot happen: the group holds >= need
            if (tid == 0) atomicCAS(status, DEV_OK, DEV_INTERNAL);
            st.need = st.group;
            break;
        }
        st.prefix = (st.prefix << W) | dg; st.nbits += W; st.need -= above; st.group = at;
        if (pass >= DH_PASSES) break;
    }

    // ---- S2b: winners of the block's own range into its bitmap; boundary members to the global list ----
    const uint64_t T = st.nbits >= 62 ? st.prefix : (st.prefix << (62 - st.nbits));
    const uint64_t T_above = boundary ? ((st.prefix + 1) << (62 - st.nbits)) : T;
    if (fast) {
        const uint32_t nc = min(s.ncand, SS_CAND);
        for (uint32_t i = tid; i < nc; i += SS_THREADS) {
            const uint2 e = s.cand[i];
            const uint64_t c = composite(e.x, e.y);
            if (c >= T_above) {
                atomicOr(&s.bm[(e.y - c0) >> 5], 1u << (e.y & 31u));
            } else if (c >= T) {
                const uint32_t slot = atomicAdd(&P.ctrl[CT_BCOUNT], 1u);
                if (slot < BCAP) P.blist[slot] = e;
            }
        }
    } else {
        for (uint32_t it = 0; it < nrows; ++it) {
            float acc[4];
            const uint32_t p = leader_quad(it, acc);
            uint32_t nib = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (p + c < c1 && composite(mag_key(acc[c]), p + c) >= T) nib |= 1u << c;
            if (nib) atomicOr(&s.bm[(p - c0) >> 5], nib << ((p - c0) & 31u));      // (p is a multiple of 4)
        }
    }
    __syncthreads();
    // selected coordinates of every tile of the range, then their exclusive prefix (block-local)
    const uint32_t ntl = t1 - t0;                                      // <= SS_TILES
    auto count_tiles = [&] {
        if (warp < ntl) {
            const uint32_t cnt = warp_sum(uint32_t(__popc(s.bm[warp * 32 + lane])));
            if (lane == 0) s.tpre[warp + 1] = cnt;
        }
        __syncthreads();
        if (tid == 0) {
            s.tpre[0] = 0;
            for (uint32_t j = 0; j < ntl; ++j) s.tpre[j + 1] += s.tpre[j];
        }
        __syncthreads();
    };
    count_tiles();
    if (tid == 0) P.block_tot[blockIdx.x] = s.tpre[ntl];
    SS_STAMP(4);
    SS_BARRIER();
    SS_STAMP(5);

    // ---- S3: blocks before this one; the boundary group ----
    {
        uint32_t part = 0;
        for (uint32_t b = tid; b < blockIdx.x; b += SS_THREADS) part += __ldcg(&P.block_tot[b]);
        uint32_t* kh = s.hist;                                         // [512] histogram of the members' last 9 key bits
        uint32_t* ties = kh + 512;                                     // [BCAP] members sharing the k-th key
        if (tid == 0) { s.part = 0; s.res[3] = 0; }
        if (boundary) {
            const uint32_t cnt = st.group;                             // <= BCAP
            if (tid == 0 && __ldcg(&P.ctrl[CT_BCOUNT]) != cnt) atomicCAS(status, DEV_OK, DEV_INTERNAL);
            for (uint32_t i = tid; i < 512; i += SS_THREADS) kh[i] = 0;
            uint2 mine[BCAP / SS_THREADS];
#pragma unroll
            for (int r = 0; r < int(BCAP / SS_THREADS); ++r) {
                const uint32_t i = tid + r * SS_THREADS;
                mine[r] = i < cnt ? __ldcg(&P.blist[i]) : make_uint2(0u, 0u);
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < int(BCAP / SS_THREADS); ++r)
                if (tid + r * SS_THREADS < cnt) atomicAdd(&kh[mine[r].x & 511u], 1u);
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
            auto win = [&](uint32_t idx) {
                if (idx < c0) ++part;
                else if (idx < c1) atomicOr(&s.bm[(idx - c0) >> 5], 1u << (idx & 31u));
            };
#pragma unroll
            for (int r = 0; r < int(BCAP / SS_THREADS); ++r)
                if (tid + r * SS_THREADS < cnt) {
                    const uint32_t kl = mine[r].x & 511u;
                    if (kl > kstar) win(mine[r].y);
                    else if (kl == kstar) ties[atomicAdd(&s.res[3], 1u)] = mine[r].y;
                }
            __syncthreads();
            const uint32_t nties = s.res[3];
            for (uint32_t i = tid; i < nties; i += SS_THREADS) {       // lower index first among equal keys
                const uint32_t idx = ties[i];
                uint32_t before = 0;
                for (uint32_t j = 0; j < nties; ++j) before += ties[j] < idx ? 1u : 0u;
                if (before < need_ties) win(idx);
            }
        }
        part = warp_sum(part);
        __syncthreads();
        if (lane == 0 && part) atomicAdd(&s.part, part);
        __syncthreads();
        if (boundary) count_tiles();                                   // the boundary winners changed the tile counts
        if (blockIdx.x == nblocks - 1 && tid == 0 && s.part + s.tpre[ntl] != k)
            atomicCAS(status, DEV_OK, DEV_INTERNAL);                   // the winners must number exactly k
    }

    SS_STAMP(6);
    // ---- leave the scratch clean and the hint for the next launch (nobody reads the histograms any more) ----
    if (!P.fine_hist_next && fast) zero_words(P.fine_hist, NFINE, gtid, gsize);
    if (fast) for (size_t i = gtid; i <= WIN; i += gsize) P.coarse_win[i] = 0;
    if (pass) zero_words(P.digit_hist, size_t(pass) * DH_BINS, gtid, gsize);
    if (gtid == 0) {
        P.ctrl[CT_CAND] = 0; P.ctrl[CT_OVERFLOW] = 0;
        if (P.use_hint) {
            if (hint && !used_hint) P.ctrl[CT_MARGIN] = hint_overflowed ? 0u : 1u;
            else if (used_hint && M > 3u * k) P.ctrl[CT_MARGIN] = 0u;
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

    SS_STAMP(7);
    // ---- S4: the learner pass over the block's own tiles (two tiles at a time, 256 threads each) ----
    if (P.n <= 4) small_learner_tiles<4>(P, s, t0, ntl);
    else small_learner_tiles<SS_MAXN>(P, s, t0, ntl);
    SS_STAMP(8);
    span_end(P.spans);
#undef SS_STAMP
#undef SS_BARRIER
}

}  // namespace sc
