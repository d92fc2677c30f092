// Chunk-wise leader selection (Section 4: the buffer is cut into chunks that are searched
// independently; Appendix E's demonstration keeps one index per chunk).
//
// The d coordinates form k consecutive chunks, chunk j = [floor(j*d/k), floor((j+1)*d/k)) -- or,
// with per-layer rates, each layer is cut that way into its own number of chunks -- and each chunk
// contributes the coordinate of acc = m + g that comes first in the order "larger |acc| first,
// lower index first".  One streaming read of g and m, one grid barrier:
//   S1  stream: one warp per chunk (lanes read the chunk in coalesced rows of 32), a hardware warp
//       max finds the largest key, a warp min the lowest index holding it; the owner stores the
//       composite (key << 31) | (2^31 - 1 - idx) in best[j]
//   S2  after the barrier: thread j turns best[j] into the bitmap bit and the index list entry;
//       a tile's prefix count needs no scan -- exactly one coordinate is kept per chunk, so the
//       count before coordinate p0 is the number of chunks before p0's chunk, plus one if that
//       chunk's pick lies before p0
#pragma once
#include "common.cuh"

namespace sc {

constexpr int CS_THREADS = 512;
constexpr int CS_BLOCKS_PER_SM = 2;
constexpr int CS_GROUP = 3;                     // chunks a warp works on at a time
constexpr int CS_UNROLL = 4;                    // rows of 32 coordinates of each of them in flight
constexpr int CS_RUN = 4 * CS_GROUP;            // consecutive chunks a warp takes before moving on

struct ChunkParams {
    const float* g;
    const float* m;
    uint32_t d, k;
    uint32_t spin_limit;
    unsigned long long* best;           // [k] composite of every chunk's pick, rewritten by every launch
    uint32_t* bitmap;                   // [ntiles * 32]
    uint32_t* tile_prefix;              // [ntiles + 1]
    uint32_t ntiles;
    uint32_t* ctrl;                     // status word at [CT_STATUS], path at [CT_PATH]
    unsigned long long* barrier;        // arrival counter used by this kernel only
    int32_t* out_idx;                   // [k] or nullptr
    unsigned long long* spans;          // nullptr, or where to accumulate the kernel's time span
    // layers (a single one when the whole vector has one rate): layer s covers coordinates
    // [layer_off[s], layer_off[s+1]) and owns chunks [layer_chunk0[s], layer_chunk0[s+1]) of the k chunks,
    // chunk jj of it being [floor(jj*size/keep), floor((jj+1)*size/keep)) past the layer's start
    uint32_t nl;
    const uint32_t* layer_off;          // [nl + 1]
    const uint32_t* layer_chunk0;       // [nl + 1]
};

constexpr uint32_t CS_MAX_LAYERS = 2048;

// Largest s with tab[s] <= x (tab ascending, tab[0] <= x < tab[n]).
__device__ __forceinline__ uint32_t layer_of(const uint32_t* tab, uint32_t n, uint32_t x) {
    uint32_t lo = 0, hi = n;                                            // answer in [lo, hi)
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (tab[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Chunk of coordinate p: the j with j*d < (p+1)*k <= (j+1)*d.
__device__ __forceinline__ uint32_t chunk_of(uint32_t p, uint32_t d, uint32_t k, double inv_d) {
    const uint64_t x = (uint64_t(p) + 1u) * k;
    uint64_t j = uint64_t(__double2ull_rd(double(x - 1u) * inv_d));       // within one of the answer
    if (j * d >= x) --j;
    else if ((j + 1u) * d < x) ++j;
    return uint32_t(j);
}

template <bool VEC, bool LAYERS>
__global__ void __launch_bounds__(CS_THREADS, CS_BLOCKS_PER_SM) chunk_select_kernel(const ChunkParams P) {
    __shared__ int flag;
    __shared__ uint32_t s_off[CS_MAX_LAYERS + 1], s_ch0[CS_MAX_LAYERS + 1];
    const uint32_t tid = threadIdx.x, lane = lane_id();
    const uint32_t nblocks = gridDim.x;
    const size_t gtid = size_t(blockIdx.x) * CS_THREADS + tid;
    const size_t gsize = size_t(nblocks) * CS_THREADS;
    const uint32_t d = P.d, k = P.k;
    GridBarrier gb;
    gb.arrive = P.barrier; gb.nblocks = nblocks; gb.status = P.ctrl + 1; gb.spin_limit = P.spin_limit;
    span_begin(P.spans);

    for (uint32_t i = threadIdx.x; i <= P.nl; i += CS_THREADS) { s_off[i] = P.layer_off[i]; s_ch0[i] = P.layer_chunk0[i]; }
    __syncthreads();
    // the bitmap is first written after the barrier
    {
        const size_t nv = size_t(P.ntiles) * 8;
        uint4* pv = reinterpret_cast<uint4*>(P.bitmap);
        for (size_t i = gtid; i < nv; i += gsize) pv[i] = make_uint4(0, 0, 0, 0);
    }

    // ---------------- S1: one warp per chunk ---------------------------------------------------------
    // Lane i reads elements lo + i, lo + i + 32, ... of a chunk (coalesced 128-byte rows; a chunk need
    // not start on a 16-byte boundary), keeps its best, and a hardware warp max plus a warp min pick the
    // chunk's winner.  Every chunk has one owner: plain stores, no atomics.
    const uint32_t warps = nblocks * (CS_THREADS / 32);
    const uint32_t gw = blockIdx.x * (CS_THREADS / 32) + (tid >> 5);

    // chunks j .. j+CS_GROUP-1 (those below jend), chunk g being [lo[g], lo[g+1])
    auto process_group = [&](const uint32_t (&lo)[CS_GROUP + 1], uint32_t j, uint32_t jend) {
        uint32_t bk[CS_GROUP], bi[CS_GROUP];                            // this lane's best key and its index, per chunk
        bool have[CS_GROUP];
#pragma unroll
        for (int g = 0; g < CS_GROUP; ++g) { bk[g] = 0; bi[g] = 0xFFFFFFFFu; have[g] = false; }
        uint32_t longest = 0;
#pragma unroll
        for (int g = 0; g < CS_GROUP; ++g) longest = max(longest, lo[g + 1] - lo[g]);
        if (LAYERS && longest <= 32u) {
            // no chunk longer than a row (the 25X layers: 25 coordinates per chunk; a layer sent whole: one):
            // one load per chunk and lane, no running best
            float g1[CS_GROUP], m1[CS_GROUP];
#pragma unroll
            for (int g = 0; g < CS_GROUP; ++g) {
                const uint32_t p = lo[g] + lane;
                if (p < lo[g + 1]) { g1[g] = P.g[p]; m1[g] = P.m[p]; }
            }
#pragma unroll
            for (int g = 0; g < CS_GROUP; ++g) {
                if (j + g >= jend) break;                               // warp-uniform
                const uint32_t p = lo[g] + lane;
                const bool in = p < lo[g + 1];
                const uint32_t key = in ? mag_key(__fadd_rn(m1[g], g1[g])) : 0u;
                const uint32_t mx = __reduce_max_sync(FULL, key);
                const uint32_t best_idx = __reduce_min_sync(FULL, (in && key == mx) ? p : 0xFFFFFFFFu);
                if (lane == 0) P.best[j + g] = composite(mx, best_idx);
            }
            return;
        }
        // rows of 32 coordinates, CS_UNROLL rows of every chunk of the group in flight at a time
        for (uint32_t off = 0; off < longest; off += 32u * CS_UNROLL) {
            float gv[CS_GROUP][CS_UNROLL], mv[CS_GROUP][CS_UNROLL];
#pragma unroll
            for (int g = 0; g < CS_GROUP; ++g)
#pragma unroll
                for (int u = 0; u < CS_UNROLL; ++u) {
                    const uint32_t p = lo[g] + off + u * 32u + lane;
                    if (p < lo[g + 1]) { gv[g][u] = P.g[p]; mv[g][u] = P.m[p]; }
                }
#pragma unroll
            for (int g = 0; g < CS_GROUP; ++g)
#pragma unroll
                for (int u = 0; u < CS_UNROLL; ++u) {
                    const uint32_t p = lo[g] + off + u * 32u + lane;
                    if (p < lo[g + 1]) {
                        const uint32_t key = mag_key(__fadd_rn(mv[g][u], gv[g][u]));
                        if (!have[g] || key > bk[g]) { bk[g] = key; bi[g] = p; have[g] = true; }   // strict: lower index stays on ties
                    }
                }
        }
#pragma unroll
        for (int g = 0; g < CS_GROUP; ++g) {
            if (j + g >= jend) break;                                   // warp-uniform
            const uint32_t mx = __reduce_max_sync(FULL, have[g] ? bk[g] : 0u);
            // among lanes holding the maximum, the lowest index wins
            const uint32_t best_idx = __reduce_min_sync(FULL, (have[g] && bk[g] == mx) ? bi[g] : 0xFFFFFFFFu);
            if (lane == 0) P.best[j + g] = composite(mx, best_idx);
        }
    };

    if (!LAYERS) {
        // one rate for the whole vector: groups of chunks dealt round-robin to the warps; j*d = q*k + r
        // is carried from one group of a warp to its next, so no division at all inside the loop
        const uint32_t dq = d / k, dr = d % k;                          // d = dq*k + dr
        const uint64_t sd = uint64_t(warps) * CS_GROUP * d;             // a warp advances by warps*CS_GROUP chunks
        const uint32_t sq = uint32_t(sd / k), sr = uint32_t(sd % k);    // sd = sq*k + sr
        const uint64_t j0 = uint64_t(gw) * CS_GROUP;
        uint32_t q = uint32_t(j0 * d / k), r = uint32_t(j0 * d % k);    // j*d = q*k + r for the group's first chunk
        for (uint64_t j = j0; j < k; j += uint64_t(warps) * CS_GROUP) {
            uint32_t lo[CS_GROUP + 1];
            uint32_t qq = q, rr = r;
            lo[0] = qq;
#pragma unroll
            for (int g = 1; g <= CS_GROUP; ++g) {
                qq += dq; rr += dr;                                     // rr, dr < k <= 2^31: no overflow
                if (rr >= k) { rr -= k; ++qq; }
                lo[g] = (j + g <= k) ? qq : lo[g - 1];                  // chunks past the last one are empty
            }
            process_group(lo, uint32_t(j), k);
            q += sq; r += sr;
            if (r >= k) { r -= k; ++q; }
        }
    } else {
        // per-layer rates: runs of consecutive chunks dealt round-robin to the warps; inside a run the
        // bounds advance without divisions: within layer s, jj*size = q*keep + r is carried along
        for (uint64_t j0 = uint64_t(gw) * CS_RUN; j0 < k; j0 += uint64_t(warps) * CS_RUN) {
            const uint32_t jend = uint32_t(min(uint64_t(k), j0 + CS_RUN));
            // layer of the run's first chunk and the chunk's position inside it
            uint32_t sl = layer_of(s_ch0, P.nl, uint32_t(j0));
            uint32_t size = s_off[sl + 1] - s_off[sl], keep = s_ch0[sl + 1] - s_ch0[sl];
            uint32_t jj = uint32_t(j0) - s_ch0[sl];
            uint32_t dq = size / keep, dr = size % keep;                // size = dq*keep + dr
            uint32_t q = uint32_t(uint64_t(jj) * size / keep), r = uint32_t(uint64_t(jj) * size % keep);
            uint32_t next_lo = s_off[sl] + q;                           // first coordinate of chunk j
            for (uint32_t j = uint32_t(j0); j < jend; j += CS_GROUP) {
                uint32_t lo[CS_GROUP + 1];
                lo[0] = next_lo;
#pragma unroll
                for (int g = 1; g <= CS_GROUP; ++g) {
                    if (j + g <= jend) {
                        // advance to the next chunk: same layer, or the first chunk of the next one
                        ++jj;
                        if (jj == keep && sl + 1 < P.nl) {
                            ++sl;
                            size = s_off[sl + 1] - s_off[sl]; keep = s_ch0[sl + 1] - s_ch0[sl];
                            dq = size / keep; dr = size % keep;
                            jj = 0; q = 0; r = 0;
                        } else {
                            q += dq; r += dr;                           // r, dr < keep <= 2^31: no overflow
                            if (r >= keep) { r -= keep; ++q; }
                        }
                        next_lo = s_off[sl] + q;                        // chunk k does not exist: this gives d
                    }
                    lo[g] = (j + g <= jend) ? next_lo : lo[g - 1];      // chunks past the run's end are empty here
                }
                process_group(lo, j, jend);
            }
        }
    }
    if (!grid_barrier(gb, &flag)) return;

    // ---------------- S2: bitmap, index list, tile prefixes ----------------------------------------
    for (size_t jj = gtid; jj < k; jj += gsize) {
        const unsigned long long b = __ldcg(&P.best[jj]);
        const uint32_t idx = 0x7FFFFFFFu - uint32_t(b & 0x7FFFFFFFull);
        if (b == 0ull || idx >= d) {                                    // every chunk holds at least one coordinate
            atomicCAS(P.ctrl + 1, DEV_OK, DEV_INTERNAL);
        } else {
            atomicOr(&P.bitmap[idx >> 5], 1u << (idx & 31u));
            if (P.out_idx) P.out_idx[jj] = int32_t(idx);
        }
    }
    for (size_t tile = gtid; tile <= P.ntiles; tile += gsize) {
        uint32_t prefix = k;                                            // the sentinel entry at ntiles
        if (tile < P.ntiles) {
            const uint32_t p0 = uint32_t(tile) * TILE;                  // < d
            const uint32_t sl = layer_of(s_off, P.nl, p0);
            const uint32_t size = s_off[sl + 1] - s_off[sl], keep = s_ch0[sl + 1] - s_ch0[sl];
            const uint32_t jt = s_ch0[sl] + chunk_of(p0 - s_off[sl], size, keep, 1.0 / double(size));
            const unsigned long long b = __ldcg(&P.best[jt]);
            const uint32_t idx = 0x7FFFFFFFu - uint32_t(b & 0x7FFFFFFFull);
            prefix = jt + (idx < p0 ? 1u : 0u);
        }
        P.tile_prefix[tile] = prefix;
    }
    if (gtid == 0) { P.ctrl[2] = 3u; P.ctrl[3] = k; }                   // path 3: chunk-wise; "candidates" = k
    span_end(P.spans);
}

}  // namespace sc
