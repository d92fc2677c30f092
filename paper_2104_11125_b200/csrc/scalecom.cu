// C-ABI of the CLT-k step (see include/scalecom.h): argument checks, workspace, launches.
#include "../../include/scalecom.h"

#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "chunk_select.cuh"
#include "diagnostics.cuh"
#include "exchange.cuh"
#include "layer_topk.cuh"
#include "learner_pass.cuh"
#include "small_step.cuh"
#include "topk_select.cuh"

using namespace sc;

struct scalecom_ctx {
    int device = 0;
    int64_t d = 0, k = 0;
    int32_t n = 0;
    float beta = 0.f, lr = 0.f;
    cudaStream_t stream = nullptr;

    // workspace (one allocation)
    void* ws = nullptr;
    size_t ws_bytes = 0;
    uint32_t *samp_hist = nullptr, *coarse_win = nullptr, *fine_hist = nullptr, *digit_hist = nullptr;
    uint32_t *ctrl = nullptr, *bitmap = nullptr, *tile_prefix = nullptr, *leader_hint = nullptr;
    uint32_t *block_tot = nullptr;
    uint32_t *small_tot = nullptr;     // [sms] winners per block of the one-kernel step
    uint32_t small_blocks = 0;         // its grid, 0: the vector is not eligible (too large, too many learners)
    bool fused_small = true;           // option: use the one-kernel step where it applies
    uint32_t tiles_per_block = 0;
    mutable uint32_t fine_parity = 0;  // which of the two fine histograms the next top-k launch counts in
    unsigned long long* barrier = nullptr;
    uint2* cand = nullptr;
    uint2* blist = nullptr;
    uint32_t seg_cap = 0, ntiles = 0;
    size_t ctrl_region_bytes = 0;      // prefix of the workspace that reset() clears

    // launch geometry
    int sms = 0;
    uint32_t topk_blocks = 0, lp_blocks = 0;
    mutable bool select_fresh = false; // the bitmap and prefix counts are those of this handle's last scalecom_select
    mutable bool bitmap_zero = false;  // the bitmap holds no bits (scalecom_compress leaves it so; selection kernels do not)
    uint32_t samp_stride = 1, samp_target = 1;
    float keep_frac = 0.0f;            // share of the leader's lines a step's selection asks L2 to hold for the learner pass
    bool l2_keep = true;               // SCALECOM_OPT_L2_KEEP

    // options
    uint32_t force_exact = 0;
    uint32_t use_hint = 1;
    int selector = SCALECOM_SELECTOR_TOPK;
    unsigned long long* chunk_best = nullptr;   // [k], allocated when the chunk-wise selector is first chosen
    uint32_t chunk_blocks = 0;
    void* lt_ws = nullptr;             // scratch of the per-layer exact selector (sized by nlayers), or nullptr
    size_t lt_bytes = 0;
    uint32_t lt_blocks = 0, lt_seg_cap = 0;
    uint32_t nlayers = 0;              // per-layer rates of the chunk-wise selector (0: one rate for the whole vector)
    uint32_t* layer_tab = nullptr;     // device [2][nlayers + 1]: coordinate offsets, chunk offsets
    uint32_t* one_layer_tab = nullptr; // device {0, d, 0, k}: the whole vector as one layer
    uint32_t spin_limit = 1u << 22;
    bool timing = false;
    bool fuse_update = true;
    float* gathered = nullptr;
    // in-kernel time spans: a ring of {selection ~start, end, learner pass ~start, end} per step
    unsigned long long* spans = nullptr;     // [EV_RING * 4] device words, allocated when first switched on
    bool span_timing = false;
    int64_t span_steps = 0;

    // host-buffer entry point
    float* stage_g = nullptr;          // n*d
    int32_t* stage_idx = nullptr;      // k
    float* stage_val = nullptr;        // k

    // kernel timing: a ring of 4 events per step
    static constexpr int EV_RING = 256;
    cudaEvent_t* ev = nullptr;         // [EV_RING * 4], created when timing is first switched on
    int64_t ev_steps = 0;              // steps recorded since the last read
    bool ev_has_update[EV_RING] = {};  // whether the step recorded the fourth event
    bool poisoned = false;
    int64_t launches = 0;

    // diagnostics scratch, allocated on first use
    float* diag_mean = nullptr;        // [d]
    float* diag_zero = nullptr;        // [d], all zero
    uint32_t* diag_bitmap = nullptr;   // [ntiles * 32]
    double* diag_acc = nullptr;        // [4]: overlap count (as u64) and three dot products

    int32_t* scratch_idx = nullptr;    // [k] index list the learner pass writes when the caller already has one
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <bool VEC>
cudaError_t launch_topk(const scalecom_ctx* c, const TopkParams& params) {
    c->bitmap_zero = false;
    c->select_fresh = false;
    // two copies of the fine histogram used in turn: a launch counts in one and clears the other behind its stream
    TopkParams P = params;
    P.fine_hist = c->fine_hist + size_t(c->fine_parity) * NFINE;
    P.fine_hist_next = c->fine_hist + size_t(c->fine_parity ^ 1u) * NFINE;
    c->fine_parity ^= 1u;
    void* args[] = {&P};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(&topk_select_kernel<VEC>), dim3(c->topk_blocks),
                                       dim3(TK_THREADS), args, sizeof(TopkShared), c->stream);
}

template <bool VEC>
cudaError_t launch_chunk(const scalecom_ctx* c, const ChunkParams& P) {
    c->bitmap_zero = false;
    c->select_fresh = false;
    void* args[] = {const_cast<ChunkParams*>(&P)};
    const void* fn = P.nl > 1 ? reinterpret_cast<const void*>(&chunk_select_kernel<VEC, true>)
                              : reinterpret_cast<const void*>(&chunk_select_kernel<VEC, false>);
    return cudaLaunchCooperativeKernel(fn, dim3(c->chunk_blocks), dim3(CS_THREADS), args, 0, c->stream);
}

// Scratch of the per-layer exact selector, made at the first launch after the layers were set.
int ensure_layer_ws(scalecom_ctx* c) {
    if (c->lt_ws) return SCALECOM_OK;
    int occ = 0, occ_unaligned = 0;
    if (cudaFuncSetAttribute(layer_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(sizeof(LayerTopkShared))) != cudaSuccess ||
        cudaFuncSetAttribute(layer_topk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(sizeof(LayerTopkShared))) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, layer_topk_kernel<true>, LT_THREADS, sizeof(LayerTopkShared)) !=
            cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_unaligned, layer_topk_kernel<false>, LT_THREADS,
                                                      sizeof(LayerTopkShared)) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    if (occ_unaligned < occ) occ = occ_unaligned;          // one grid serves both instantiations of the cooperative kernel
    if (occ < 1) return SCALECOM_ERR_CUDA;
    if (occ > LT_BLOCKS_PER_SM) occ = LT_BLOCKS_PER_SM;
    c->lt_blocks = uint32_t(c->sms * occ);
    const size_t nl = c->nlayers;
    // a warp's segment of undecided coordinates: an eighth of the coordinates it classifies (a few per cent are
    // expected); when one overflows the kernel falls back to its streaming route
    const size_t warps = size_t(c->lt_blocks) * LT_WARPS;
    c->lt_seg_cap = uint32_t((((size_t(c->d) / 8 + warps - 1) / warps + 31) / 32) * 32);
    if (c->lt_seg_cap < 128u) c->lt_seg_cap = 128u;
    c->lt_bytes = align_up(nl * LT_ROW * 4 + nl * 16 + 256 + size_t(c->lt_blocks) * 4, 256) + warps * c->lt_seg_cap * 8;
    if (cudaMalloc(&c->lt_ws, c->lt_bytes) != cudaSuccess) {
        cudaGetLastError();
        c->lt_ws = nullptr;
        return SCALECOM_ERR_ALLOC;
    }
    if (cudaMemsetAsync(c->lt_ws, 0, c->lt_bytes, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    return SCALECOM_OK;
}

LayerTopkParams make_layer_params(const scalecom_ctx* c, const float* g, const float* m, int32_t* out_idx,
                                  unsigned long long* span_slot) {
    LayerTopkParams P;
    const size_t nl = c->nlayers;
    char* base = static_cast<char*>(c->lt_ws);
    P.g = g; P.m = m; P.d = uint32_t(c->d); P.k = uint32_t(c->k);
    P.spin_limit = c->spin_limit;
    P.nl = c->nlayers;
    P.layer_off = c->layer_tab;
    P.layer_k0 = c->layer_tab + (nl + 1);
    P.ghist = reinterpret_cast<uint32_t*>(base);
    P.lstate = reinterpret_cast<uint4*>(base + nl * LT_ROW * 4);
    P.ctl = reinterpret_cast<uint32_t*>(base + nl * LT_ROW * 4 + nl * 16);
    P.block_tot = reinterpret_cast<uint32_t*>(base + nl * LT_ROW * 4 + nl * 16 + 256);
    P.cand = reinterpret_cast<uint2*>(base + align_up(nl * LT_ROW * 4 + nl * 16 + 256 + size_t(c->lt_blocks) * 4, 256));
    P.seg_cap = c->lt_seg_cap;
    P.force_stream = c->force_exact;
    P.bitmap = c->bitmap; P.tile_prefix = c->tile_prefix; P.ntiles = c->ntiles;
    P.ctrl = c->ctrl;
    P.barrier = c->barrier + 16;               // its own arrival counter (its grid differs from the other selectors')
    P.out_idx = out_idx;
    P.spans = span_slot;
    return P;
}

template <bool VEC>
cudaError_t launch_layer_topk(const scalecom_ctx* c, const LayerTopkParams& P) {
    c->bitmap_zero = false;
    c->select_fresh = false;
    void* args[] = {const_cast<LayerTopkParams*>(&P)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(&layer_topk_kernel<VEC>), dim3(c->lt_blocks),
                                       dim3(LT_THREADS), args, sizeof(LayerTopkShared), c->stream);
}

template <int N, bool VEC, int T, int L = LP_UNROLL / T, bool ONE = false,
          int MINB = (ONE ? LP_ONE_BLOCKS_PER_SM : LP_BLOCKS_PER_SM), bool EARLY = ONE, bool N1 = ONE>
cudaError_t launch_learner(const scalecom_ctx* c, int n, const float* const* grads, float* const* mem, const LearnerParams& P,
                           const PeerTable* peers = nullptr) {
    PeerTable pt;
    pt.n = 0;
    pt.tag = 0u;
    pt.done = nullptr;
    if (peers) pt = *peers;
    PtrTable<N> tab;
    for (int i = 0; i < N; ++i) {
        tab.g[i] = i < n ? grads[i] : nullptr;
        tab.m[i] = i < n ? mem[i] : nullptr;
    }
    const uint32_t nsuper = (c->ntiles + T - 1) / T;
    const uint32_t want = uint32_t(c->sms) * MINB;
    const uint32_t blocks = want < nsuper ? want : nsuper;
    learner_pass_kernel<N, VEC, T, L, ONE, MINB, EARLY, N1><<<blocks, LP_THREADS, 0, c->stream>>>(tab, P, pt);
    return cudaGetLastError();
}

// burst shape (tiles x learners) by learner count: few learners take more tiles per burst
inline int burst_tiles(int n) { return n >= 8 ? 1 : n >= 4 ? 2 : n >= 2 ? 4 : 0; }   // (1, 2, 4, 0: "8 or more", "4 to 7", "2 or 3", "1")

template <int N, bool VEC>
cudaError_t launch_learner_t(const scalecom_ctx* c, int n, const float* const* grads, float* const* mem,
                             const LearnerParams& P) {
    switch (burst_tiles(n)) {
        case 1:
            // 16 learners and more: one learner per burst at 6 blocks per SM, first burst requested early -- a block
            // then reads two vectors at a time instead of sixteen, which the DRAM system serves 3-7 % faster once
            // 32 and more vectors are streamed side by side
            if (n >= 16) return launch_learner<N, VEC, 1, 1, false, LP_MANY_BLOCKS_PER_SM, true>(c, n, grads, mem, P);
            // 9 to 14 learners: two bursts of equal size instead of eight and the rest
            if (N == 16 && n > 8 && n <= 10) return launch_learner<N, VEC, 1, 5>(c, n, grads, mem, P);
            if (N == 16 && n > 10 && n <= 12) return launch_learner<N, VEC, 1, 6>(c, n, grads, mem, P);
            if (N == 16 && n > 12 && n <= 14) return launch_learner<N, VEC, 1, 7>(c, n, grads, mem, P);
            return launch_learner<N, VEC, 1>(c, n, grads, mem, P);
        case 2: return launch_learner<N, VEC, LP_MID_T, 4, false, LP_MID_BLOCKS_PER_SM, LP_MID_EARLY>(c, n, grads, mem, P);
        // few learners: more blocks per SM and the first burst requested early
        case 4: return launch_learner<N, VEC, LP_FEW2_T, 2, false, LP_FEW2_BLOCKS_PER_SM, true>(c, n, grads, mem, P);
        default: return launch_learner<N, VEC, LP_FEW_T, 1, false, LP_FEW_BLOCKS_PER_SM, true, true>(c, n, grads, mem, P);
    }
}

// n learners of the caller's tables through the learner pass (n may be less than the handle's)
template <bool VEC>
cudaError_t launch_learner_n(const scalecom_ctx* c, int n, const float* const* grads, float* const* mem,
                             const LearnerParams& P) {
    if (n <= 16) return launch_learner_t<16, VEC>(c, n, grads, mem, P);
    if (n <= 128) return launch_learner_t<128, VEC>(c, n, grads, mem, P);
    return launch_learner_t<SCALECOM_MAX_LEARNERS, VEC>(c, n, grads, mem, P);
}

int init_workspace(scalecom_ctx* c) {
    c->bitmap_zero = false;
    c->select_fresh = false;
    c->fine_parity = 0;
    if (cudaMemsetAsync(c->ws, 0, c->ctrl_region_bytes, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    if (c->chunk_best && cudaMemsetAsync(c->chunk_best, 0, size_t(c->k) * 8, c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    if (c->lt_ws && cudaMemsetAsync(c->lt_ws, 0, c->lt_bytes, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    return SCALECOM_OK;
}

int check_step_args(scalecom_ctx* c, const void* const* grads, const void* const* mem, const void* weights, int64_t t,
                    const void* out_idx, const void* out_val) {
    if (!c || !grads || !mem || !out_idx || !out_val) return SCALECOM_ERR_NULL_PTR;
    if (t < 0) return SCALECOM_ERR_INVALID_ARG;
    if (c->poisoned) return SCALECOM_ERR_BAD_STATE;
    for (int i = 0; i < c->n; ++i)
        if (!grads[i] || !mem[i]) return SCALECOM_ERR_NULL_PTR;
    if (out_idx == out_val || out_idx == weights || out_val == weights) return SCALECOM_ERR_ALIAS;
    for (int i = 0; i < c->n; ++i) {
        const void* a[2] = {grads[i], mem[i]};
        for (const void* x : a)
            if (x == weights || x == out_idx || x == out_val) return SCALECOM_ERR_ALIAS;
        if (grads[i] == mem[i]) return SCALECOM_ERR_ALIAS;
    }
    if (c->n <= 64) {            // quadratic check only where it is cheap; mem buffers are written, so they must be distinct
        for (int i = 0; i < c->n; ++i)
            for (int j = 0; j < c->n; ++j) {
                if (i != j && mem[i] == mem[j]) return SCALECOM_ERR_ALIAS;
                if (grads[i] == mem[j]) return SCALECOM_ERR_ALIAS;
            }
    }
    return SCALECOM_OK;
}

TopkParams make_topk_params(const scalecom_ctx* c, const float* g, const float* m, uint32_t* leader_hint, bool use_hint,
                            unsigned long long* span_slot) {
    TopkParams tp;
    tp.g = g;
    tp.m = m;
    tp.d = uint32_t(c->d);
    tp.k = uint32_t(c->k);
    tp.samp_stride = c->samp_stride;
    tp.samp_target = c->samp_target;
    tp.force_exact = c->force_exact;
    tp.use_hint = use_hint ? c->use_hint : 0u;
    tp.leader_hint = leader_hint;
    tp.all_hints = leader_hint ? c->leader_hint : nullptr;
    tp.n_hints = uint32_t(c->n);
    tp.spin_limit = c->spin_limit;
    tp.keep_frac = 0.0f;           // set by a step, whose learner pass reads the leader's vectors again
    tp.samp_hist = c->samp_hist;
    tp.coarse_win = c->coarse_win;
    tp.fine_hist = nullptr;        // set by launch_topk
    tp.fine_hist_next = nullptr;
    tp.digit_hist = c->digit_hist;
    tp.ctrl = c->ctrl;
    tp.barrier = c->barrier;
    tp.cand = c->cand;
    tp.seg_cap = c->seg_cap;
    tp.blist = c->blist;
    tp.bitmap = c->bitmap;
    tp.tile_prefix = c->tile_prefix;
    tp.block_tot = c->block_tot;
    tp.ntiles = c->ntiles;
    tp.tiles_per_block = c->tiles_per_block;
    tp.out_idx = nullptr;          // (scalecom_select asks for the list; a step's learner pass writes it from its ranks)
    tp.spans = span_slot;
    return tp;
}

// The whole step as one cooperative kernel (vectors whose g and m fit the L2 cache; see small_step.cuh).
cudaError_t launch_small_step(scalecom_ctx* c, const float* const* grads, float* const* mem, float* weights, int leader,
                              int32_t* out_idx, float* out_val, unsigned long long* span_slot) {
    SmallParams P;
    for (int i = 0; i < SS_MAXN; ++i) {
        P.tab.g[i] = i < c->n ? grads[i] : nullptr;
        P.tab.m[i] = i < c->n ? mem[i] : nullptr;
    }
    P.d = uint32_t(c->d); P.k = uint32_t(c->k); P.ntiles = c->ntiles;
    P.n = c->n; P.leader = leader;
    P.beta = c->beta; P.omb = 1.0f - c->beta; P.lr = c->lr; P.nf = float(c->n);
    P.force_exact = c->force_exact; P.use_hint = c->use_hint; P.spin_limit = c->spin_limit;
    P.leader_hint = c->leader_hint + leader; P.all_hints = c->leader_hint; P.n_hints = uint32_t(c->n);
    P.key_hist = c->samp_hist; P.coarse_win = c->coarse_win;
    P.fine_hist = c->fine_hist + size_t(c->fine_parity) * NFINE;
    P.fine_hist_next = c->fine_hist + size_t(c->fine_parity ^ 1u) * NFINE;
    c->fine_parity ^= 1u;
    P.digit_hist = c->digit_hist; P.block_tot = c->small_tot; P.ctrl = c->ctrl;
    P.barrier = c->barrier + 24;               // its own arrival counter: its grid differs from the other kernels'
    P.blist = c->blist;
    P.out_idx = out_idx; P.out_val = out_val; P.gathered = c->gathered;
    P.weights = (weights && c->fuse_update) ? weights : nullptr;
    P.spans = span_slot;
    c->bitmap_zero = false;
    c->select_fresh = false;
    void* args[] = {&P};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(&small_step_kernel), dim3(c->small_blocks),
                                       dim3(SS_THREADS), args, sizeof(SmallShared), c->stream);
}

int do_step(scalecom_ctx* c, const float* const* grads, float* const* mem, float* weights, int64_t t, int32_t* out_idx,
            float* out_val) {
    const int leader = int(t % c->n);
    if (c->selector == SCALECOM_SELECTOR_LAYER_TOPK) {
        if (!c->nlayers) return SCALECOM_ERR_BAD_STATE;        // this selector has no meaning without layers
        const int rc = ensure_layer_ws(c);
        if (rc != SCALECOM_OK) return rc;
    }

    unsigned long long* const span_slot =
        (c->span_timing && c->spans) ? c->spans + 4 * (c->span_steps % scalecom_ctx::EV_RING) : nullptr;
    // a slot of the ring that already holds an earlier step's span starts from zero again
    if (span_slot && c->span_steps >= scalecom_ctx::EV_RING &&
        cudaMemsetAsync(span_slot, 0, 4 * sizeof(unsigned long long), c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    TopkParams tp = make_topk_params(c, grads[leader], mem[leader], c->leader_hint + leader, true, span_slot);
    tp.keep_frac = c->l2_keep ? c->keep_frac : 0.0f;

    LearnerParams lp;
    lp.d = uint32_t(c->d);
    lp.k = uint32_t(c->k);
    lp.ntiles = c->ntiles;
    lp.n = c->n;
    lp.beta = c->beta;
    lp.omb = 1.0f - c->beta;
    lp.lr = c->lr;
    lp.nf = float(c->n);
    lp.bitmap = c->bitmap; lp.bitmap_clear = nullptr;
    lp.tile_prefix = c->tile_prefix;
    lp.out_val = out_val;
    lp.out_idx = out_idx;
    lp.gathered = c->gathered;
    lp.weights = (weights && c->fuse_update) ? weights : nullptr;
    lp.spans = span_slot ? span_slot + 2 : nullptr;
    lp.status = c->ctrl + CT_STATUS;

    bool vec_all = true;
    for (int i = 0; i < c->n; ++i) vec_all = vec_all && aligned16(grads[i]) && aligned16(mem[i]);
    const bool vec_leader = aligned16(tp.g) && aligned16(tp.m);

    const bool tm = c->timing && c->ev;
    cudaEvent_t* ev = tm ? c->ev + 4 * (c->ev_steps % scalecom_ctx::EV_RING) : nullptr;
    if (tm && cudaEventRecord(ev[0], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    cudaError_t e;
    if (c->small_blocks && c->fused_small && vec_all && c->selector == SCALECOM_SELECTOR_TOPK) {
        // one kernel for the whole step; in the per-kernel figures it takes the learner pass's place and the
        // selection's interval is empty
        if (tm && cudaEventRecord(ev[1], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
        e = launch_small_step(c, grads, mem, weights, leader, out_idx, out_val, span_slot ? span_slot + 2 : nullptr);
        if (e != cudaSuccess) { cudaGetLastError(); return SCALECOM_ERR_CUDA; }
        ++c->launches;
        if (tm && cudaEventRecord(ev[2], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
        if (weights && !c->fuse_update) {
            const uint32_t blocks = uint32_t((c->k + 255) / 256);
            apply_update_kernel<<<blocks < 4096u ? blocks : 4096u, 256, 0, c->stream>>>(weights, out_idx, out_val,
                                                                                       uint32_t(c->k), c->lr, c->ctrl + CT_STATUS);
            if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
            ++c->launches;
        }
        if (tm) {
            c->ev_has_update[c->ev_steps % scalecom_ctx::EV_RING] = weights && !c->fuse_update;
            if (weights && !c->fuse_update && cudaEventRecord(ev[3], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
            ++c->ev_steps;
        }
        if (span_slot) ++c->span_steps;
        return SCALECOM_OK;
    }
    if (c->selector == SCALECOM_SELECTOR_CHUNK) {
        ChunkParams cp;
        cp.g = tp.g; cp.m = tp.m; cp.d = tp.d; cp.k = tp.k;
        cp.spin_limit = c->spin_limit;
        cp.best = c->chunk_best;
        cp.bitmap = c->bitmap; cp.tile_prefix = c->tile_prefix; cp.ntiles = c->ntiles;
        cp.ctrl = c->ctrl;
        cp.barrier = c->barrier + 8;               // its own arrival counter: the grid differs from the top-k kernel's
        cp.out_idx = nullptr;                      // written by the learner pass
        cp.spans = span_slot;
        // one layer spanning the whole vector unless the caller set per-layer rates
        cp.nl = c->nlayers ? c->nlayers : 1u;
        cp.layer_off = c->nlayers ? c->layer_tab : c->one_layer_tab;
        cp.layer_chunk0 = cp.layer_off + (cp.nl + 1);
        e = vec_leader ? launch_chunk<true>(c, cp) : launch_chunk<false>(c, cp);
    } else if (c->selector == SCALECOM_SELECTOR_LAYER_TOPK) {
        const LayerTopkParams P = make_layer_params(c, tp.g, tp.m, nullptr, span_slot);
        e = vec_leader ? launch_layer_topk<true>(c, P) : launch_layer_topk<false>(c, P);
    } else {
        e = vec_leader ? launch_topk<true>(c, tp) : launch_topk<false>(c, tp);
    }
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    if (tm && cudaEventRecord(ev[1], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    e = vec_all ? launch_learner_n<true>(c, c->n, grads, mem, lp) : launch_learner_n<false>(c, c->n, grads, mem, lp);
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    if (tm && cudaEventRecord(ev[2], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    if (weights && !c->fuse_update) {
        const uint32_t blocks = uint32_t((c->k + 255) / 256);
        apply_update_kernel<<<blocks < 4096u ? blocks : 4096u, 256, 0, c->stream>>>(weights, out_idx, out_val,
                                                                                   uint32_t(c->k), c->lr, c->ctrl + CT_STATUS);
        if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
        ++c->launches;
    }
    if (tm) {
        // without a separate update kernel the third interval is empty: one event fewer on the stream
        c->ev_has_update[c->ev_steps % scalecom_ctx::EV_RING] = weights && !c->fuse_update;
        if (weights && !c->fuse_update && cudaEventRecord(ev[3], c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
        ++c->ev_steps;
    }
    if (span_slot) ++c->span_steps;
    return SCALECOM_OK;
}

}  // namespace

extern "C" {

int scalecom_create(scalecom_ctx** out, int64_t d, int32_t n, int64_t k, float beta, float lr) {
    if (!out) return SCALECOM_ERR_NULL_PTR;
    *out = nullptr;
    if (d < 1 || d > 2147483647LL || n < 1 || n > SCALECOM_MAX_LEARNERS || k < 1 || k > d) return SCALECOM_ERR_INVALID_ARG;
    if (!(beta > 0.0f) || !(beta <= 1.0f) || !std::isfinite(lr)) return SCALECOM_ERR_INVALID_ARG;

    scalecom_ctx* c = new (std::nothrow) scalecom_ctx;
    if (!c) return SCALECOM_ERR_ALLOC;
    c->d = d; c->n = n; c->k = k; c->beta = beta; c->lr = lr;

    int coop = 0, occ_topk = 0, occ_lp = 0;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
    // one grid serves both instantiations of the cooperative selection kernel: the smaller occupancy counts
    occ_topk = 1 << 20;
    auto prepare = [&](auto kernel) {
        int o = 0;
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(TopkShared)));
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kernel, TK_THREADS, sizeof(TopkShared));
        if (o < occ_topk) occ_topk = o;
    };
    prepare(topk_select_kernel<true>);
    prepare(topk_select_kernel<false>);
    if (e == cudaSuccess)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_lp, learner_pass_kernel<16, true, 1, LP_UNROLL>, LP_THREADS, 0);
    if (e != cudaSuccess || !coop || occ_topk < 1 || occ_lp < 1) {
        cudaGetLastError();
        delete c;
        return SCALECOM_ERR_CUDA;
    }
    if (occ_topk > TK_BLOCKS_PER_SM) occ_topk = TK_BLOCKS_PER_SM;

    c->ntiles = uint32_t((d + TILE - 1) / TILE);
    // persistent selection grid: every resident slot, but no more blocks than there are chunks of work
    const uint32_t chunks = uint32_t((d + TK_CHUNK - 1) / TK_CHUNK);
    c->topk_blocks = uint32_t(c->sms * occ_topk);
    if (c->topk_blocks > chunks) c->topk_blocks = chunks;
    if (c->topk_blocks < 1) c->topk_blocks = 1;
    c->tiles_per_block = (c->ntiles + c->topk_blocks - 1) / c->topk_blocks;
    {
        // the one-kernel step: at most SS_MAXN learners, a block's share of the tiles within its shared-memory
        // bitmap, and all g and m of a step (8 n d bytes) within 64 MB, about half the L2 cache
        int occ_small = 0;
        const bool fits = n <= SS_MAXN && uint64_t(c->ntiles) <= uint64_t(SS_TILES) * uint64_t(c->sms) &&
                          uint64_t(n) * uint64_t(d) <= (1ull << 23);
        if (fits &&
            cudaFuncSetAttribute(small_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(SmallShared))) == cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_small, small_step_kernel, SS_THREADS, sizeof(SmallShared)) == cudaSuccess &&
            occ_small >= 1)
            c->small_blocks = c->ntiles < uint32_t(c->sms) ? c->ntiles : uint32_t(c->sms);
        cudaGetLastError();
    }
    c->lp_blocks = uint32_t(c->sms * occ_lp);
    if (c->lp_blocks > c->ntiles) c->lp_blocks = c->ntiles;

    // The learner pass reads the leader's g and m again: the selection marks a share of those lines to be replaced
    // last -- a quarter of them (measured best on d = 25.6 M), and no more than 0.4 of the L2 cache.  Vectors of
    // which the cache could hold under a twentieth are streamed with the default policy (the marked stream measured
    // 5 % slower on d = 354 M, where there is nothing to gain).
    {
        int l2 = 0;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, c->device) != cudaSuccess) { l2 = 0; cudaGetLastError(); }
        const double share = 0.4 * double(l2) / (8.0 * double(d));
        c->keep_frac = share < KEEP_SHARE_MIN ? 0.0f : float(share < KEEP_SHARE ? share : KEEP_SHARE);
    }

    // sampling rate: about 2^18 sampled keys or 1/64 of the vector, whichever is more
    uint32_t stride = 1;
    while (stride < 64 && (d / (2 * stride)) >= (1 << 18)) stride *= 2;
    c->samp_stride = stride;
    {
        const int64_t span = int64_t(SAMPLE_GRANULE) * stride;
        const int64_t full = d / span, rem = d % span;
        const int64_t ns = full * SAMPLE_GRANULE + (rem < SAMPLE_GRANULE ? rem : SAMPLE_GRANULE);
        if (stride == 1) {
            c->samp_target = uint32_t(k);                                  // the "sample" is the whole vector: exact bin
        } else {
            const double ks = double(k) * double(ns) / double(d);
            double tgt = std::ceil(ks + 6.0 * std::sqrt(ks) + 8.0);
            if (tgt > double(ns)) tgt = double(ns);
            c->samp_target = uint32_t(tgt);
        }
    }
    {
        // candidate segment per warp of the selection grid: room for 6k survivors overall plus slack
        // for uneven spread, never more than the warp's share of the vector
        const int64_t warps = int64_t(c->topk_blocks) * TK_WARPS;
        int64_t cap = (6 * k + warps - 1) / warps + 32;
        const int64_t share = (d + warps - 1) / warps + 32;
        if (cap > share) cap = share;
        c->seg_cap = uint32_t(cap);
    }

    // carve the workspace; the first region (histograms, counters) is what reset() clears
    size_t off = 0;
    auto carve = [&](size_t bytes) { const size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_samp = carve(NCOARSE * 4), o_cw = carve((WIN + 1) * 4), o_ctrl = carve(CT_WORDS * 4), o_bar = carve(256);
    const size_t o_lh = carve(size_t(n) * 4), o_bt = carve(size_t(c->topk_blocks) * 4), o_st = carve(size_t(c->sms) * 4);
    const size_t o_fine = carve(2 * size_t(NFINE) * 4), o_dh = carve(size_t(DH_PASSES) * DH_BINS * 4);
    c->ctrl_region_bytes = off;                 // everything the kernel expects to find zero
    const size_t o_cand = carve(size_t(c->seg_cap) * c->topk_blocks * TK_WARPS * 8), o_bl = carve(size_t(BCAP) * 8);
    const size_t o_bm = carve(size_t(c->ntiles) * 32 * 4), o_tp = carve((size_t(c->ntiles) + 1) * 4);
    c->ws_bytes = off;
    if (cudaMalloc(&c->ws, c->ws_bytes) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return SCALECOM_ERR_ALLOC;
    }
    char* base = static_cast<char*>(c->ws);
    c->samp_hist = reinterpret_cast<uint32_t*>(base + o_samp);
    c->coarse_win = reinterpret_cast<uint32_t*>(base + o_cw);
    c->ctrl = reinterpret_cast<uint32_t*>(base + o_ctrl);
    c->barrier = reinterpret_cast<unsigned long long*>(base + o_bar);
    c->block_tot = reinterpret_cast<uint32_t*>(base + o_bt);
    c->small_tot = reinterpret_cast<uint32_t*>(base + o_st);
    c->leader_hint = reinterpret_cast<uint32_t*>(base + o_lh);
    c->fine_hist = reinterpret_cast<uint32_t*>(base + o_fine);
    c->digit_hist = reinterpret_cast<uint32_t*>(base + o_dh);
    c->cand = reinterpret_cast<uint2*>(base + o_cand);
    c->blist = reinterpret_cast<uint2*>(base + o_bl);
    c->bitmap = reinterpret_cast<uint32_t*>(base + o_bm);
    c->tile_prefix = reinterpret_cast<uint32_t*>(base + o_tp);

    const bool ok = init_workspace(c) == SCALECOM_OK;
    if (!ok || cudaStreamSynchronize(c->stream) != cudaSuccess) {
        cudaGetLastError();
        scalecom_destroy(c);
        return SCALECOM_ERR_CUDA;
    }
    *out = c;
    return SCALECOM_OK;
}

int scalecom_step(scalecom_ctx* c, const float* const* grads, float* const* mem, float* weights, int64_t t,
                  int32_t* out_idx, float* out_val) {
    const int rc = check_step_args(c, reinterpret_cast<const void* const*>(grads),
                                   reinterpret_cast<const void* const*>(mem), weights, t, out_idx, out_val);
    if (rc != SCALECOM_OK) return rc;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    return do_step(c, grads, mem, weights, t, out_idx, out_val);
}

int scalecom_step_host(scalecom_ctx* c, const float* const* host_grads, float* const* mem, float* weights, int64_t t,
                       int32_t* host_idx, float* host_val) {
    // every argument is checked before anything is allocated, copied or launched (host and device pointers share
    // one address space, so the distinctness checks of scalecom_step apply as they are)
    int rc = check_step_args(c, reinterpret_cast<const void* const*>(host_grads), reinterpret_cast<const void* const*>(mem),
                             weights, t, host_idx, host_val);
    if (rc != SCALECOM_OK) return rc;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    if (!c->stage_g) {
        const size_t gbytes = size_t(c->n) * size_t(c->d) * 4;
        if (cudaMalloc(reinterpret_cast<void**>(&c->stage_g), gbytes) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&c->stage_idx), size_t(c->k) * 4) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&c->stage_val), size_t(c->k) * 4) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(c->stage_g); cudaFree(c->stage_idx); cudaFree(c->stage_val);
            c->stage_g = nullptr; c->stage_idx = nullptr; c->stage_val = nullptr;
            return SCALECOM_ERR_ALLOC;
        }
    }
    const float* dev_g[SCALECOM_MAX_LEARNERS];
    for (int i = 0; i < c->n; ++i) {
        float* dst = c->stage_g + size_t(i) * size_t(c->d);
        dev_g[i] = dst;
        if (cudaMemcpyAsync(dst, host_grads[i], size_t(c->d) * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
            return SCALECOM_ERR_CUDA;
    }
    rc = do_step(c, dev_g, mem, weights, t, c->stage_idx, c->stage_val);
    if (rc != SCALECOM_OK) return rc;
    if (cudaMemcpyAsync(host_idx, c->stage_idx, size_t(c->k) * 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaMemcpyAsync(host_val, c->stage_val, size_t(c->k) * 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    return SCALECOM_OK;
}

void scalecom_destroy(scalecom_ctx* c) {
    if (!c) return;
    DeviceGuard guard(c->device);
    cudaStreamSynchronize(c->stream);
    if (c->ev) {
        for (int i = 0; i < scalecom_ctx::EV_RING * 4; ++i)
            if (c->ev[i]) cudaEventDestroy(c->ev[i]);
        delete[] c->ev;
    }
    cudaFree(c->ws);
    cudaFree(c->chunk_best);
    cudaFree(c->lt_ws);
    cudaFree(c->layer_tab);
    cudaFree(c->one_layer_tab);
    cudaFree(c->spans);
    cudaFree(c->diag_mean);
    cudaFree(c->diag_zero);
    cudaFree(c->diag_bitmap);
    cudaFree(c->diag_acc);
    cudaFree(c->scratch_idx);
    cudaFree(c->stage_g);
    cudaFree(c->stage_idx);
    cudaFree(c->stage_val);
    cudaGetLastError();
    delete c;
}

int scalecom_set_stream(scalecom_ctx* c, void* cuda_stream) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;   // scratch is shared between steps
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    return SCALECOM_OK;
}

int scalecom_set_layers(scalecom_ctx* c, int32_t nlayers, const int64_t* sizes, const int64_t* keep) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;   // a step may still read the old table
    if (nlayers == 0) {
        cudaFree(c->layer_tab);
        cudaFree(c->lt_ws);
        c->layer_tab = nullptr;
        c->lt_ws = nullptr;
        c->nlayers = 0;
        return SCALECOM_OK;
    }
    if (nlayers < 0 || nlayers > int32_t(CS_MAX_LAYERS)) return SCALECOM_ERR_INVALID_ARG;
    if (!sizes || !keep) return SCALECOM_ERR_NULL_PTR;
    uint32_t* h = new (std::nothrow) uint32_t[2 * (size_t(nlayers) + 1)];
    if (!h) return SCALECOM_ERR_ALLOC;
    int64_t off = 0, ch = 0;
    bool ok = true;
    for (int32_t s = 0; s < nlayers && ok; ++s) {
        ok = sizes[s] >= 1 && keep[s] >= 1 && keep[s] <= sizes[s] && sizes[s] <= c->d - off;
        h[s] = uint32_t(off);
        h[nlayers + 1 + s] = uint32_t(ch);
        off += sizes[s];
        ch += keep[s];
    }
    ok = ok && off == c->d && ch == c->k;
    h[nlayers] = uint32_t(c->d);
    h[2 * nlayers + 1] = uint32_t(c->k);
    int rc = ok ? SCALECOM_OK : SCALECOM_ERR_INVALID_ARG;
    if (ok) {
        uint32_t* dev = nullptr;
        const size_t bytes = 2 * (size_t(nlayers) + 1) * 4;
        if (cudaMalloc(reinterpret_cast<void**>(&dev), bytes) != cudaSuccess) {
            cudaGetLastError();
            rc = SCALECOM_ERR_ALLOC;
        } else if (cudaMemcpy(dev, h, bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(dev);
            rc = SCALECOM_ERR_CUDA;
        } else {
            cudaFree(c->layer_tab);
            cudaFree(c->lt_ws);                    // sized by the number of layers: made again at the next launch
            c->lt_ws = nullptr;
            c->layer_tab = dev;
            c->nlayers = uint32_t(nlayers);
        }
    }
    delete[] h;
    return rc;
}

int scalecom_set_gathered(scalecom_ctx* c, float* dev_gathered) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    c->gathered = dev_gathered;
    return SCALECOM_OK;
}

int scalecom_apply_update(scalecom_ctx* c, float* weights, const int32_t* idx, const float* val, int64_t k, float lr) {
    if (!c || !weights || !idx || !val) return SCALECOM_ERR_NULL_PTR;
    if (k < 0 || k > c->d || !std::isfinite(lr)) return SCALECOM_ERR_INVALID_ARG;
    if (k == 0) return SCALECOM_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    const uint32_t blocks = uint32_t((k + 255) / 256);
    apply_update_kernel<<<blocks < 4096u ? blocks : 4096u, 256, 0, c->stream>>>(weights, idx, val, uint32_t(k), lr,
                                                                               c->ctrl + CT_STATUS);
    if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    return SCALECOM_OK;
}

int scalecom_select(scalecom_ctx* c, const float* g, const float* m, int32_t* out_idx) {
    if (!c || !g || !m || !out_idx) return SCALECOM_ERR_NULL_PTR;
    if (c->poisoned) return SCALECOM_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    const bool vec = aligned16(g) && aligned16(m);
    cudaError_t e;
    if (c->selector == SCALECOM_SELECTOR_CHUNK) {
        ChunkParams cp;
        cp.g = g; cp.m = m; cp.d = uint32_t(c->d); cp.k = uint32_t(c->k);
        cp.spin_limit = c->spin_limit;
        cp.best = c->chunk_best;
        cp.bitmap = c->bitmap; cp.tile_prefix = c->tile_prefix; cp.ntiles = c->ntiles;
        cp.ctrl = c->ctrl;
        cp.barrier = c->barrier + 8;
        cp.out_idx = out_idx;
        cp.spans = nullptr;
        cp.nl = c->nlayers ? c->nlayers : 1u;
        cp.layer_off = c->nlayers ? c->layer_tab : c->one_layer_tab;
        cp.layer_chunk0 = cp.layer_off + (cp.nl + 1);
        e = vec ? launch_chunk<true>(c, cp) : launch_chunk<false>(c, cp);
    } else if (c->selector == SCALECOM_SELECTOR_LAYER_TOPK) {
        if (!c->nlayers) return SCALECOM_ERR_BAD_STATE;
        const int rc = ensure_layer_ws(c);
        if (rc != SCALECOM_OK) return rc;
        const LayerTopkParams P = make_layer_params(c, g, m, out_idx, nullptr);
        e = vec ? launch_layer_topk<true>(c, P) : launch_layer_topk<false>(c, P);
    } else {
        // one vector, one hint slot: the handle of a learner-per-GPU rank always sees the same learner
        TopkParams tp = make_topk_params(c, g, m, c->leader_hint, true, nullptr);
        tp.out_idx = out_idx;
        e = vec ? launch_topk<true>(c, tp) : launch_topk<false>(c, tp);
    }
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    c->select_fresh = true;
    return SCALECOM_OK;
}

int scalecom_compress(scalecom_ctx* c, const float* g, float* m, const int32_t* idx, float* out_gathered) {
    return scalecom_compress_scatter(c, g, m, idx, out_gathered, nullptr, 0, nullptr, 0u);
}

int scalecom_compress_scatter(scalecom_ctx* c, const float* g, float* m, const int32_t* idx, float* out_gathered,
                              float* const* dst, int32_t n_dst, uint32_t* const* flag_dst, uint32_t tag) {
    if (!c || !g || !m || !out_gathered || (n_dst > 0 && !dst)) return SCALECOM_ERR_NULL_PTR;
    if (n_dst < 0 || n_dst > LP_MAX_PEERS || (flag_dst && tag == 0u)) return SCALECOM_ERR_INVALID_ARG;
    PeerTable peers;
    peers.n = n_dst;
    peers.tag = (flag_dst && n_dst > 0) ? tag : 0u;
    peers.done = c->ctrl + CT_PEER_DONE;
    for (int i = 0; i < n_dst; ++i) {
        peers.flag[i] = nullptr;
        if (peers.tag) {
            if (!flag_dst[i]) return SCALECOM_ERR_NULL_PTR;
            peers.flag[i] = flag_dst[i];
        }
        if (!dst[i]) return SCALECOM_ERR_NULL_PTR;
        if (static_cast<const void*>(dst[i]) == g || static_cast<const void*>(dst[i]) == m ||
            (idx && static_cast<const void*>(dst[i]) == idx))
            return SCALECOM_ERR_ALIAS;
        peers.dst[i] = dst[i];
    }
    if (static_cast<const void*>(g) == static_cast<const void*>(m) || (idx && static_cast<const void*>(idx) == out_gathered))
        return SCALECOM_ERR_ALIAS;
    if (c->poisoned || (!idx && !c->select_fresh)) return SCALECOM_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    if (!c->scratch_idx && cudaMalloc(reinterpret_cast<void**>(&c->scratch_idx), size_t(c->k) * 4) != cudaSuccess) {
        cudaGetLastError();
        c->scratch_idx = nullptr;
        return SCALECOM_ERR_ALLOC;
    }
    // the received index list -> bitmap and tile prefixes in the handle's workspace
    // (the single-learner pass below zeroes every bitmap word it has read, so only a bitmap that a selection
    // kernel wrote since, or a fresh workspace, has to be cleared here)
    // idx == NULL: the list is the one this handle's own scalecom_select has just produced, and the bitmap and
    // prefix counts it left in the workspace are used as they are
    if (idx) {
        if (!c->bitmap_zero &&
            cudaMemsetAsync(c->bitmap, 0, size_t(c->ntiles) * 32 * 4, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
        const uint32_t want = uint32_t((c->k + 255) / 256), cap = uint32_t(c->sms) * 16u;
        indices_to_bitmap_kernel<<<want < cap ? want : cap, 256, 0, c->stream>>>(idx, uint32_t(c->k), uint32_t(c->d),
                                                                                c->ntiles, c->bitmap, c->tile_prefix,
                                                                                c->ctrl + CT_STATUS);
        if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
        ++c->launches;
    }
    c->bitmap_zero = true;                 // (the pass below leaves it so)
    c->select_fresh = false;
    // this learner's share of steps 1, 3 and 4: a learner pass over one learner; with n = 1 the
    // "average" it writes is the gathered value itself (x / 1 is exact)
    LearnerParams lp;
    lp.d = uint32_t(c->d); lp.k = uint32_t(c->k); lp.ntiles = c->ntiles;
    lp.n = 1;
    lp.beta = c->beta; lp.omb = 1.0f - c->beta; lp.lr = c->lr; lp.nf = 1.0f;
    lp.bitmap = c->bitmap; lp.bitmap_clear = c->bitmap; lp.tile_prefix = c->tile_prefix;
    lp.out_val = out_gathered; lp.out_idx = c->scratch_idx;
    lp.gathered = nullptr; lp.weights = nullptr; lp.spans = nullptr;
    lp.status = c->ctrl + CT_STATUS;
    const float* gp[1] = {g};
    float* mp[1] = {m};
    const cudaError_t e = (aligned16(g) && aligned16(m)) ? launch_learner<16, true, LP_ONE_T, 1, true>(c, 1, gp, mp, lp, &peers)
                                                         : launch_learner<16, false, LP_ONE_T, 1, true>(c, 1, gp, mp, lp, &peers);
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    return SCALECOM_OK;
}

int scalecom_enable_peer_access(scalecom_ctx* c, int32_t peer_device) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) { cudaGetLastError(); return SCALECOM_ERR_CUDA; }
    if (peer_device < 0 || peer_device >= ndev) return SCALECOM_ERR_INVALID_ARG;
    if (peer_device == c->device) return SCALECOM_OK;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    int can = 0;
    if (cudaDeviceCanAccessPeer(&can, c->device, peer_device) != cudaSuccess) { cudaGetLastError(); return SCALECOM_ERR_CUDA; }
    if (!can) return SCALECOM_ERR_INVALID_ARG;
    const cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
    if (e == cudaErrorPeerAccessAlreadyEnabled) { cudaGetLastError(); return SCALECOM_OK; }
    if (e != cudaSuccess) { cudaGetLastError(); return SCALECOM_ERR_CUDA; }
    return SCALECOM_OK;
}

int scalecom_reduce_rows(scalecom_ctx* c, const float* rows, int32_t n_rows, float* out_val, const int32_t* idx,
                         float* weights, const uint32_t* wait_flags, uint32_t tag) {
    if (!c || !rows || !out_val || (weights && !idx)) return SCALECOM_ERR_NULL_PTR;
    if (n_rows < 1 || (wait_flags && (tag == 0u || n_rows > LP_MAX_PEERS))) return SCALECOM_ERR_INVALID_ARG;
    if (static_cast<const void*>(rows) == out_val || static_cast<const void*>(weights) == out_val ||
        static_cast<const void*>(weights) == rows || static_cast<const void*>(idx) == out_val)
        return SCALECOM_ERR_ALIAS;
    if (c->poisoned) return SCALECOM_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    const uint32_t want = uint32_t((c->k + 255) / 256), cap = uint32_t(c->sms) * 8u;
    reduce_rows_kernel<<<want < cap ? want : cap, 256, 0, c->stream>>>(rows, n_rows, uint32_t(c->k), float(n_rows), out_val,
                                                                      idx, weights, uint32_t(c->d), c->lr,
                                                                      c->ctrl + CT_STATUS, wait_flags, tag, c->spin_limit);
    if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    return SCALECOM_OK;
}

int scalecom_status(scalecom_ctx* c) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    uint32_t st = 0;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
        cudaMemcpy(&st, c->ctrl + CT_STATUS, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
        c->poisoned = true;
        return SCALECOM_ERR_CUDA;
    }
    if (st == DEV_OK) return SCALECOM_OK;
    c->poisoned = true;
    return st == DEV_TIMEOUT ? SCALECOM_ERR_TIMEOUT : SCALECOM_ERR_INTERNAL;
}

int scalecom_reset(scalecom_ctx* c) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    if (init_workspace(c) != SCALECOM_OK || cudaStreamSynchronize(c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    c->poisoned = false;
    return SCALECOM_OK;
}

int scalecom_set_option(scalecom_ctx* c, int option, int64_t value) {
    if (!c) return SCALECOM_ERR_NULL_PTR;
    switch (option) {
        case SCALECOM_OPT_FORCE_EXACT_PATH: c->force_exact = value ? 1u : 0u; return SCALECOM_OK;
        case SCALECOM_OPT_SPIN_LIMIT:
            if (value < 0 || value > 0x7FFFFFFFLL) return SCALECOM_ERR_INVALID_ARG;
            c->spin_limit = uint32_t(value);
            return SCALECOM_OK;
        case SCALECOM_OPT_KERNEL_TIMING: {
            if (value && !c->ev) {
                DeviceGuard guard(c->device);
                c->ev = new (std::nothrow) cudaEvent_t[scalecom_ctx::EV_RING * 4]();
                if (!c->ev) return SCALECOM_ERR_ALLOC;
                for (int i = 0; i < scalecom_ctx::EV_RING * 4; ++i)
                    if (cudaEventCreate(&c->ev[i]) != cudaSuccess) return SCALECOM_ERR_CUDA;
            }
            c->timing = value != 0;
            c->ev_steps = 0;
            return SCALECOM_OK;
        }
        case SCALECOM_OPT_FUSE_UPDATE: c->fuse_update = value != 0; return SCALECOM_OK;
        case SCALECOM_OPT_USE_HINT: c->use_hint = value ? 1u : 0u; return SCALECOM_OK;
        case SCALECOM_OPT_FUSED_SMALL: c->fused_small = value != 0; return SCALECOM_OK;
        case SCALECOM_OPT_L2_KEEP: c->l2_keep = value != 0; return SCALECOM_OK;
        case SCALECOM_OPT_KERNEL_SPANS: {
            DeviceGuard guard(c->device);
            const size_t bytes = size_t(scalecom_ctx::EV_RING) * 4 * 8;
            if (value && !c->spans && cudaMalloc(reinterpret_cast<void**>(&c->spans), bytes) != cudaSuccess) {
                cudaGetLastError();
                c->spans = nullptr;
                return SCALECOM_ERR_ALLOC;
            }
            if (c->spans && cudaMemsetAsync(c->spans, 0, bytes, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
            c->span_timing = value != 0;
            c->span_steps = 0;
            return SCALECOM_OK;
        }
        case SCALECOM_OPT_SELECTOR: {
            if (value != SCALECOM_SELECTOR_TOPK && value != SCALECOM_SELECTOR_CHUNK && value != SCALECOM_SELECTOR_LAYER_TOPK)
                return SCALECOM_ERR_INVALID_ARG;
            if (value == SCALECOM_SELECTOR_CHUNK && !c->chunk_best) {
                DeviceGuard guard(c->device);
                int occ = 0;
                // the smallest occupancy of the four instantiations: one grid serves them all
                {
                    int o[4] = {0, 0, 0, 0};
                    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[0], chunk_select_kernel<true, true>, CS_THREADS, 0) != cudaSuccess ||
                        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[1], chunk_select_kernel<true, false>, CS_THREADS, 0) != cudaSuccess ||
                        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[2], chunk_select_kernel<false, true>, CS_THREADS, 0) != cudaSuccess ||
                        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[3], chunk_select_kernel<false, false>, CS_THREADS, 0) != cudaSuccess)
                        return SCALECOM_ERR_CUDA;
                    occ = o[0];
                    for (int q = 1; q < 4; ++q) occ = o[q] < occ ? o[q] : occ;
                    if (occ < 1) return SCALECOM_ERR_CUDA;
                }
                if (occ > CS_BLOCKS_PER_SM) occ = CS_BLOCKS_PER_SM;
                const int64_t per_block = int64_t(CS_THREADS / 32) * CS_RUN;                   // chunks one block takes per round
                const uint32_t need = uint32_t((c->k + per_block - 1) / per_block);
                c->chunk_blocks = uint32_t(c->sms * occ) < need ? uint32_t(c->sms * occ) : need;
                const size_t bytes = size_t(c->k) * 8;
                if (cudaMalloc(reinterpret_cast<void**>(&c->chunk_best), bytes) != cudaSuccess) {
                    cudaGetLastError();
                    c->chunk_best = nullptr;
                    return SCALECOM_ERR_ALLOC;
                }
                const uint32_t one[4] = {0u, uint32_t(c->d), 0u, uint32_t(c->k)};
                if (cudaMalloc(reinterpret_cast<void**>(&c->one_layer_tab), sizeof one) != cudaSuccess) {
                    cudaGetLastError();
                    cudaFree(c->chunk_best);
                    c->chunk_best = nullptr;
                    c->one_layer_tab = nullptr;
                    return SCALECOM_ERR_ALLOC;
                }
                if (cudaMemsetAsync(c->chunk_best, 0, bytes, c->stream) != cudaSuccess ||
                    cudaMemcpy(c->one_layer_tab, one, sizeof one, cudaMemcpyHostToDevice) != cudaSuccess)
                    return SCALECOM_ERR_CUDA;
            }
            c->selector = int(value);
            return SCALECOM_OK;
        }
        default: return SCALECOM_ERR_INVALID_ARG;
    }
}

int scalecom_query(scalecom_ctx* c, int item, int64_t* out) {
    if (!c || !out) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    uint32_t w[CT_WORDS];
    switch (item) {
        case SCALECOM_Q_WORKSPACE_BYTES:
            *out = int64_t(c->ws_bytes) + (c->stage_g ? int64_t(c->n) * c->d * 4 + c->k * 8 : 0);
            return SCALECOM_OK;
        case SCALECOM_Q_TOPK_BLOCKS: *out = c->topk_blocks; return SCALECOM_OK;
        case SCALECOM_Q_KERNEL_LAUNCHES: *out = c->launches; return SCALECOM_OK;
        case SCALECOM_Q_FUSED_SMALL:
            *out = (c->small_blocks && c->fused_small && c->selector == SCALECOM_SELECTOR_TOPK) ? c->small_blocks : 0;
            return SCALECOM_OK;
        case SCALECOM_Q_LAST_TOPK_PATH:
        case SCALECOM_Q_LAST_CANDIDATES:
            if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
                cudaMemcpy(w, c->ctrl, sizeof w, cudaMemcpyDeviceToHost) != cudaSuccess)
                return SCALECOM_ERR_CUDA;
            *out = item == SCALECOM_Q_LAST_TOPK_PATH ? w[CT_PATH] : w[CT_M];
            return SCALECOM_OK;
        default:
            if (item >= SCALECOM_Q_PHASE_STAMP0 && item < SCALECOM_Q_PHASE_STAMP0 + CT_NSTAMPS) {
                if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
                    cudaMemcpy(w, c->ctrl, sizeof w, cudaMemcpyDeviceToHost) != cudaSuccess)
                    return SCALECOM_ERR_CUDA;
                *out = w[CT_STAMP + item - SCALECOM_Q_PHASE_STAMP0];
                return SCALECOM_OK;
            }
            return SCALECOM_ERR_INVALID_ARG;
    }
}

int scalecom_kernel_ms(scalecom_ctx* c, float ms[3], int32_t* nsteps) {
    if (!c || !ms || !nsteps) return SCALECOM_ERR_NULL_PTR;
    if (!c->timing || !c->ev) return SCALECOM_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    const int64_t kept = c->ev_steps < scalecom_ctx::EV_RING ? c->ev_steps : scalecom_ctx::EV_RING;
    ms[0] = ms[1] = ms[2] = 0.f;
    for (int64_t s = c->ev_steps - kept; s < c->ev_steps; ++s) {
        cudaEvent_t* ev = c->ev + 4 * (s % scalecom_ctx::EV_RING);
        const int nint = c->ev_has_update[s % scalecom_ctx::EV_RING] ? 3 : 2;
        for (int i = 0; i < nint; ++i) {
            float x = 0.f;
            if (cudaEventElapsedTime(&x, ev[i], ev[i + 1]) != cudaSuccess) return SCALECOM_ERR_CUDA;
            ms[i] += x;
        }
    }
    *nsteps = int32_t(kept);
    c->ev_steps = 0;
    return SCALECOM_OK;
}

extern "C++" {
namespace {

int ensure_diag(scalecom_ctx* c) {
    if (c->diag_mean) return SCALECOM_OK;
    const size_t vec = size_t(c->d) * 4, bm = size_t(c->ntiles) * 32 * 4;
    if (cudaMalloc(reinterpret_cast<void**>(&c->diag_mean), vec) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&c->diag_zero), vec) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&c->diag_bitmap), bm) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&c->diag_acc), 4 * sizeof(double)) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(c->diag_mean); cudaFree(c->diag_zero); cudaFree(c->diag_bitmap); cudaFree(c->diag_acc);
        c->diag_mean = c->diag_zero = nullptr; c->diag_bitmap = nullptr; c->diag_acc = nullptr;
        return SCALECOM_ERR_ALLOC;
    }
    if (cudaMemsetAsync(c->diag_zero, 0, vec, c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    return SCALECOM_OK;
}

template <int N, bool VEC>
cudaError_t launch_mean(const scalecom_ctx* c, const float* const* grads, const float* const* mem) {
    PtrTable<N> tab;
    for (int i = 0; i < N; ++i) {
        tab.g[i] = i < c->n ? grads[i] : nullptr;
        tab.m[i] = i < c->n ? const_cast<float*>(mem[i]) : nullptr;
    }
    const uint32_t quads = uint32_t((c->d + 3) / 4);
    const uint32_t want = (quads + 255u) / 256u, cap = uint32_t(c->sms) * 8u;
    mean_acc_kernel<N, VEC><<<want < cap ? want : cap, 256, 0, c->stream>>>(tab, c->n, uint32_t(c->d), float(c->n), c->diag_mean);
    return cudaGetLastError();
}

template <bool VEC>
cudaError_t launch_mean_n(const scalecom_ctx* c, const float* const* grads, const float* const* mem) {
    if (c->n <= 16) return launch_mean<16, VEC>(c, grads, mem);
    if (c->n <= 128) return launch_mean<128, VEC>(c, grads, mem);
    return launch_mean<SCALECOM_MAX_LEARNERS, VEC>(c, grads, mem);
}

}  // namespace
}  // extern "C++"

int scalecom_overlap(scalecom_ctx* c, const float* const* grads, const float* const* mem, int64_t t, int64_t* host_hamming_d) {
    if (!c || !grads || !mem || !host_hamming_d) return SCALECOM_ERR_NULL_PTR;
    if (t < 0) return SCALECOM_ERR_INVALID_ARG;
    if (c->poisoned) return SCALECOM_ERR_BAD_STATE;
    for (int i = 0; i < c->n; ++i)
        if (!grads[i] || !mem[i]) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    int rc = ensure_diag(c);
    if (rc != SCALECOM_OK) return rc;
    const int leader = int(t % c->n);
    const size_t bm_words = size_t(c->ntiles) * 32;
    bool vec_all = true;
    for (int i = 0; i < c->n; ++i) vec_all = vec_all && aligned16(grads[i]) && aligned16(mem[i]);

    // leader's set I^k(acc_L): the exact selector, hints neither used nor left behind
    TopkParams tp = make_topk_params(c, grads[leader], mem[leader], nullptr, false, nullptr);
    cudaError_t e = (aligned16(tp.g) && aligned16(tp.m)) ? launch_topk<true>(c, tp) : launch_topk<false>(c, tp);
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    if (cudaMemcpyAsync(c->diag_bitmap, c->bitmap, bm_words * 4, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    // true top-k: the same selection on the all-reduced vector
    e = vec_all ? launch_mean_n<true>(c, grads, mem) : launch_mean_n<false>(c, grads, mem);
    if (e != cudaSuccess) return SCALECOM_ERR_CUDA;
    tp = make_topk_params(c, c->diag_mean, c->diag_zero, nullptr, false, nullptr);
    if (launch_topk<true>(c, tp) != cudaSuccess) return SCALECOM_ERR_CUDA;
    if (cudaMemsetAsync(c->diag_acc, 0, 4 * sizeof(double), c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    const uint32_t want = uint32_t((bm_words + 255) / 256), cap = uint32_t(c->sms) * 8u;
    overlap_kernel<<<want < cap ? want : cap, 256, 0, c->stream>>>(c->diag_bitmap, c->bitmap, bm_words,
                                                                  reinterpret_cast<unsigned long long*>(c->diag_acc));
    if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
    c->launches += 4;
    unsigned long long common = 0;
    if (cudaMemcpyAsync(&common, c->diag_acc, 8, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    rc = scalecom_status(c);
    if (rc != SCALECOM_OK) return rc;
    *host_hamming_d = c->k - int64_t(common);
    return SCALECOM_OK;
}

int scalecom_cosine_distance(scalecom_ctx* c, const float* x, const float* y, double* host_out) {
    if (!c || !x || !y || !host_out) return SCALECOM_ERR_NULL_PTR;
    DeviceGuard guard(c->device);
    if (!guard.ok) return SCALECOM_ERR_CUDA;
    const int rc = ensure_diag(c);
    if (rc != SCALECOM_OK) return rc;
    if (cudaMemsetAsync(c->diag_acc, 0, 4 * sizeof(double), c->stream) != cudaSuccess) return SCALECOM_ERR_CUDA;
    const uint32_t want = uint32_t((c->d + 255) / 256), cap = uint32_t(c->sms) * 8u;
    dot3_kernel<<<want < cap ? want : cap, 256, 0, c->stream>>>(x, y, uint32_t(c->d), c->diag_acc + 1);
    if (cudaGetLastError() != cudaSuccess) return SCALECOM_ERR_CUDA;
    ++c->launches;
    double h[3];
    if (cudaMemcpyAsync(h, c->diag_acc + 1, sizeof h, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    *host_out = 1.0 - h[0] / (std::sqrt(h[1]) * std::sqrt(h[2]));
    return SCALECOM_OK;
}

int scalecom_kernel_span_ms(scalecom_ctx* c, float ms[2], int32_t* nsteps) {
    if (!c || !ms || !nsteps) return SCALECOM_ERR_NULL_PTR;
    if (!c->span_timing || !c->spans) return SCALECOM_ERR_BAD_STATE;
    DeviceGuard guard(c->device);
    static_assert(scalecom_ctx::EV_RING * 4 * 8 <= 16384, "span ring copied to the stack");
    unsigned long long h[scalecom_ctx::EV_RING * 4];
    if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
        cudaMemcpy(h, c->spans, sizeof h, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(c->spans, 0, sizeof h) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    const int64_t kept = c->span_steps < scalecom_ctx::EV_RING ? c->span_steps : scalecom_ctx::EV_RING;
    double sum[2] = {0.0, 0.0};
    for (int64_t s = 0; s < kept; ++s)
        for (int i = 0; i < 2; ++i) {
            const unsigned long long start = ~h[4 * s + 2 * i], end = h[4 * s + 2 * i + 1];
            if (end > start) sum[i] += double(end - start) * 1e-6;
        }
    ms[0] = float(sum[0]);
    ms[1] = float(sum[1]);
    *nsteps = int32_t(kept);
    c->span_steps = 0;
    return SCALECOM_OK;
}

const char* scalecom_strerror(int code) {
    switch (code) {
        case SCALECOM_OK: return "success";
        case SCALECOM_ERR_INVALID_ARG: return "invalid argument";
        case SCALECOM_ERR_NULL_PTR: return "null pointer";
        case SCALECOM_ERR_ALLOC: return "allocation failed";
        case SCALECOM_ERR_CUDA: return "CUDA runtime error";
        case SCALECOM_ERR_TIMEOUT: return "device-side wait timed out";
        case SCALECOM_ERR_BAD_STATE: return "the handle cannot take this call in its present state (after a device error: scalecom_reset)";
        case SCALECOM_ERR_INTERNAL: return "device-side consistency check failed";
        case SCALECOM_ERR_ALIAS: return "buffers overlap";
        default: return "unknown error";
    }
}

}  // extern "C"
