// scalecom_topk_static: the leader's top-k selection with no allocation at all.
//
// Some callers cannot allocate device memory when they need a selection: the
// process may have handed every byte of the GPU to a framework's caching
// allocator or been given a fixed memory partition (so cudaMalloc fails), or
// it may sit in a latency-critical loop where cudaMalloc's implicit device-wide
// synchronisation is not acceptable.  For them the selection kernel's scratch
// lives in the file-scope device array below instead of a per-handle workspace.
#include "../../include/scalecom.h"

#include <cuda_runtime.h>

#include <cmath>
#include <mutex>

#include "topk_select.cuh"

using namespace sc;

namespace {

constexpr uint32_t MAX_D = SCALECOM_STATIC_MAX_D;
constexpr uint32_t MAX_TILES = (MAX_D + TILE - 1) / TILE;
constexpr uint32_t MAX_BLOCKS = 512;
constexpr int MAX_DEVICES = 64;

constexpr size_t al(size_t x) { return (x + 255) / 256 * 256; }
// the first OFF_CLEAR_END bytes must be zero when the kernel starts
constexpr size_t OFF_SAMP = 0;
constexpr size_t OFF_CW = OFF_SAMP + al(NCOARSE * 4);
constexpr size_t OFF_CTRL = OFF_CW + al((WIN + 1) * 4);
constexpr size_t OFF_BAR = OFF_CTRL + al(CT_WORDS * 4);
constexpr size_t OFF_BT = OFF_BAR + al(256);
constexpr size_t OFF_FINE = OFF_BT + al(MAX_BLOCKS * 4);
constexpr size_t OFF_DH = OFF_FINE + al(NFINE * 4);
constexpr size_t OFF_CLEAR_END = OFF_DH + al(size_t(DH_PASSES) * DH_BINS * 4);
constexpr size_t OFF_BM = OFF_CLEAR_END;
constexpr size_t OFF_TP = OFF_BM + al(size_t(MAX_TILES) * 32 * 4);
constexpr size_t OFF_BL = OFF_TP + al((size_t(MAX_TILES) + 1) * 4);
constexpr size_t OFF_CAND = OFF_BL + al(size_t(BCAP) * 8);
constexpr size_t CAND_ENTRIES = size_t(MAX_D) + 32u * MAX_BLOCKS * TK_WARPS;   // every warp's share of the vector + slack
constexpr size_t SCRATCH_BYTES = OFF_CAND + al(CAND_ENTRIES * 8);

// About 11 MB, held by every GPU on which this entry point has been called, until the process exits.
// In host code this name is only a stand-in for the symbol, never a device
// address: the address the kernel gets comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_scratch[SCRATCH_BYTES];

struct DeviceSetup {
    bool done = false;
    unsigned char* scratch = nullptr;   // device address of g_scratch on this device
    int max_blocks = 0;                 // co-resident blocks of the selection kernel
};
DeviceSetup g_setup[MAX_DEVICES];
std::mutex g_mu;

int setup_device(int dev, DeviceSetup& su) {
    // (with lazy module loading this is also where the runtime places the array in device memory)
    void* p = nullptr;
    const cudaError_t es = cudaGetSymbolAddress(&p, g_scratch);
    if (es == cudaErrorMemoryAllocation) return SCALECOM_ERR_ALLOC;
    if (es != cudaSuccess || !p) return SCALECOM_ERR_CUDA;
    int sms = 0, coop = 0, occ = 0, o2 = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop ||
        cudaFuncSetAttribute(topk_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(sizeof(TopkShared))) != cudaSuccess ||
        cudaFuncSetAttribute(topk_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(sizeof(TopkShared))) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, topk_select_kernel<true>, TK_THREADS,
                                                      sizeof(TopkShared)) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o2, topk_select_kernel<false>, TK_THREADS,
                                                      sizeof(TopkShared)) != cudaSuccess)
        return SCALECOM_ERR_CUDA;
    if (o2 < occ) occ = o2;
    if (occ < 1) return SCALECOM_ERR_CUDA;
    if (occ > TK_BLOCKS_PER_SM) occ = TK_BLOCKS_PER_SM;
    su.scratch = static_cast<unsigned char*>(p);
    su.max_blocks = sms * occ;
    if (su.max_blocks > int(MAX_BLOCKS)) su.max_blocks = int(MAX_BLOCKS);
    su.done = true;
    return SCALECOM_OK;
}

}  // namespace

extern "C" int scalecom_topk_static(const float* g, const float* m, int64_t d, int64_t k, int32_t* out_idx,
                                    int32_t* dev_status, void* cuda_stream) {
    if (!g || !m || !out_idx) return SCALECOM_ERR_NULL_PTR;
    if (d < 1 || d > int64_t(MAX_D) || k < 1 || k > d) return SCALECOM_ERR_INVALID_ARG;
    if (static_cast<const void*>(g) == static_cast<const void*>(out_idx) ||
        static_cast<const void*>(m) == static_cast<const void*>(out_idx))
        return SCALECOM_ERR_ALIAS;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SCALECOM_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    std::lock_guard<std::mutex> lock(g_mu);
    DeviceSetup& su = g_setup[dev];
    if (!su.done) {
        const int rc = setup_device(dev, su);
        if (rc != SCALECOM_OK) { cudaGetLastError(); return rc; }
    }
    unsigned char* base = su.scratch;

    TopkParams P;
    P.g = g;
    P.m = m;
    P.d = uint32_t(d);
    P.k = uint32_t(k);
    // same sampling rule as a handle: about 2^18 sampled keys or 1/64 of the vector
    uint32_t stride = 1;
    while (stride < 64 && (d / (2 * stride)) >= (1 << 18)) stride *= 2;
    P.samp_stride = stride;
    {
        const int64_t span = int64_t(SAMPLE_GRANULE) * stride;
        const int64_t full = d / span, rem = d % span;
        const int64_t ns = full * SAMPLE_GRANULE + (rem < SAMPLE_GRANULE ? rem : SAMPLE_GRANULE);
        if (stride == 1) {
            P.samp_target = uint32_t(k);
        } else {
            const double ks = double(k) * double(ns) / double(d);
            double tgt = std::ceil(ks + 6.0 * std::sqrt(ks) + 8.0);
            if (tgt > double(ns)) tgt = double(ns);
            P.samp_target = uint32_t(tgt);
        }
    }
    P.force_exact = 0;
    P.keep_frac = 0.0f;
    P.use_hint = 0;               // the scratch is shared by unrelated callers: no carry-over between calls
    P.leader_hint = nullptr;
    P.all_hints = nullptr;
    P.n_hints = 0;
    P.spin_limit = 1u << 22;
    P.samp_hist = reinterpret_cast<uint32_t*>(base + OFF_SAMP);
    P.coarse_win = reinterpret_cast<uint32_t*>(base + OFF_CW);
    P.ctrl = reinterpret_cast<uint32_t*>(base + OFF_CTRL);
    P.barrier = reinterpret_cast<unsigned long long*>(base + OFF_BAR);
    P.block_tot = reinterpret_cast<uint32_t*>(base + OFF_BT);
    P.fine_hist = reinterpret_cast<uint32_t*>(base + OFF_FINE);
    P.fine_hist_next = nullptr;   // one copy: the memset before every launch clears it
    P.digit_hist = reinterpret_cast<uint32_t*>(base + OFF_DH);
    P.bitmap = reinterpret_cast<uint32_t*>(base + OFF_BM);
    P.tile_prefix = reinterpret_cast<uint32_t*>(base + OFF_TP);
    P.cand = reinterpret_cast<uint2*>(base + OFF_CAND);
    P.blist = reinterpret_cast<uint2*>(base + OFF_BL);
    P.ntiles = uint32_t((d + TILE - 1) / TILE);
    const uint32_t chunks = uint32_t((d + TK_CHUNK - 1) / TK_CHUNK);
    uint32_t blocks = uint32_t(su.max_blocks);
    if (blocks > chunks) blocks = chunks;
    if (blocks < 1) blocks = 1;
    {
        // one candidate segment per warp, carved from the fixed candidate area
        const int64_t warps = int64_t(blocks) * TK_WARPS;
        int64_t cap = (4 * k + warps - 1) / warps + 32;
        const int64_t share = (d + warps - 1) / warps + 32;
        if (cap > share) cap = share;
        if (cap * warps > int64_t(CAND_ENTRIES)) cap = int64_t(CAND_ENTRIES) / warps;
        P.seg_cap = uint32_t(cap);
    }
    P.tiles_per_block = (P.ntiles + blocks - 1) / blocks;
    P.out_idx = out_idx;
    P.spans = nullptr;

    // Every call shares the array and finds the previous call's contents in it: the
    // counters, the histograms and the barrier word must start at zero (the kernel
    // itself clears the rest before using it).
    if (cudaMemsetAsync(base, 0, OFF_CLEAR_END, stream) != cudaSuccess) { cudaGetLastError(); return SCALECOM_ERR_CUDA; }
    const bool vec = ((reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(m)) & 15u) == 0;
    void* args[] = {&P};
    const void* fn = vec ? reinterpret_cast<const void*>(&topk_select_kernel<true>)
                         : reinterpret_cast<const void*>(&topk_select_kernel<false>);
    if (cudaLaunchCooperativeKernel(fn, dim3(blocks), dim3(TK_THREADS), args, sizeof(TopkShared), stream) != cudaSuccess) {
        cudaGetLastError();
        return SCALECOM_ERR_CUDA;
    }
    if (dev_status &&
        cudaMemcpyAsync(dev_status, P.ctrl + CT_STATUS, 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
        cudaGetLastError();
        return SCALECOM_ERR_CUDA;
    }
    return SCALECOM_OK;
}
