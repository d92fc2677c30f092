/*
 * scalecom.h -- C ABI of the B200 (sm_100a) CLT-k compression step.
 *
 * One call of scalecom_step() is one iteration t of ScaleCom's Algorithm 1 for
 * n logical learners whose gradients and error-feedback memories live as n + n
 * fp32 vectors of d values in one GPU's memory:
 *
 *   1. acc_i = m_i + g_i                       error feedback, Algorithm 1 line 6
 *   2. I = top-k index set of |acc_L|,         Eq. 2, leader L = t mod n
 *      exactly k indices, ties to the lower index, returned ascending
 *   3. G[i][j] = acc_i[I[j]] (CLT-k, Eq. 3);   val[j] = (G[0][j]+...+G[n-1][j]) / n
 *      summed in learner order                 Algorithm 1 line 10, Eq. 1
 *   4. m_i <- (1-beta) m_i + beta (acc_i - CLT-k(acc_i))          Eq. 4
 *   5. theta[I[j]] <- theta[I[j]] - lr * val[j]                   Algorithm 1 line 12
 *
 * Every fp32 operation above is a separately rounded IEEE-754 operation (no
 * fused multiply-add, no flush to zero), so results do not depend on launch
 * geometry and are reproducible bit for bit.
 *
 * Conventions
 *   - "DEVICE" pointers address memory of the GPU that was current when the
 *     handle was created; "HOST" pointers address host memory.
 *   - All functions return 0 (SCALECOM_OK) or a negative scalecom_error; none
 *     throws, aborts or traps.  Nothing is launched when an argument is rejected.
 *   - A handle owns only scratch memory.  All algorithm state (m_i, theta, t)
 *     belongs to the caller, so a run can be resumed with a fresh handle.
 *   - A handle is bound to one CUDA stream (default: the legacy default stream);
 *     calls on one handle must not be made concurrently from several threads.
 */
#ifndef SCALECOM_H
#define SCALECOM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct scalecom_ctx scalecom_ctx;

typedef enum scalecom_error {
    SCALECOM_OK               = 0,
    SCALECOM_ERR_INVALID_ARG  = -1,  /* a size or hyper-parameter out of range          */
    SCALECOM_ERR_NULL_PTR     = -2,  /* a required pointer is NULL                      */
    SCALECOM_ERR_ALLOC        = -3,  /* host or device allocation failed                */
    SCALECOM_ERR_CUDA         = -4,  /* a CUDA runtime call or a launch failed          */
    SCALECOM_ERR_TIMEOUT      = -5,  /* a bounded device-side wait expired              */
    SCALECOM_ERR_BAD_STATE    = -6,  /* the handle cannot take this call as it stands: poisoned by an earlier
                                        device error, a per-layer selector without layers, no selection to reuse */
    SCALECOM_ERR_INTERNAL     = -7,  /* a device-side consistency check failed          */
    SCALECOM_ERR_ALIAS        = -8   /* buffers that must be distinct overlap           */
} scalecom_error;

/* Largest number of learners one handle accepts (pointer tables travel as kernel arguments). */
#define SCALECOM_MAX_LEARNERS 1024

/*
 * Create a handle for vectors of d coordinates, n learners and k kept
 * coordinates (Algorithm 1's inputs; 0 < beta <= 1 is Eq. 4's discounting
 * factor, lr is the step size alpha of line 12).
 *   out    HOST, receives the handle.
 *   d      1 <= d <= 2^31 - 1.      n   1 <= n <= SCALECOM_MAX_LEARNERS.
 *   k      1 <= k <= d.             beta in (0, 1].   lr finite.
 * Allocates the scratch workspace on the current device with one cudaMalloc: about
 * d/8 + d/128 + 48*k bytes + 0.4 MB (selection bitmap, per-tile counts, candidate
 * segments, histograms); SCALECOM_Q_WORKSPACE_BYTES reports the exact figure.
 * Errors: INVALID_ARG, NULL_PTR, ALLOC, CUDA.
 */
int scalecom_create(scalecom_ctx** out, int64_t d, int32_t n, int64_t k, float beta, float lr);

/*
 * One iteration of Algorithm 1 (steps 1-5 above), asynchronous on the handle's
 * stream: no host synchronisation, no device-to-host copy.
 *   grads    HOST array of n DEVICE pointers, each fp32[d], read only.
 *   mem      HOST array of n DEVICE pointers, each fp32[d], updated in place (Eq. 4).
 *   weights  DEVICE fp32[d], updated in place at the k selected coordinates;
 *            NULL skips step 5 (the caller applies its own optimiser to out_val).
 *   t        iteration index >= 0; the leader is learner t mod n.
 *   out_idx  DEVICE int32[k], written: the selected coordinates, ascending.
 *   out_val  DEVICE fp32[k], written: the averaged reduced values at out_idx.
 * The two pointer arrays are read during the call and may be reused at once.
 * grads[i], mem[i], weights and the outputs must not overlap one another
 * (exact pointer equality is rejected with ALIAS; partial overlap is undefined).
 * Any alignment is accepted; 16-byte aligned vectors take the fast path.
 * Errors: NULL_PTR, INVALID_ARG (t < 0), ALIAS, BAD_STATE, CUDA.
 */
int scalecom_step(scalecom_ctx* ctx,
                  const float* const* grads,
                  float* const* mem,
                  float* weights,
                  int64_t t,
                  int32_t* out_idx,
                  float* out_val);

/*
 * The same iteration for callers whose gradients and results live in HOST
 * memory (Algorithm 1 lines 9 and 11, "upload"/"download"): copies the n
 * gradients to a device staging area owned by the handle (allocated on first
 * use, n*d*4 bytes), runs scalecom_step, copies out_idx and out_val back and
 * waits for the stream.  mem and weights stay DEVICE pointers (they are state,
 * not per-iteration traffic).  Pinned host memory makes the copies asynchronous.
 *   host_grads  HOST array of n HOST pointers, each fp32[d].
 *   host_idx    HOST int32[k], written.     host_val  HOST fp32[k], written.
 * Errors: as scalecom_step, plus ALLOC.
 */
int scalecom_step_host(scalecom_ctx* ctx,
                       const float* const* host_grads,
                       float* const* mem,
                       float* weights,
                       int64_t t,
                       int32_t* host_idx,
                       float* host_val);

/* Release the workspace.  NULL is accepted.  Synchronises the handle's stream first. */
void scalecom_destroy(scalecom_ctx* ctx);

/* Bind the handle to a CUDA stream (a cudaStream_t passed as void*; NULL = legacy default). */
int scalecom_set_stream(scalecom_ctx* ctx, void* cuda_stream);

/*
 * Ask every later step to also write the per-learner gathered values of Eq. 3:
 * G[i*k + j] = acc_i[out_idx[j]] into the caller's DEVICE fp32[n*k] buffer.
 * NULL (the default) turns the extra output off.
 */
int scalecom_set_gathered(scalecom_ctx* ctx, float* dev_gathered);

/*
 * Per-layer compression rates for the chunk-wise selector (Section 4: the rate of a layer follows its
 * FLOPs per gradient -- 25X, 50X or 400X -- and the first layer is sent uncompressed).  The d
 * coordinates are the concatenation of nlayers layers; layer s has sizes[s] coordinates and keeps
 * keep[s] of them by the chunk-wise rule applied inside the layer (keep[s] == sizes[s]: sent whole).
 *   nlayers  1 .. 2048, or 0 to go back to one rate for the whole vector.
 *   sizes, keep  HOST int64[nlayers]; sizes[s] >= 1, 1 <= keep[s] <= sizes[s], sum sizes = d, sum keep = k.
 * SCALECOM_SELECTOR_CHUNK and SCALECOM_SELECTOR_LAYER_TOPK look at the layers; SCALECOM_SELECTOR_TOPK
 * (Eq. 2 over the whole vector) ignores them.
 * Waits for the stream.  Errors: NULL_PTR, INVALID_ARG, ALLOC, CUDA.
 */
int scalecom_set_layers(scalecom_ctx* ctx, int32_t nlayers, const int64_t* sizes, const int64_t* keep);

/*
 * The step taken apart, for the learner-per-GPU deployment the paper describes (Section 4, Appendix E:
 * the leading worker's indices are broadcast, every worker compresses its own error-feedback gradient
 * with them, the kept values are reduced across workers).  One handle per rank, created with the
 * global d and k; the collectives between the three calls are the caller's (NCCL or any other):
 *
 *   leader rank (t mod world):   scalecom_select(g, m, idx)                          step 2
 *   all ranks, after the broadcast of idx:
 *                                scalecom_compress(g, m, idx, gathered)              steps 1, 3 (gather), 4
 *   all ranks, after an all-gather of the `gathered` rows into rows[world][k] (rank order):
 *                                scalecom_reduce_rows(rows, world, val, idx, theta)  step 3 (reduce) and step 5
 *
 * Summing the gathered rows locally in rank order (k values per rank cross the links, as in the paper)
 * keeps the result identical, bit for bit, to scalecom_step on one GPU holding all the learners.
 * All pointers DEVICE; all three calls are asynchronous on the handle's stream.
 *   scalecom_select    g, m fp32[d] read only; out_idx int32[k] written, ascending (selector as set by
 *                      SCALECOM_OPT_SELECTOR).
 *   scalecom_compress  g fp32[d] read only; m fp32[d] updated in place (Eq. 4); idx int32[k] strictly
 *                      ascending, < d (otherwise scalecom_status reports INTERNAL and nothing is written
 *                      out of bounds); out_gathered fp32[k] = (m + g)[idx[j]] written.  idx == NULL on the
 *                      leader: the list is the one this handle's scalecom_select produced in the call just
 *                      before (nothing else on the handle in between, else BAD_STATE); the selection's own
 *                      bitmap is used and the list is not read again.
 *   scalecom_reduce_rows  rows fp32[n_rows * k] read only; out_val fp32[k] = (sum over rows, in order) / n_rows
 *                      written.  weights fp32[d], if not NULL, gets Algorithm 1 line 12 in the same kernel:
 *                      weights[idx[j]] -= lr * out_val[j], with idx int32[k] the broadcast list (an entry >= d
 *                      is skipped and scalecom_status reports INTERNAL); weights NULL: no update, idx unused.
 *                      wait_flags NULL: the rows are complete when the kernel starts (stream order, or a fence
 *                      the caller placed).  wait_flags DEVICE uint32[n_rows] with tag != 0 (n_rows <= 64): row
 *                      i is read only after wait_flags[i] holds tag (see scalecom_compress_scatter); the wait
 *                      is bounded by SCALECOM_OPT_SPIN_LIMIT polls per word, after which nothing is written
 *                      and scalecom_status reports TIMEOUT.
 * Errors (all three): NULL_PTR, ALIAS, BAD_STATE, ALLOC (compress, first call), CUDA; INVALID_ARG for n_rows < 1.
 */
int scalecom_select(scalecom_ctx* ctx, const float* g, const float* m, int32_t* out_idx);
int scalecom_compress(scalecom_ctx* ctx, const float* g, float* m, const int32_t* idx, float* out_gathered);

/*
 * scalecom_compress that also sends: besides out_gathered, every kept value is stored, as the pass produces
 * it, into n_dst further rows dst[0 .. n_dst) -- this rank's row of every rank's gathered-rows buffer, i.e.
 * the all-gather of the step fused into the kernel as plain stores (the paper's exchange of the k kept values,
 * Section 4 / Appendix E).
 *   dst    HOST array of n_dst DEVICE pointers, each to fp32[k]; they may point into other GPUs' memory that
 *          this device can address (peer access enabled, or a CUDA IPC mapping).  0 <= n_dst <= 64.
 * The kernel waits for nobody.  Before a destination is read (scalecom_reduce_rows there) its owner must know
 * that all senders' kernels have finished -- a barrier or any collective after this call on every rank -- and
 * a row must not be overwritten by the next step while its owner still reads it (two buffers, used in turn).
 *   flag_dst, tag   NULL / 0: no signalling, as described so far.  Otherwise flag_dst is a HOST array of n_dst
 *          DEVICE pointers to one 32-bit word each (beside the destination's rows, same addressability) and
 *          tag != 0: after the kernel's last block is through, tag is stored into every flag_dst[i] with
 *          release semantics at system scope.  scalecom_reduce_rows given those words and the same tag waits
 *          for them inside its kernel, so no collective is needed between the two calls.  Tags must differ from
 *          step to step on the same words (the step number plus one will do).
 * Errors: those of scalecom_compress; INVALID_ARG for n_dst outside 0..64 or flag_dst with tag 0; NULL_PTR,
 * ALIAS for a bad dst[i] or flag_dst[i].
 */
int scalecom_compress_scatter(scalecom_ctx* ctx, const float* g, float* m, const int32_t* idx, float* out_gathered,
                              float* const* dst, int32_t n_dst, uint32_t* const* flag_dst, uint32_t tag);

/*
 * Give the handle's device access to the memory of another device of this process (cudaDeviceEnablePeerAccess
 * with the handle's device current), which the stores of scalecom_compress_scatter into a peer's rows and the
 * polls of scalecom_reduce_rows need when the rows live on another GPU (the exchange of the kept values in the
 * paper's deployment, Section 4 / Appendix E).  peer_device is a device ordinal of this process.  Already enabled
 * counts as success; the handle's own device is accepted and does nothing.
 * Errors: NULL_PTR, INVALID_ARG (no such device, or the hardware offers no peer access between the two), CUDA.
 */
int scalecom_enable_peer_access(scalecom_ctx* ctx, int32_t peer_device);
int scalecom_reduce_rows(scalecom_ctx* ctx, const float* rows, int32_t n_rows, float* out_val, const int32_t* idx,
                         float* weights, const uint32_t* wait_flags, uint32_t tag);

/*
 * Algorithm 1 line 12 on its own: theta[idx[j]] <- theta[idx[j]] - lr * val[j]
 * for j < k, on the handle's stream, for callers that ran scalecom_step with
 * weights == NULL.  All pointers DEVICE; idx entries must be distinct and < d.
 */
int scalecom_apply_update(scalecom_ctx* ctx, float* weights, const int32_t* idx,
                          const float* val, int64_t k, float lr);

/*
 * Wait for the handle's stream and report the device-side status of the steps
 * issued so far: SCALECOM_OK, SCALECOM_ERR_TIMEOUT or SCALECOM_ERR_INTERNAL
 * (after either of which the handle refuses further steps until scalecom_reset;
 * the kernels queued behind the one that failed see the status word and do
 * nothing, so the failing step's outputs, memories and weights are left as they
 * were, except where INTERNAL was raised by an index that scalecom_compress or
 * scalecom_reduce_rows skipped), or SCALECOM_ERR_CUDA.
 */
int scalecom_status(scalecom_ctx* ctx);

/* Clear a device-side error and re-initialise the workspace (synchronises). */
int scalecom_reset(scalecom_ctx* ctx);

/* Options for scalecom_set_option. */
#define SCALECOM_OPT_FORCE_EXACT_PATH 1  /* 1: skip the sampled pre-filter, always run the full radix select */
#define SCALECOM_OPT_SPIN_LIMIT       2  /* iteration bound of the in-kernel grid barrier wait (>= 0)       */
#define SCALECOM_OPT_KERNEL_TIMING    3  /* 1: bracket each kernel of a step with CUDA events                */
#define SCALECOM_OPT_FUSE_UPDATE      4  /* 1 (default): step 5 runs inside the learner pass; 0: own kernel  */
#define SCALECOM_OPT_USE_HINT         5  /* 1 (default): a step starts its pre-filter from the threshold the
                                            previous step of this handle found; 0: always sample afresh.
                                            Affects speed only, never results                              */
#define SCALECOM_OPT_SELECTOR         6  /* how the leader's index set is found (results DO differ):
                                            SCALECOM_SELECTOR_TOPK (default): the exact top-k set of Eq. 2;
                                            SCALECOM_SELECTOR_CHUNK: the chunk-wise selection of Section 4 /
                                            Appendix E -- the d coordinates form k consecutive chunks,
                                            chunk j = [floor(j*d/k), floor((j+1)*d/k)), and each keeps its
                                            largest-magnitude coordinate (lower index on ties).  Steps 1, 3,
                                            4, 5 are unchanged.  First use allocates 8*k bytes;
                                            SCALECOM_SELECTOR_LAYER_TOPK: Eq. 2 applied inside every layer
                                            set by scalecom_set_layers -- layer s keeps its keep[s] largest
                                            magnitudes, ties to the lower index (steps and scalecom_select
                                            return BAD_STATE while no layers are set).  Its first launch
                                            after scalecom_set_layers allocates 8 KB per layer + d bytes;
                                            SCALECOM_OPT_FORCE_EXACT_PATH = 1 makes it stream g and m in
                                            every round instead of collecting the undecided coordinates    */
#define SCALECOM_OPT_KERNEL_SPANS     7  /* 1: every kernel of a step records the time from its first block's
                                            start to its last block's end on the GPU's nanosecond timer
                                            (two atomics per block); read with scalecom_kernel_span_ms     */
#define SCALECOM_OPT_FUSED_SMALL      8  /* 1 (default): with the exact top-k selector, at most 8 learners, 16-byte
                                            aligned vectors and 8*n*d <= 64 MB (all of a step's g and m fit the L2
                                            cache), scalecom_step runs as ONE cooperative kernel -- selection and
                                            learner pass share a launch and two grid barriers; 0: always the two
                                            general kernels.  Affects speed only, never results; per-kernel times
                                            then report the one kernel in the learner pass's place             */
#define SCALECOM_OPT_L2_KEEP          9  /* 1 (default): the exact top-k selection of scalecom_step loads a share of
                                            the leader's g and m (a quarter of the lines, at most 0.4 of the L2
                                            cache; none for vectors of which the cache holds under a twentieth) with
                                            a replace-last L2 hint and the rest with a replace-first hint, because
                                            the learner pass reads both vectors again.  The marked lines keep their
                                            priority until something replaces them; 0: default L2 policy.  Affects
                                            speed only, never results                                            */
#define SCALECOM_SELECTOR_TOPK  0
#define SCALECOM_SELECTOR_CHUNK 1
#define SCALECOM_SELECTOR_LAYER_TOPK 2
int scalecom_set_option(scalecom_ctx* ctx, int option, int64_t value);

/* Items for scalecom_query (each synchronises the stream when it reads device state). */
#define SCALECOM_Q_WORKSPACE_BYTES  1  /* device bytes owned by the handle                                    */
#define SCALECOM_Q_LAST_TOPK_PATH   2  /* last step's selection path: 0 = sampled pre-filter, 1 = full select,
                                          2 = pre-filter started from the previous step's threshold,
                                          3 = chunk-wise selector, 4 = exact top-k per layer (collecting
                                          route), 5 = the same by its streaming route                         */
#define SCALECOM_Q_LAST_CANDIDATES  3  /* last step's number of pre-filter survivors                          */
#define SCALECOM_Q_TOPK_BLOCKS      4  /* thread blocks of the persistent selection kernel                    */
#define SCALECOM_Q_KERNEL_LAUNCHES  5  /* kernels launched by this handle since creation                      */
#define SCALECOM_Q_FUSED_SMALL      6  /* thread blocks of the one-kernel step if scalecom_step would use it for
                                          16-byte aligned vectors (see SCALECOM_OPT_FUSED_SMALL), else 0        */
#define SCALECOM_Q_PHASE_STAMP0     100 /* +i, i < 13: low 32 bits of the GPU nanosecond timer at phase boundary i of
                                          the last top-k selection kernel (profiling aid): 0-7 as seen by block 0
                                          (start; sample, barrier, bound; filter pass; barrier; k-th key located;
                                          winners marked), 8-9 start and end of the completing work of the block
                                          that finished last, 10-12 inside the marking phase of block 0        */
int scalecom_query(scalecom_ctx* ctx, int item, int64_t* out);

/*
 * With SCALECOM_OPT_KERNEL_TIMING on, every step brackets its kernels with CUDA
 * events on the handle's stream (the most recent 256 steps are kept).  This call
 * waits for the stream, writes the durations in milliseconds SUMMED over the
 * steps recorded since the previous call (or since timing was switched on) and
 * forgets them: ms[0] selection (step 2), ms[1] learner pass (steps 1, 3, 4, and
 * 5 when fused), ms[2] separate weight update (0 when fused); *nsteps receives
 * the number of steps summed.  BAD_STATE when timing is off.
 */
int scalecom_kernel_ms(scalecom_ctx* ctx, float ms[3], int32_t* nsteps);

/*
 * Leader selection (step 2 only) for callers that cannot allocate device memory.
 * The paper has no counterpart: this entry point exists for deployment reasons.
 * A process whose GPU memory is already fully owned by a framework's caching
 * allocator, or capped by a fixed partition, gets an error from cudaMalloc; a
 * latency-critical loop cannot afford the device-wide synchronisation cudaMalloc
 * implies.  Here the selection kernels' scratch is a fixed array inside the
 * library image (about 11 MB per GPU that uses this entry point, held until the
 * process exits), and the call itself performs no cudaMalloc, cudaFree or any
 * other allocating call.  The CUDA runtime places that array in device memory
 * when the module is first used on a device, i.e. during the FIRST call on that
 * device: make that call at start-up, before the rest of the application takes
 * the GPU's memory (a first call made with no memory left fails with ALLOC) and
 * before any stream capture begins.  Only the calls after it are allocation-free.
 *   g, m        DEVICE fp32[d]: the leader's gradient and memory; keys are |m + g|.
 *   d           1 <= d <= SCALECOM_STATIC_MAX_D (larger vectors: INVALID_ARG; use a handle).
 *   k           1 <= k <= d.
 *   out_idx     DEVICE int32[k], written: the same ascending index list scalecom_step returns.
 *   dev_status  DEVICE int32, optional (NULL to skip): receives 0, or 5 if a bounded
 *               in-kernel wait expired, or 7 if a consistency check failed (out_idx is
 *               then undefined).
 *   cuda_stream cudaStream_t as void*; the work is asynchronous on it, on the current device.
 * The first call on each device also looks up the array's device address and the
 * kernels' launch limits.
 * All calls on a device share the one array, which still holds the previous
 * call's contents: each call clears what must start at zero, and two calls whose
 * GPU work overlaps (different streams, no dependency) race on it -- order them.
 * Errors: NULL_PTR, INVALID_ARG, ALIAS, ALLOC (first call on a device only), CUDA.
 */
#define SCALECOM_STATIC_MAX_D (1 << 20)
int scalecom_topk_static(const float* g, const float* m, int64_t d, int64_t k, int32_t* out_idx,
                         int32_t* dev_status, void* cuda_stream);

/*
 * Diagnostics of Sections 2-3; they read the state and change none of it (scratch of about 8.2*d
 * bytes is allocated on first use; both calls wait for the stream).
 *
 * scalecom_overlap: Eq. 5's d between the leader's top-k set I^k(acc_L), L = t mod n, and the "true
 * top-k" set I^k((1/n) sum_i acc_i) of the all-reduced error-feedback gradient: the Hamming distance of
 * the two indicator vectors is H = 2d, 0 <= d <= k (Fig. 3 plots d/k; Lemma 1 turns it into the
 * contraction factor).  grads / mem as in scalecom_step, all read only.
 *
 * scalecom_cosine_distance: 1 - x.y / (|x| |y|) of two DEVICE fp32[d] vectors, e.g. two learners'
 * memories (Section 2, "memory similarity"); products accumulated in double.
 */
int scalecom_overlap(scalecom_ctx* ctx, const float* const* grads, const float* const* mem, int64_t t,
                     int64_t* host_hamming_d);
int scalecom_cosine_distance(scalecom_ctx* ctx, const float* x, const float* y, double* host_out);

/*
 * With SCALECOM_OPT_KERNEL_SPANS on: waits for the stream and writes the in-kernel durations in
 * milliseconds (first block start to last block end, no launch gap, no event overhead) SUMMED over the
 * steps recorded since the previous call (at most the last 256): ms[0] selection kernel, ms[1] learner
 * pass; *nsteps receives the number of steps summed.  BAD_STATE when the option is off.
 */
int scalecom_kernel_span_ms(scalecom_ctx* ctx, float ms[2], int32_t* nsteps);

/* Static, never NULL. */
const char* scalecom_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SCALECOM_H */
