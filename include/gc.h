/*
 * gc.h -- C ABI of libgc: sparse gradient compression with error feedback on one
 * NVIDIA B200 (sm_100a).
 *
 * Per training iteration and per worker the library
 *   1. folds the error-feedback residual into the fresh gradient      a = g + r   (fp32)
 *   2. selects, per tensor, the k entries of largest magnitude (exact top-k, ties to the
 *      lower index) or, in threshold mode, every entry at or above a sampled threshold
 *   3. emits them as index-sorted (uint32 flat index, fp32 value) pairs
 *   4. writes the residual back: +0 where sent, a elsewhere
 * and, across W workers,
 *   5. decodes and sums the W sparse sets into one dense fp32 buffer in worker order.
 *
 * Where the definitions come from.  The source paper of this project (erasure-coded fault
 * tolerance for recommendation-model training) defines none of these steps; its only words
 * on gradient compression are a remark in its Section 3.3.2 that its own deltas are dense.
 * Every operation below therefore follows the problem statement of the benchmark workload,
 * and each comment says which clause.
 *
 * Conventions
 *   - All tensors of a plan live back to back in one flat fp32 buffer ("flat layout");
 *     indices in the output are offsets into that flat buffer.
 *   - "device" pointers are CUDA device memory on the plan's device; "host" pointers are
 *     ordinary process memory.  The caller owns every buffer it passes in, including the
 *     workspace; the plan owns only its own small host and device tables.
 *   - gc_compress and gc_decompress_accumulate enqueue work on the given stream and return
 *     without synchronising (they may be captured in a CUDA graph; a plan option must not be
 *     changed between capture and replay).  No call allocates device memory except gc_plan.
 *   - A plan is bound to one device.  Every call that touches the device (compress, decode,
 *     gc_last_*, gc_compress_host) must be made while that device is the current one and
 *     returns GC_E_INVALID otherwise; gc_plan leaves the caller's current device as it was.
 *   - Return value: 0 = GC_OK, negative = error, positive = warning.  Conditions detected on
 *     the device (truncation in threshold mode, an internal wait that ran out) are written
 *     to a status word at the head of the workspace; read it with gc_last_status.
 *   - Nothing here aborts, throws or traps.
 *
 * Limits: total elements per plan <= 2^31 - 1; at most GC_MAX_WORKERS sparse sets per
 * gc_decompress_accumulate call (chain calls with zero_first = 0 for more).
 */
#ifndef GC_H_
#define GC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gc_plan_s gc_plan_t;

/* status codes */
#define GC_OK             0
#define GC_E_INVALID     (-1)   /* bad argument (null pointer, misaligned buffer, density out of (0,1]) */
#define GC_E_UNSUPPORTED (-2)   /* not available in this build / on this device                        */
#define GC_E_CUDA        (-3)   /* a CUDA runtime call failed; see gc_last_cuda_error                   */
#define GC_E_TOO_LARGE   (-4)   /* size beyond a stated limit                                           */
#define GC_E_TIMEOUT     (-5)   /* a bounded device-side wait gave up (device status only)              */
#define GC_W_TRUNCATED     1    /* threshold mode: more hits than capacity; the rest stayed in r       */

/* selection modes */
#define GC_TOPK       0
#define GC_THRESHOLD  1

#define GC_MAX_WORKERS 64

/* gc_plan_query keys.  "tensor" is ignored for plan-wide keys. */
#define GC_Q_N_TENSORS          0   /* number of tensors                                            */
#define GC_Q_TOTAL_N            1   /* elements in the flat buffer                                  */
#define GC_Q_TOTAL_CAP          2   /* length of out_idx / out_val (sum of per-tensor capacities)   */
#define GC_Q_WORKSPACE_BYTES    3   /* bytes of device workspace gc_compress / decode need          */
#define GC_Q_TENSOR_N           4   /* elements of tensor t                                         */
#define GC_Q_TENSOR_K           5   /* k of tensor t = min(n, max(1, ceil(density*n)))              */
#define GC_Q_TENSOR_CAP         6   /* output capacity of tensor t (= k in top-k mode)              */
#define GC_Q_TENSOR_OFFSET      7   /* first flat index of tensor t                                 */
#define GC_Q_TENSOR_OUT_OFFSET  8   /* first output slot of tensor t                                */
#define GC_Q_TENSOR_STRIDE      9   /* threshold mode: sampling stride used for tensor t            */
#define GC_Q_MODE              10
#define GC_Q_KERNEL_LAUNCHES   11   /* kernels + memsets enqueued by the library so far (host count) */
#define GC_Q_CANDIDATE_CAPACITY 12  /* slots of the internal candidate list (top-k mode)            */
#define GC_Q_COMPRESS_ROUTE     13  /* which kernels gc_compress takes for this plan: GC_ROUTE_*    */

/* values of GC_Q_COMPRESS_ROUTE (a diagnostic: the result never depends on the route) */
#define GC_ROUTE_NONE             0 /* nothing to launch (host-only plan, or no elements)                      */
#define GC_ROUTE_TOPK_ONE         1 /* one cooperative launch, one-tensor kernel                               */
#define GC_ROUTE_TOPK_MANY        2 /* one cooperative launch, many-tensor kernel                              */
#define GC_ROUTE_TOPK_GENERAL     3 /* one cooperative launch, general candidate kernel (global histograms per
                                       level): plans the two kernels above do not take -- candidate sets too
                                       large for a CTA's region (densities of several per cent on large
                                       tensors), tensors beyond their tile limits, unsampled tensors          */
#define GC_ROUTE_TOPK_STAGED      4 /* the general candidate path as separate launches                         */
#define GC_ROUTE_EXACT            5 /* exact multi-pass kernels only                                           */
#define GC_ROUTE_THRESHOLD_ONE    6 /* threshold mode, one cooperative launch, one-tensor kernel               */
#define GC_ROUTE_THRESHOLD_MANY   7 /* threshold mode, one cooperative launch, many-tensor kernel              */
#define GC_ROUTE_THRESHOLD_STAGED 8 /* threshold mode, sample levels and the emission as separate launches     */

/*
 * gc_plan -- describe the flat gradient once; computes k per tensor, output offsets and the
 * workspace size.  (Problem statement: "top-k at density d applied per tensor" for layer-wise
 * workloads, "global top-k" when the model is given as one tensor.  k = min(n, max(1,
 * ceil(density * n))) with density in double precision -- the statement prints k = 10,486
 * for 1 % of 1,048,576 elements, which excludes a floor.)
 *
 *   out            host; receives the new plan
 *   device         CUDA device ordinal the plan is bound to; -1 = host-only plan that answers
 *                  gc_plan_query but makes every compute call return GC_E_UNSUPPORTED
 *   n_tensors      number of tensors (may be 0)
 *   sizes          host; n_tensors element counts (zeros allowed); the tensors are laid back
 *                  to back in that order in every flat buffer
 *   density        in (0, 1]
 *   mode           GC_TOPK or GC_THRESHOLD
 *   sample_stride  threshold mode: sample one 4-element group out of this many (0 = 64);
 *                  tensors of <= 65,536 elements are always sampled in full.  Every sampled
 *                  group is a scattered 32-byte DRAM access in g and in r, and on tensors of
 *                  100M elements and more that is a tenth of the call at stride 64 (110M
 *                  elements: 262 us against 238 us at stride 512, whose sample still holds
 *                  214,000 elements); the stride is part of the result's definition, so the
 *                  library does not choose it
 *   cap_factor     threshold mode: per-tensor output capacity = min(n, ceil(cap_factor*k))
 *                  (0 = 2.0; must be >= 1)
 * Allocates a few KB of device memory for the tensor table (freed by gc_destroy).
 * Errors: GC_E_INVALID, GC_E_TOO_LARGE (total > 2^31-1), GC_E_CUDA.
 */
int gc_plan(gc_plan_t **out, int device, uint32_t n_tensors, const uint64_t *sizes,
            double density, int mode, uint32_t sample_stride, double cap_factor);

/*
 * gc_plan_set_option -- host; tune or steer a plan before it is used (never while work that
 * uses it is in flight).  The selected set never depends on these options, only the route.
 *   GC_OPT_PATH                  GC_PATH_AUTO (default): one-pass candidate path with the exact
 *                                multi-pass kernels as its safety net, all in one cooperative launch;
 *                                GC_PATH_STAGED: sample, candidate extraction, candidate select and
 *                                emission as separate launches (global histograms per level);
 *                                GC_PATH_EXACT: multi-pass kernels only
 *   GC_OPT_SAMPLE_RANK_PERMILLE  scales the sample rank that sets the candidate threshold
 *                                (1000 = default; small values make the candidate set too small
 *                                and so exercise the safety net -- a testing aid).  The workspace
 *                                size reported at plan creation stays sufficient.
 *   GC_OPT_CANDIDATE_CAPACITY    lowers the candidate-list capacity (testing aid for overflow)
 *   GC_OPT_DECODE_ROUTE          which tiled decode kernel gc_decompress_accumulate and
 *                                gc_decompress_apply_momentum take: GC_DECODE_AUTO (default) picks
 *                                by the expected number of pairs per worker and 8192-element tile --
 *                                GC_DECODE_NARROW pre-loads 4 x (256 / W) pairs per worker in
 *                                registers, GC_DECODE_WIDE keeps up to 4096 / W pairs per worker in
 *                                shared-memory rings (many workers, dense lists).  Same result.
 *   GC_OPT_DECODE_ORDER          GC_ORDER_FIXED (default): every element's contributions are added in
 *                                worker order 0..W-1, so the result is bit-reproducible.
 *                                GC_ORDER_ANY: the contributions of an element that several workers
 *                                hit are added in an order that may change from run to run (shared-
 *                                memory atomics; faster for 16 and more workers); each result lies
 *                                within (hits - 1) x 2^-24 x sum |values| of the fixed-order one and
 *                                equals it where one worker hits.  Applies to the tiled decode of
 *                                both decode calls; lists with counts of many-tensor plans keep
 *                                their fixed-order kernel.
 *   GC_OPT_WORKSPACE_PRIVATE     0 (default): every gc_compress starts with a launch that clears the
 *                                control block of the workspace, so a workspace may be shared by
 *                                plans or refilled by the caller between calls.  1: the caller
 *                                promises that between two gc_compress calls of THIS plan on a
 *                                workspace nothing else writes to it (the decode calls of this plan
 *                                are fine, and so is a zero-filled or a fresh workspace for the first
 *                                call).  The fused top-k kernels (one tensor, many tensors, and the
 *                                shared launch of gc_compress_workers) clean the control block as
 *                                they go (each section right after the grid barrier that follows its
 *                                last reader, the rest at the start of the next launch), so their
 *                                calls then do without the clearing launch.  A broken promise is
 *                                caught by a mark in the workspace header: the kernel leaves at once
 *                                and GC_E_INVALID is recorded in the device status; after any error
 *                                status read through gc_last_status the next call clears again.
 *                                The threshold, staged and exact routes ignore the option.
 * Errors: GC_E_INVALID (unknown option or value), GC_E_CUDA.
 */
#define GC_OPT_PATH                  0
#define GC_OPT_SAMPLE_RANK_PERMILLE  1
#define GC_OPT_CANDIDATE_CAPACITY    2
#define GC_OPT_DECODE_ROUTE          3
#define GC_DECODE_AUTO   0
#define GC_DECODE_NARROW 1
#define GC_DECODE_WIDE   2
#define GC_OPT_DECODE_ORDER          4
#define GC_OPT_WORKSPACE_PRIVATE     5
#define GC_ORDER_FIXED   0
#define GC_ORDER_ANY     1
#define GC_PATH_AUTO   0
#define GC_PATH_EXACT  1
#define GC_PATH_STAGED 2
int gc_plan_set_option(gc_plan_t *plan, int option, uint64_t value);

/* gc_plan_query -- host-side lookup of plan facts; never touches the device.
 * Errors: GC_E_INVALID for an unknown key, a null pointer or tensor >= n_tensors. */
int gc_plan_query(const gc_plan_t *plan, int what, uint32_t tensor, uint64_t *value);

/*
 * gc_compress -- one worker, one iteration (problem statement: "fold the error-feedback
 * residual into the fresh gradient, select the top-k entries by magnitude, compact them
 * into (index, value) pairs, write back the residual").
 *
 *   grad       device, const, fp32[total_n], 16-byte aligned
 *   residual   device, in/out, fp32[total_n], 16-byte aligned; on return (after the stream
 *              drains) holds +0 where an entry was sent and g + r elsewhere
 *   out_idx    device, uint32[total_cap]; pairs of tensor t start at its out offset and are in
 *              ascending flat index; magnitude = bit pattern with the sign cleared, ties go to
 *              the lower index, so the selected set is unique
 *   out_val    device, fp32[total_cap]; bit copy of a = g + r at each sent index
 *   out_count  device, uint32[2 * n_tensors] or NULL: [t] = pairs written for tensor t,
 *              [n_tensors + t] = hits (threshold mode: entries at or above the threshold,
 *              which may exceed the capacity; top-k mode: both equal k)
 *   workspace  device, GC_Q_WORKSPACE_BYTES bytes, 256-byte aligned; scratch -- contents
 *              need not survive between calls, but two calls in flight at once must not
 *              share one workspace
 *   stream     cudaStream_t (0 = legacy default stream)
 * Threshold mode (own reading; nothing external defines it): sample = elements whose
 * 4-element group number within the tensor is a multiple of the stride; tau = the
 * max(1, ceil(density*|sample|))-th largest sampled magnitude; every element with magnitude
 * >= tau is a hit; hits are sent in index order up to the capacity.
 * Errors: GC_E_INVALID (null / misaligned pointer), GC_E_CUDA.  Asynchronous.
 */
int gc_compress(gc_plan_t *plan, const float *grad, float *residual,
                uint32_t *out_idx, float *out_val, uint32_t *out_count,
                void *workspace, void *stream);

/*
 * gc_compress_bf16 -- gc_compress for a gradient stored as bfloat16 (total_n 16-bit values, 16-byte
 * aligned, same flat layout).  Every value is widened exactly (16 zero bits appended) and then
 * treated as the fp32 gradient of gc_compress: a = fl32(g + r), same selection, same outputs,
 * fp32 residual.  Reads 2 instead of 4 bytes per element of g: 10n + 8k bytes per call.
 * No counterpart in the source paper.  Top-k mode with the default route only
 * (GC_E_UNSUPPORTED otherwise, and for plans the two fused top-k kernels do not take).
 */
int gc_compress_bf16(gc_plan_t *plan, const void *grad_bf16, float *residual,
                     uint32_t *out_idx, float *out_val, uint32_t *out_count,
                     void *workspace, void *stream);

/*
 * gc_compress_workers -- gc_compress for W simulated workers of one plan in one go: worker w
 * folds residuals[w] into grads[w], writes its pairs to out_idx[w] / out_val[w] (and its counts
 * to out_count[w]) and uses workspaces[w]; every result is exactly what W separate gc_compress
 * calls would give.  No counterpart in the source paper: the problem statement only says that
 * the 8-worker workload runs its workers on one GPU, and this call is how that is done without
 * paying a kernel's cold phases once per worker.  For top-k plans of several tensors on the
 * default route the workers share cooperative launches: the resident CTAs are dealt out evenly
 * among up to 12 workers per launch, each group of CTAs runs the many-tensor kernel on its own
 * worker and synchronises only with itself.  Every other plan (one tensor, threshold mode,
 * GC_PATH_EXACT / GC_PATH_STAGED) is served by W consecutive gc_compress calls.
 *
 *   W            1..GC_MAX_WORKERS (0 does nothing)
 *   grads, residuals, out_idx, out_val, workspaces
 *                host arrays of W device pointers, each as in gc_compress; no two workers may
 *                share a residual, an output array or a workspace (GC_E_INVALID): the workers'
 *                kernels run at the same time
 *   out_count    host array of W device pointers, or NULL for none
 * Errors: GC_E_INVALID, GC_E_TOO_LARGE (W > GC_MAX_WORKERS), GC_E_CUDA.  Asynchronous.
 */
int gc_compress_workers(gc_plan_t *plan, uint32_t W, const float *const *grads, float *const *residuals,
                        uint32_t *const *out_idx, float *const *out_val, uint32_t *const *out_count,
                        void *const *workspaces, void *stream);

/*
 * gc_decompress_accumulate -- decode W sparse sets and sum them into a dense buffer
 * (problem statement: "decode and sum the sparse contributions of W simulated workers into
 * one dense buffer"; a sum, not a mean).  For every flat index the additions happen in
 * worker order 0..W-1 in fp32, so the result is reproducible bit for bit.
 *
 *   W          number of sparse sets, 1..GC_MAX_WORKERS (0 with zero_first just clears)
 *   idx, val   host arrays of W device pointers, each laid out as gc_compress wrote them
 *   count      host array of W device pointers to the out_count arrays gc_compress wrote, or
 *              NULL = every tensor carries exactly its capacity (top-k mode)
 *   dense_out  device, fp32[total_n]
 *   zero_first non-zero: dense_out is set to +0 first; zero: sums are added to its content
 *   workspace  device, GC_Q_WORKSPACE_BYTES bytes, 256-byte aligned; either one that
 *              gc_compress has used (ordered before this call on the stream) or zero-filled
 *              by the caller -- this call does not reset the status word
 * With count = NULL every list must be exactly as gc_compress wrote it in top-k mode (total_cap
 * pairs, ascending index): the dense buffer is then built tile by tile in shared memory and
 * written once; so are one-tensor plans with count arrays (the list's length is its count).
 * Plans of several tensors with count arrays take the same tile loop cut at the tensor
 * boundaries: tensor t's live pairs are slots [out offset of t, + count[t]) of the list, the
 * slots up to its capacity are ignored (GC_OPT_DECODE_ROUTE and GC_OPT_DECODE_ORDER do not
 * apply to such lists: one kernel, fixed worker order).  A live pair whose index lies outside
 * its tensor is skipped and GC_E_INVALID is recorded.
 * An index >= total_n (or a list that is not ascending) is skipped and GC_E_INVALID is recorded
 * in the device status.
 * Errors: GC_E_INVALID, GC_E_TOO_LARGE (W > GC_MAX_WORKERS), GC_E_CUDA.  Asynchronous.
 */
int gc_decompress_accumulate(gc_plan_t *plan, uint32_t W,
                             const uint32_t *const *idx, const float *const *val,
                             const uint32_t *const *count,
                             float *dense_out, int zero_first,
                             void *workspace, void *stream);

/*
 * gc_last_status -- copy the device status word of a workspace to the host.  This call
 * SYNCHRONISES the stream.  *status receives GC_OK, GC_W_TRUNCATED, GC_E_TIMEOUT or
 * GC_E_INVALID as recorded by the kernels since the last gc_compress on that workspace;
 * *detail (may be NULL) receives a code-specific value (e.g. the tensor that overflowed).
 */
int gc_last_status(gc_plan_t *plan, const void *workspace, void *stream,
                   int32_t *status, uint64_t *detail);

/*
 * gc_decompress_apply_momentum -- the decode with the optimizer fused behind it: the summed
 * gradient is never written out.  For every element i:
 *     s_i  = sum over workers w = 0..W-1, in that order, of the values sent for i (+0 if none)
 *     v_i' = fl(fl(momentum * v_i) + fl(scale * s_i))
 *     p_i' = fl(p_i - fl(lr * v_i'))
 * (momentum SGD in its accumulate-then-step form; scale = 1 for a sum, 1/W for a mean; every
 * operation rounded once, no fused multiply-add).  No counterpart in the source paper; it is
 * the fusion a data-parallel step performs right after aggregation, and it replaces 24 bytes
 * per element of traffic (write the sum, read it again with p and v, write p and v) by 16.
 *   idx, val, count  as for gc_decompress_accumulate
 *   param, velocity  device, fp32[total_n], 16-byte aligned, updated in place
 *   workspace        device; only its status word is written (out-of-range or unordered
 *                    index -> GC_E_INVALID recorded, the entry is skipped)
 * Errors: GC_E_INVALID, GC_E_TOO_LARGE (W > GC_MAX_WORKERS), GC_E_UNSUPPORTED, GC_E_CUDA.
 * Asynchronous.
 */
int gc_decompress_apply_momentum(gc_plan_t *plan, uint32_t W, const uint32_t *const *idx,
                                 const float *const *val, const uint32_t *const *count,
                                 float *param, float *velocity, float lr, float momentum, float scale,
                                 void *workspace, void *stream);

/*
 * gc_compress_host -- gc_compress for a gradient that lives in HOST memory, with the
 * compressed pairs returned to HOST memory (what a worker would hand to its network stack).
 * Enqueues: copy host_grad -> grad_staging, gc_compress, copy the pairs device -> host.  The
 * compress and the copy of the pairs run on the caller's stream.  The host -> device copy runs
 * on a stream owned by the plan and is ordered after the last compress that read the same
 * grad_staging buffer, so a caller that alternates two staging buffers (and two host buffers)
 * gets the next gradient's copy under way while the current one is compressed and its pairs
 * travel back.  (While gc_profile_enable is on, the copy stays on the caller's stream.)
 * host_grad must not change before the caller's stream has passed this call.  No counterpart in
 * the source paper; it exists so that end-to-end throughput including both PCIe copies can be
 * measured through this ABI.
 *
 *   host_grad     host (pinned for a truly asynchronous copy), fp32[total_n]
 *   grad_staging  device, fp32[total_n], 16-byte aligned; overwritten
 *   host_idx/val  host (pinned recommended), uint32/fp32[total_cap]; valid after the stream drains
 *   the other arguments are those of gc_compress
 * Bytes moved per call: 4*total_n host->device, 8*total_cap device->host.
 */
int gc_compress_host(gc_plan_t *plan, const float *host_grad, float *grad_staging, float *residual,
                     uint32_t *out_idx, float *out_val, uint32_t *out_count,
                     uint32_t *host_idx, float *host_val, void *workspace, void *stream);

/*
 * Per-kernel timing with CUDA events (a measuring aid; not part of the hot path).
 * gc_profile_enable(plan, max_records): from now on every kernel or memset the library
 * enqueues for this plan is bracketed by a pair of CUDA events recorded on the same stream,
 * up to max_records launches (later ones run untimed).  max_records = 0 switches timing off
 * and frees the events.  gc_profile_read synchronises the device, sums the elapsed time and
 * the launches per kernel id (GC_K_*; arrays of GC_K_COUNT entries) and clears the records.
 */
#define GC_K_CLEAR_CTRL     0   /* zeroing of the workspace control block (and of out_count) */
#define GC_K_FOLD_HIST      1   /* fold + level-0 histogram (reads g, r; writes r)        */
#define GC_K_HIST_REFINE    2   /* level-1 / level-2 histogram over r                      */
#define GC_K_COMPACT        3   /* ordered compaction + residual zeroing                   */
#define GC_K_DECODE_CLEAR   4   /* memset of the dense output                              */
#define GC_K_DECODE_ADD     5   /* sparse set added into the dense output                  */
#define GC_K_COPY           6   /* host<->device copies of gc_compress_host                */
#define GC_K_OTHER          7
#define GC_K_SAMPLE         8   /* strided sample histograms that set the candidate threshold */
#define GC_K_FOLD_CAND      9   /* fold + candidate extraction (reads g, r; writes r, candidates) */
#define GC_K_CAND_REFINE   10   /* radix-select levels over the candidate lists              */
#define GC_K_CAND_COMPACT  11   /* ordered emission from the candidate lists                 */
#define GC_K_THRESHOLD_EMIT 12  /* threshold mode: fold + send everything at or above tau    */
#define GC_K_FUSED         13   /* whole top-k compress as one cooperative launch            */
#define GC_K_SMALL         14   /* small tensors, each selected exactly by one CTA           */
#define GC_K_DECODE_TILES  15   /* tiled decode: W sorted lists summed into the dense buffer */
#define GC_K_COUNT         16
int gc_profile_enable(gc_plan_t *plan, uint32_t max_records);
int gc_profile_read(gc_plan_t *plan, float *total_ms, uint32_t *launches);
const char *gc_kernel_name(int kernel_id);

/*
 * gc_compress_noalloc -- exact top-k compression of ONE tensor without any device allocation
 * (nothing in the source paper corresponds to this call; it is an addition of this library).
 *
 * Who needs it: code that runs where allocating is off the table -- a gradient hook called by
 * a training framework whose caching allocator already owns nearly all device memory (so a
 * cudaMalloc can fail, and would in any case stall every stream of the device while it
 * runs), or a latency-bound loop that may not touch the allocator.  Such callers cannot use
 * gc_plan, which allocates its tensor table.  Here the scratch the kernels need (histograms,
 * tile words, selection record; 41,728 bytes, about 41 KB) is a fixed array inside the library image, so
 * every GPU that loads libgc carries it until the process exits.
 *
 *   grad, residual  device, fp32[n], 16-byte aligned; residual is in/out exactly as in gc_compress
 *   n               elements, at most GC_NOALLOC_MAX_N; larger -> GC_E_TOO_LARGE (use gc_plan)
 *   k               entries to keep, k <= n (k > n -> GC_E_INVALID); same selection rule,
 *                   same output order and same residual rule as gc_compress in top-k mode.
 *                   k = 0 sends nothing and still folds: the residual becomes g + r
 *   out_idx/out_val device, uint32/fp32[k] (may be NULL when k = 0)
 *   device_status   device int32 or NULL: receives GC_OK or GC_E_TIMEOUT when the work is done
 *                   (on every path that returns GC_OK, n = 0 and k = 0 included)
 *   stream          cudaStream_t; the call is asynchronous
 * The current device is used.  The first call on each device resolves the device address of
 * the array (cudaGetSymbolAddress) and sizes its grids; make that first call outside any
 * stream capture.  All calls on a device share the one array: each call clears what it
 * needs, so back-to-back calls on one stream are fine, but two calls whose kernels can
 * overlap on the GPU (different streams, different threads) race on it -- serialise them.
 * Calls no cudaMalloc/cudaFree and no allocating library routine.
 */
#define GC_NOALLOC_MAX_N (1u << 24)
int gc_compress_noalloc(const float *grad, float *residual, uint32_t n, uint32_t k,
                        uint32_t *out_idx, float *out_val, int32_t *device_status, void *stream);

/*
 * gc_last_counters -- diagnostic twin of gc_last_status (SYNCHRONISES the stream): copies
 * three counters of the most recent gc_compress on this workspace to the host:
 *   counters[0] = candidates extracted by the one-pass path, counters[1] = 1 if the candidate
 *   list overflowed (every tensor was redone by the exact kernels), counters[2] = tensors
 *   whose candidate set was smaller than k (redone individually).
 */
int gc_last_counters(gc_plan_t *plan, const void *workspace, void *stream, uint32_t counters[3]);

/*
 * gc_last_phase_times -- diagnostic (SYNCHRONISES the stream): durations in nanoseconds of the
 * phases of the most recent fused top-k launch on this workspace, as stamped by its first CTA
 * (phase i ends at barrier i).  *n_phases receives how many of ns[0..19] are valid.
 */
int gc_last_phase_times(gc_plan_t *plan, const void *workspace, void *stream, uint64_t ns[20],
                        uint32_t *n_phases);

/* gc_last_cuda_error -- host; the cudaError_t value of the most recent failed runtime call
 * made on behalf of this plan (0 if none). */
int gc_last_cuda_error(const gc_plan_t *plan);

/* gc_destroy -- free the plan and its device table.  NULL is accepted. */
int gc_destroy(gc_plan_t *plan);

/* gc_version -- ABI version of the loaded library (host, constant). */
uint32_t gc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GC_H_ */
