/*
 * libdeft — the gradient-selection hot path of DEFT (Yoon & Oh, "DEFT: Exploiting
 * Gradient Norm Difference between Model Layers for Scalable Gradient
 * Sparsification", ICPP 2023) for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Plain pointers and sizes only.  Pointer names end in `_h` (host memory)
 * or `_d` (device memory of the current CUDA device).  The library never allocates
 * or frees device memory: the caller owns every buffer, including the workspace
 * sized by deft_workspace_bytes().  Host calls are pure functions, thread-safe,
 * and touch no CUDA state.  Device calls enqueue work on `stream` (a cudaStream_t
 * passed as void*; NULL is the legacy default stream) and return without waiting;
 * results are valid once the stream has reached that point.
 *
 * Every call returns a deft_status: 0 = DEFT_OK, > 0 a warning (results valid),
 * < 0 an error (outputs unspecified unless stated).  Nothing throws or aborts.
 *
 * Vocabulary (Section 4 of the paper): the flat gradient vector has n_g elements;
 * Algorithm 2 cuts it into L contiguous "layers"; `layer_start[L+1]` holds their
 * boundaries in address order and a layer id is a position in that table; N is the
 * number of workers; k = d * n_g gradients are selected per step, k_l of them in
 * layer l.  One call of deft_select() does the work of ONE worker (rank).
 */
#ifndef DEFT_H_
#define DEFT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Every entry point is exported with default visibility; nothing else leaves the library. */
#if defined(__GNUC__)
#define DEFT_API __attribute__((visibility("default")))
#else
#define DEFT_API
#endif

typedef int32_t deft_status;

#define DEFT_OK                   0
#define DEFT_WARN_K_INEXACT       1   /* PAPER mode only: sum of k_l differs from k              */
#define DEFT_ERR_INVALID_ARG     -1   /* null pointer, non-positive size, unsorted table, ...    */
#define DEFT_ERR_INFEASIBLE_K    -2   /* EXACT mode needs L <= k <= n_g                          */
#define DEFT_ERR_NONFINITE_NORM  -3   /* a norm is NaN, infinite or negative; nothing written    */
#define DEFT_ERR_CAPACITY        -4   /* an output buffer or the workspace is too small          */
#define DEFT_ERR_CUDA            -5   /* a CUDA call failed; see deft_last_cuda_error()          */
#define DEFT_ERR_TOO_LARGE       -6   /* valid arguments, but one selection launch cannot hold them:
                                         see deft_select_launch_max_elems()                      */

#define DEFT_MODE_PAPER 0  /* Algorithm 3 exactly as listed                                      */
#define DEFT_MODE_EXACT 1  /* Algorithm 3 followed by an integer repair so that sum k_l == k     */

/* Load model of the bin packing (Algorithm 4). */
#define DEFT_COST_EQ3  0   /* cost_l = size_l * ln(k_l): Eq. 3                                     */
#define DEFT_COST_SIZE 1   /* cost_l = size_l: the bytes a worker scans (no counterpart in the paper) */

/* Largest layer a plan accepts (a layer's positions are 32-bit).  What one selection launch can
 * scan is smaller on today's devices: see deft_select_launch_max_elems(). */
#define DEFT_MAX_LAYER_ELEMS 2147483647LL

/*
 * Elements one selection launch can scan on the current CUDA device: every CTA (one per SM) owns
 * at most 4096 tiles of 2048 elements, so 148 SMs give 1 241 513 984.  A single layer, or the n
 * of deft_topk_baseline / deft_threshold_select, beyond this returns DEFT_ERR_TOO_LARGE (nothing
 * launched); so does a call whose share per CTA holds more than 256 layers of more than 16384
 * elements.  deft_select_update_all answers that status by running one launch per worker.
 * Host-side query; needs a current device.
 */
DEFT_API int64_t deft_select_launch_max_elems(void);

/* Human-readable name of a status code (static string). */
DEFT_API const char* deft_status_string(deft_status s);

/* The cudaError_t value behind the calling thread's most recent DEFT_ERR_CUDA (0 if none). */
DEFT_API int32_t deft_last_cuda_error(void);

/*
 * Diagnostic: which selection kernel later calls use.  single_pass = 0: the five-step kernel alone;
 * 1: the single-pass kernel whenever a call's layers allow it (at least half of its elements in sparse
 * layers of moderate k_l, at most 1024 layers of which at most 256 larger than 16384 elements); -1 (the default): the single-pass
 * kernel for such calls of 48 M elements or more, the five-step kernel for smaller ones.  Results never
 * differ.  Not thread-safe; for measurements and tests.
 */
DEFT_API void deft_debug_select_kernel(int32_t single_pass);

/*
 * Diagnostic: how the single-pass kernel reads the vector.  on != 0 (the default): whole tiles come
 * through a ring of sixteen 8 KB stages in shared memory filled by bulk copies (cp.async.bulk, one
 * mbarrier per stage), which keeps 128 KB per SM in flight whatever the warps are busy with; the ring
 * takes its room from the shared-memory staging area.  on = 0: every warp loads its tile into
 * registers with sixteen 16-byte loads per lane and waits for them.  Results never differ.  Not
 * thread-safe; for measurements and tests.
 */
DEFT_API void deft_debug_select_ring(int32_t on);

/*
 * Diagnostic: whether deft_step, when it runs all workers' selections in one launch on a vector the
 * single-pass kernel takes, stages during the accumulate pass.  on != 0 (the default): the kernel that
 * adds the gradient and sums the squares also puts every entry at or above its layer's remembered cut
 * into the layer's staging region (the cut is taken from where the previous step found the layer's
 * threshold, lowered by how much that has been moving from step to step: this step's norms and k_l do
 * not exist yet), and the selection launch, which then knows k_l, finishes every layer for which at
 * least k_l entries were staged without reading the vector at all; the other layers are read and
 * searched in full inside the same launch.  on = 0: the selection launch does its own read.  Results
 * never differ.  Not thread-safe; for measurements and tests.
 */
DEFT_API void deft_debug_step_staging(int32_t on);

/*
 * Diagnostic: when timing_d (DEVICE, 1024 x uint64, zeroed by the caller) is not NULL every
 * later selection launch records GPU-timer stamps in nanoseconds (max over CTAs) and counters.
 * Both kernels: [0] kernel start, [14] / [15] staged entries (max over CTAs or layers / total).
 * Five-step kernel: [1] end of the first read, [2] end of the second read, [3] level-3
 * histograms done, [4] per-tile counts done, [5] ordered write done, [6] small layers done,
 * [7] a second round of the first read done; inside the first read [8] histograms zeroed,
 * [9] tiles read, [10] flushed, [11] tickets taken; per CTA b: [16 + b] nanoseconds in the second
 * read, [176 + b] staged entries, [336 + b] local layers | local tiles << 16, [496 + b] why a cut
 * failed, [656 + b] nanoseconds in the ordered write, [816 + b] nanoseconds in the first read.
 * Single-pass kernel: [8] tables built, [1] tiles read, [2] staged entries handed to the layers'
 * regions, [10] last layer's candidates ranked, [5] layers finished, [6] small layers done,
 * [3] selected entries cleared; [20..26] nanoseconds, summed over the layers, in the finishing
 * CTA's phases (load, histogram, scan, candidates, per-tile counts, prefix, write); [12] the layer
 * with most staged entries (entries << 32 | layer << 20 | k), [13] most candidates, [28] layers
 * finished.
 * Pass NULL to switch it off.  Not thread-safe; not for production use.
 */
DEFT_API void deft_debug_select_timing(void* timing_d);

/* ------------------------------------------------------------------------------------------
 * Host planners (cheap, O(L) .. O(L^2); run on the CPU as in the paper)
 * ---------------------------------------------------------------------------------------- */

/*
 * Two-stage gradient vector partitioning — Algorithm 2, Section 4.1.
 * A tensor with size > n_g / N (tested as size * N > n_g) is cut into N contiguous
 * fragments of floor(size/N) elements, the first size % N of them one larger; all
 * other tensors stay whole.  Fragments and whole tensors are the "layers".  A
 * fragment that would be empty (size < N) is dropped.
 *   tensor_sizes_h[T]   in   element count of each tensor in address order, each >= 1
 *   layer_start_h[cap+1] out boundaries: layer l is [layer_start[l], layer_start[l+1])
 *   layer_tensor_h[cap] out  source tensor of each layer (may be NULL)
 *   L_out               out  number of layers
 * Errors: INVALID_ARG (null, T < 1, N < 1, a size < 1), CAPACITY (cap too small;
 * *L_out then holds the required count).
 */
DEFT_API deft_status deft_split_layers(const int64_t* tensor_sizes_h, int32_t T, int32_t N,
                              int64_t* layer_start_h, int32_t* layer_tensor_h, int32_t cap,
                              int32_t* L_out);

/*
 * Gradient-norm-based local k assignment — Algorithm 3, Section 4.2.
 * Layers are visited by descending norm (equal norms: lower id first).  With
 * norm_remain = the sum of the norms not yet visited (accumulated from the back,
 * so the last ratio is exactly 1) and k_remain = k minus what was handed out:
 *     k_temp = floor(k_remain * (norm_l / norm_remain))      (0 if norm_remain <= 0)
 *     k_l    = size_l if size_l < k_temp, else max(1, k_temp)
 * All of it in IEEE fp64 / int64, in exactly this operation order.
 * DEFT_MODE_PAPER stops there and returns DEFT_WARN_K_INEXACT when sum k_l != k
 * (the listing guarantees only "approximately k").  DEFT_MODE_EXACT then repairs the
 * sum with integers only: a shortfall is handed out in priority order up to each
 * layer's size; a surplus is taken back one per layer per round in priority order,
 * never below 1.
 *   norms_h[L], layer_size_h[L] in;  k_l_h[L] out (by layer id);  sum_k_out out (may be NULL)
 * Errors: INVALID_ARG, NONFINITE_NORM, INFEASIBLE_K (EXACT with k < L or k > n_g).
 */
DEFT_API deft_status deft_allocate_k(const double* norms_h, const int64_t* layer_size_h, int32_t L,
                            int64_t k, int32_t mode, int64_t* k_l_h, int64_t* sum_k_out);

/*
 * Bin-packing-based layer allocation — Algorithm 4, Section 4.3, Eq. 3.
 * cost_l = size_l * ln(k_l).  L times: the layer of largest remaining cost (lowest id
 * on ties) goes to the bin of smallest load (lowest id on ties).
 *   bin_of_layer_h[L] out  bin of each layer
 *   bin_load_h[N]     out  summed cost per bin (Eq. 4); may be NULL
 * Errors: INVALID_ARG (null, L < 1, N < 1, a size < 1, a k_l < 1).
 */
DEFT_API deft_status deft_partition(const int64_t* layer_size_h, const int64_t* k_l_h, int32_t L,
                           int32_t N, int32_t* bin_of_layer_h, double* bin_load_h);

/*
 * Algorithm 4's packing under a chosen load model.  DEFT_COST_EQ3 is deft_partition().
 * DEFT_COST_SIZE packs by layer size alone: the paper's model (Eq. 3) prices a sort-based
 * selection; the selection kernel here is linear in the elements a worker scans, so its time
 * follows bytes, and Eq. 3's cost-0 layers (k_l = 1) pile up in one bin.  k_l_h may be NULL for
 * DEFT_COST_SIZE.  Outputs and errors as deft_partition(); INVALID_ARG for an unknown model.
 */
DEFT_API deft_status deft_partition_model(const int64_t* layer_size_h, const int64_t* k_l_h, int32_t L, int32_t N,
                                          int32_t cost_model, int32_t* bin_of_layer_h, double* bin_load_h);

/*
 * Which bin a rank reads in a given iteration — Algorithm 4, lines 1-2:
 * (iteration % N + rank) % N.  Returns -1 on invalid arguments.
 */
DEFT_API int32_t deft_rank_bin(int64_t iteration, int32_t rank, int32_t N);

/*
 * The layer ids of one bin, ascending (alloc_part of Algorithm 4, line 20).
 *   my_layers_h[cap] out, n_my_out out.  Errors: INVALID_ARG, CAPACITY.
 */
DEFT_API deft_status deft_bin_layers(const int32_t* bin_of_layer_h, int32_t L, int32_t bin,
                            int32_t* my_layers_h, int32_t cap, int32_t* n_my_out);

/* ------------------------------------------------------------------------------------------
 * Device calls
 * ---------------------------------------------------------------------------------------- */

/*
 * Workspace size in bytes that is enough for every device call below on vectors of
 * up to max_elems elements cut into up to max_layers layers.  The workspace must be
 * 256-byte aligned.  Its contents need not be preserved between calls (the one area the
 * library itself carries from call to call, see deft_workspace_init, only affects speed).
 * Calls that share a workspace must not overlap on the GPU.
 */
DEFT_API size_t deft_workspace_bytes(int64_t max_elems, int32_t max_layers);

/*
 * Clears the one part of a workspace that is carried from call to call: per layer, where on
 * the magnitude axis the previous selection found its threshold and how well that has been
 * predicting the next one, from which the next selection of a model with n_layers layers
 * takes its speculative cut (see deft_select_planned), and a few counters.  Call it once
 * after allocating the workspace.  What that area holds never changes a result: stale or
 * arbitrary contents only decide whether a selection reads the vector once or twice (or, for
 * absurdly low cuts, how much it stages).  Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API deft_status deft_workspace_init(void* ws_d, size_t ws_bytes, int32_t n_layers, void* stream);

/*
 * Diagnostic counters of the single-pass selection kernel, summed over every call on this workspace
 * since deft_workspace_init: stats_h[0] layers it finished in one read, [1] layers whose remembered
 * cut failed (too few or far too many entries staged), [2] layers it had no usable cut for (nothing
 * remembered yet, or too dense); [1] and [2] were handed to the five-step kernel; [3] waits on the
 * bulk-copy ring that gave up (always 0 on a healthy device; see deft_debug_select_ring); [4] entries
 * staged for the layers counted in [0], modulo 2^32; [5..7] reserved (0).
 * stats_h: HOST, 8 x uint64.  Waits for `stream`.  Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API deft_status deft_select_stats(const void* ws_d, size_t ws_bytes, int32_t n_layers, uint64_t* stats_h,
                                       void* stream);

/*
 * Error-feedback accumulate fused with the per-layer gradient norms —
 * Algorithm 1 line 5 and the per-layer L2 norm that Section 4.2 ranks layers by.
 *   resid_acc_d[n_g]  in/out  on entry the local error e; on exit acc = e + grad
 *                             (one fp32 round-to-nearest add per element; the caller
 *                             passes the gradient already scaled by the learning rate)
 *   grad_d[n_g]       in      may be NULL: then nothing is written and the norms are
 *                             those of resid_acc_d as it stands
 *   layer_start_d[L+1] in     DEVICE copy of the layer table (int64, ascending)
 *   norms_d[L]        out     DEVICE, fp64: sqrt(sum of acc_i^2) per layer; squares are
 *                             summed in fp32 over runs of 8 elements and in fp64 beyond,
 *                             in a fixed order (bit-identical from run to run)
 * resid_acc_d and grad_d must be 16-byte aligned.  Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API deft_status deft_layer_norms(float* resid_acc_d, const float* grad_d, int64_t n_g,
                             const int64_t* layer_start_d, int32_t L, double* norms_d,
                             void* ws_d, size_t ws_bytes, void* stream);

/*
 * Layer-wise gradient selection for ONE worker — Algorithm 5, Section 4.4.
 * For each layer l in my_layers_h (ascending ids) selects the k_l entries of largest
 * magnitude.  Magnitudes compare as the IEEE-754 bit pattern with the sign cleared
 * (so NaN > Inf > finite, denormals are not flushed); equal magnitudes are won by the
 * lower index.  Output: the selected entries of all those layers in ascending global
 * index — signed values and int64 indices — exactly sum of k_l of them.
 * This one-shot form builds a single-rank plan, stages it through the workspace and
 * launches; per-step use should go through deft_plan_build/deft_select_planned.
 *   acc_d             in   the accumulated vector (16-byte aligned); not modified.  Reads are
 *                          128-bit: a layer that ends inside a 16-byte group makes the kernel
 *                          read the rest of that group too (so the buffer must be readable up to
 *                          the next multiple of 4 elements, which holds for any CUDA allocation)
 *   layer_start_h[L+1], k_l_h[L]   HOST tables for the whole model
 *   my_layers_h[n_my] HOST, ascending; n_my may be 0 (nothing is written)
 *   val_d, idx_d      out  DEVICE buffers of out_cap entries
 * Errors: INVALID_ARG (null, ids not ascending, k_l outside [1, size_l], a layer
 * larger than DEFT_MAX_LAYER_ELEMS), CAPACITY (out_cap < sum k_l, or ws too small), CUDA.
 */
DEFT_API deft_status deft_select(const float* acc_d, const int64_t* layer_start_h, const int64_t* k_l_h,
                        const int32_t* my_layers_h, int32_t n_my, float* val_d, int64_t* idx_d,
                        int64_t out_cap, void* ws_d, size_t ws_bytes, void* stream);

/*
 * deft_layer_norms for callers that cannot allocate device memory (no counterpart in the
 * paper; a deployment variant of the call above).  Some hosts of this library — a
 * communication hook that runs inside another framework's captured or memory-pooled
 * region, a plugin that is handed tensors but no allocator, code that runs after the
 * memory budget has been handed out — may not call cudaMalloc or any allocating routine,
 * so they have no workspace to pass.  This entry point takes none: its scratch (the
 * per-tile partial sums) is a fixed 128 KB array inside the library's device image.
 * Same arguments, same results (bit for bit) as deft_layer_norms.
 * Limit: ceil(n_g / 8192) + L + 1 must not exceed deft_layer_norms_static_max_slots()
 * (16384; about 100 M elements with a few thousand layers); larger inputs return
 * DEFT_ERR_CAPACITY and nothing is launched.
 * The first call on each device looks up the array's device address (a host-side query,
 * no allocation); make that first call outside of any stream capture.  All calls on one
 * device share the array, which keeps whatever the last call left in it; nothing in it has
 * to be cleared because every slot a call reads it has written first, but two calls that
 * overlap on the same GPU (different streams) race on it and must be serialised by the caller.
 * Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API int64_t deft_layer_norms_static_max_slots(void);
DEFT_API deft_status deft_layer_norms_static(float* resid_acc_d, const float* grad_d, int64_t n_g,
                                             const int64_t* layer_start_d, int32_t L, double* norms_d,
                                             void* stream);

/*
 * One step's host work in one call: Algorithm 3 (deft_allocate_k on the layer sizes implied by
 * layer_start_h), Algorithm 4 (deft_partition_model with cost_model), deft_plan_build and
 * deft_plan_upload, in that order, with the same results as the four separate calls; the
 * plan built here also carries the norms, with which the selection kernel scales the cuts it
 * remembers (speed only).  norms_h: HOST [L], this step's norms.
 * Outputs (HOST): k_l_h [L], *sum_k_out (may be NULL), bin_of_layer_h [L],
 * bin_load_h [N] (may be NULL), plan_h (plan_bytes_cap >= deft_plan_bytes(L, N); pinned
 * memory lets the upload overlap).  plan_d / ws_d: DEVICE, as for deft_plan_upload.
 * Returns DEFT_OK or DEFT_WARN_K_INEXACT (PAPER mode, sum of k_l differs from k; the plan is
 * built and uploaded all the same); errors as the four calls.
 */
DEFT_API deft_status deft_plan_step(const double* norms_h, const int64_t* layer_start_h, int32_t L, int32_t N,
                                    int64_t k, int32_t mode, int32_t cost_model, int64_t iteration,
                                    int64_t* k_l_h, int64_t* sum_k_out, int32_t* bin_of_layer_h, double* bin_load_h,
                                    void* plan_h, size_t plan_bytes_cap, void* plan_d, void* ws_d,
                                    size_t ws_bytes, void* stream);

/*
 * The per-step plan — Algorithm 4, lines 1-2 and 20 for every rank at once.
 * Once k_l (Algorithm 3) and the bins (Algorithm 4) of a step are known, the layer
 * lists of all N ranks are laid out in one position-independent blob: rank r owns the
 * layers of bin (iteration % N + r) % N, ascending.  The blob is built on the host
 * (deft_plan_build), copied to the device once (deft_plan_upload, which also clears the
 * per-layer counters in the workspace), and then deft_select_planned() runs any rank
 * with a single kernel launch and no further host-to-device traffic.  Ranks of one plan
 * use disjoint parts of the workspace.
 *
 * deft_plan_bytes: size of the blob for L layers and N ranks (0 on invalid arguments;
 * N <= 4096).
 * deft_plan_build: plan_h[plan_bytes] out (HOST; pinned memory makes the upload
 * asynchronous).  Errors: INVALID_ARG (null, a bin outside [0,N), k_l outside
 * [1, size_l], a layer above DEFT_MAX_LAYER_ELEMS), CAPACITY (blob too small).
 * deft_plan_rank_info: what rank `rank` will do: number of layers, elements scanned,
 * entries selected (sum of its k_l), and the sum of k over lower ranks (a convenient
 * offset into one shared output buffer).  Any out pointer may be NULL.
 * deft_plan_rank_table: the same four numbers for all N ranks at once (arrays of N).
 * deft_plan_upload: plan_d (DEVICE, 16-byte aligned, deft_plan_bytes) <- plan_h, on
 * `stream`.  Must be called again before the plan's ranks are re-run (the counters it
 * clears are consumed by the selection).  Errors: INVALID_ARG, CAPACITY (workspace), CUDA.
 */
DEFT_API size_t deft_plan_bytes(int32_t L, int32_t N);
DEFT_API deft_status deft_plan_build(const int64_t* layer_start_h, const int64_t* k_l_h,
                                     const int32_t* bin_of_layer_h, int32_t L, int32_t N,
                                     int64_t iteration, void* plan_h, size_t plan_bytes);
DEFT_API deft_status deft_plan_rank_info(const void* plan_h, int32_t rank, int32_t* n_layers_out,
                                         int64_t* elems_out, int64_t* k_out, int64_t* out_off_out);
DEFT_API deft_status deft_plan_rank_table(const void* plan_h, int32_t N, int32_t* n_layers_h,
                                          int64_t* elems_h, int64_t* k_h, int64_t* out_off_h);
DEFT_API deft_status deft_plan_upload(const void* plan_h, void* plan_d, void* ws_d, size_t ws_bytes,
                                      void* stream);

/*
 * Layer-wise gradient selection for rank `rank` of an uploaded plan — Algorithm 5.
 * Same result as deft_select() on that rank's layer list: the rank's selected entries in
 * ascending global index, exactly deft_plan_rank_info().k of them, written to val_d/idx_d
 * (the rank's own output; out_cap entries available).  A rank without layers writes
 * nothing.  plan_h is read on the host for the rank's sizes; plan_d is what the kernel
 * reads.  Errors: INVALID_ARG, CAPACITY (out_cap or workspace), CUDA.
 *
 * Speed, not results, depends on the workspace's history.  The kernel remembers per layer where
 * (in units of 1/256 octave of magnitude) it found the key a little below the k_l-th largest,
 * together with the layer's norm then.  The next call on the same workspace predicts the place
 * from the layer's norm now, lowers it by a running mean and twice a running deviation of the
 * earlier predictions' errors, and stages every entry above that cut while it reads the vector
 * once.  A layer for which at least k_l entries were staged is finished from those; any other
 * (nothing remembered, cut too high, far too many staged, dense layers) is read again and
 * searched in full.  Two kernels do this: a single-pass one for large calls, in which every
 * layer is finished by one CTA behind a grid barrier, and a five-step one (histogram levels of
 * 12 + 12 + 7 bits between grid barriers) for small calls and for the layers left over.
 */
DEFT_API deft_status deft_select_planned(const float* acc_d, const void* plan_h, const void* plan_d,
                                         int32_t rank, float* val_d, int64_t* idx_d, int64_t out_cap,
                                         void* ws_d, size_t ws_bytes, void* stream);

/*
 * Simulation driver: Algorithm 5 followed by the residual update (Algorithm 1 lines 11-12)
 * for the ranks rank_begin <= r < rank_end of an uploaded plan, one after the other on
 * `stream` — what N workers would each do on their own GPU, replayed on one.  Rank r
 * writes its entries at offset deft_plan_rank_info().out_off of val_d / idx_d (shared
 * buffers of out_cap >= total k entries) and zeroes them in acc_d (the selection kernel
 * does it on its way out: same result as deft_residual_update on the rank's indices).
 * Because ranks own disjoint layers the result equals zeroing the union after all selections.
 * events: NULL, or 3 cudaEvent_t per rank (HOST array of handles): [0] is recorded before
 * the rank's launch, [1] and [2] after it, for per-rank timing.
 * Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API deft_status deft_select_update_ranks(float* acc_d, int64_t n_g, const void* plan_h,
                                              const void* plan_d, int32_t rank_begin, int32_t rank_end,
                                              float* val_d, int64_t* idx_d, int64_t out_cap, void* ws_d,
                                              size_t ws_bytes, void* const* events, void* stream);

/*
 * All N workers' selections and residual updates of an uploaded plan in ONE launch: the same
 * bytes in val_d / idx_d / acc_d as deft_select_update_ranks(…, 0, N, …), for evaluating the
 * method (or simulating N workers) on a single device.  The paper has each worker run only its
 * own partition (Section 4.3); here the union of the partitions — every layer with its own
 * k_l, Algorithm 5 — is processed as one list in address order and every layer's entries land
 * where its worker's call would have put them.  Falls back to one launch per rank when the
 * plan exceeds what one launch can hold (more than 256 streamed layers or 4096 tiles per CTA)
 * or when the ranks' layers overlap.
 * Errors: INVALID_ARG, CAPACITY, CUDA.
 */
DEFT_API deft_status deft_select_update_all(float* acc_d, int64_t n_g, const void* plan_h, const void* plan_d,
                                            float* val_d, int64_t* idx_d, int64_t out_cap, void* ws_d,
                                            size_t ws_bytes, void* stream);

/*
 * One whole step of one worker (Algorithm 1 lines 5-6 and 11-12 with Algorithms 3-5 inside) in
 * one call: deft_layer_norms (acc = e + grad, norms), the norms' copy to the host, a wait for
 * them, deft_plan_step (local k, bins, plan, upload) and the selection + residual update —
 * of worker `rank` (its entries at val_d[0 ..], idx_d[0 ..]), or with rank = -1 of all N
 * workers in one launch (deft_select_update_all; every worker's entries at its plan offset).
 * The call returns after the selection has been enqueued; it blocks the host once, between
 * the norms and the planning.  norms_h: HOST [L].  If it is pinned memory the device can write
 * (cudaHostAlloc / cudaMallocHost), the norms kernel stores the norms there itself and the call
 * polls for them (at most two seconds, then it falls back) instead of copying and
 * synchronising the stream; any other host memory takes the copy + synchronise route.
 * events: NULL, or 4 cudaEvent_t handles (HOST array) recorded on `stream` before and after
 * the accumulate+norms kernels and before and after the selection launch.
 * With rank = -1 on a vector the single-pass selection kernel takes (48 M to 600 M elements, at most 1024
 * layers) the accumulate pass also stages every entry at or above its layer's remembered cut for the
 * selection, whose launch then reads nothing (see deft_debug_step_staging); the results are the same.
 * All other arguments, results and errors as in the calls it is made of.
 */
DEFT_API deft_status deft_step(float* resid_acc_d, const float* grad_d, int64_t n_g, const int64_t* layer_start_h,
                               const int64_t* layer_start_d, int32_t L, int32_t N, int64_t k, int32_t mode,
                               int32_t cost_model, int64_t iteration, int32_t rank, double* norms_d,
                               double* norms_h, int64_t* k_l_h, int64_t* sum_k_out, int32_t* bin_of_layer_h,
                               double* bin_load_h, void* plan_h, size_t plan_bytes_cap, void* plan_d,
                               float* val_d, int64_t* idx_d, int64_t out_cap, void* ws_d, size_t ws_bytes,
                               void* const* events, void* stream);

/*
 * Comparison sparsifiers of Section 3 (not part of DEFT; they reuse its selection kernel).
 *
 * Hard-threshold sparsifier (Section 3.2): selects every entry of acc_d[0, n) whose magnitude is
 * larger than |threshold| (strict; magnitudes compare as in Algorithm 5's selection, so a NaN
 * entry is larger than any threshold), one read of the vector.  Writes the first out_cap of
 * them in ascending index to val_d / idx_d (DEVICE; may be NULL when out_cap = 0) and the
 * total number to *count_d (DEVICE int64; may exceed out_cap).  zero_selected != 0 also clears
 * every selected entry in acc_d (the residual update), whether or not it fitted in out_cap.
 * ws_d: deft_workspace_bytes(n, 1).  Errors: INVALID_ARG (NaN threshold, NULL, misaligned, n
 * beyond DEFT_MAX_LAYER_ELEMS), CAPACITY (workspace), CUDA.
 */
DEFT_API deft_status deft_threshold_select(float* acc_d, int64_t n, float threshold, int32_t zero_selected,
                                           float* val_d, int64_t* idx_d, int64_t out_cap, int64_t* count_d,
                                           void* ws_d, size_t ws_bytes, void* stream);

/*
 * CLT-k (Sections 1, 3.1): the worker that selects in `iteration` — the leaders take turns —
 * or -1 for invalid arguments.  The leader's selection is deft_topk_baseline on its own vector.
 */
DEFT_API int32_t deft_clt_leader(int64_t iteration, int32_t N);

/*
 * CLT-k follower step: val_d[i] = acc_d[idx_d[i]], then acc_d[idx_d[i]] = +0, for the `count`
 * indices the leader broadcast (DEVICE; distinct, each in [0, n_g) — not checked).
 * Errors: INVALID_ARG, CUDA.
 */
DEFT_API deft_status deft_gather_update(float* acc_d, int64_t n_g, const int64_t* idx_d, int64_t count,
                                        float* val_d, void* stream);

/*
 * Algorithm 1 around the sparsifier, for runs with several workers (lines 7-10 and Eq. 2).  The
 * collectives themselves (all-gather of the index lists, all-reduce of the values) are the caller's;
 * these calls do what happens on the device before and after them.
 *
 * deft_index_union — line 7 after the all-gather: the sorted set of the indices in idx_d[0, count)
 * (any order, duplicates allowed, each in [0, n_g); others are ignored).  Writes the first out_cap of
 * them to union_d in ascending order and their number to *count_d (DEVICE int64; may exceed out_cap).
 * DEFT's workers own disjoint layers, so their lists never overlap and the union has exactly sum k_l
 * entries; with Top-k on every worker it is the place where the build-up of Section 1 shows.
 * ws_d: deft_union_workspace_bytes(n_g) bytes (a bitmap of n_g bits and one counter per 32768 of them),
 * 256-byte aligned.  Errors: INVALID_ARG, CAPACITY (workspace), CUDA.
 *
 * deft_sum_into — dst_d[i] += src_d[i] for i < count, one fp32 round-to-nearest add each: the sum of
 * line 9 where all workers live on one device (otherwise the all-reduce forms it).
 * deft_average — sum_d[i] /= n_workers, one fp32 division each: line 9's 1/n after the sum.
 *
 * deft_vector_norm — the L2 norm of x_d[0, n) in fp64 (Eq. 2: a worker's error is the norm of its
 * residual), computed like one layer's norm in deft_layer_norms; nothing is written to x_d.
 * norm_d: DEVICE double.  ws_d: deft_vector_norm_workspace_bytes(n) bytes, 256-byte aligned.
 */
/* Eq. 2 (host): the mean of the workers' errors (their residuals' norms), added in rank order. */
DEFT_API deft_status deft_error_eq2(const double* worker_error_h, int32_t n_workers, double* error_out);

DEFT_API size_t deft_union_workspace_bytes(int64_t n_g);
DEFT_API deft_status deft_index_union(const int64_t* idx_d, int64_t count, int64_t n_g, int64_t* union_d,
                                      int64_t out_cap, int64_t* count_d, void* ws_d, size_t ws_bytes, void* stream);
DEFT_API deft_status deft_sum_into(float* dst_d, const float* src_d, int64_t count, void* stream);
DEFT_API deft_status deft_average(float* sum_d, int64_t count, int32_t n_workers, void* stream);
DEFT_API size_t deft_vector_norm_workspace_bytes(int64_t n);
DEFT_API deft_status deft_vector_norm(const float* x_d, int64_t n, double* norm_d, void* ws_d, size_t ws_bytes,
                                      void* stream);

/*
 * Residual update — Algorithm 1 lines 11-12: acc[idx[j]] = +0.0f for j < count; the
 * buffer is then the next step's local error.  Indices must be distinct and < n_g.
 *   idx_d[count] DEVICE.  count may be 0.  Errors: INVALID_ARG, CUDA.
 */
DEFT_API deft_status deft_residual_update(float* acc_d, int64_t n_g, const int64_t* idx_d, int64_t count,
                                 void* stream);

/*
 * Conventional Top-k over the whole vector — the comparison sparsifier of Sections 1
 * and 3.1: the k entries of largest magnitude among acc_d[0..n), same ordering, tie
 * rule and output format as deft_select (it is deft_select with a single layer).
 * Errors: INVALID_ARG (k outside [1, n], n > DEFT_MAX_LAYER_ELEMS), CAPACITY, CUDA.
 */
DEFT_API deft_status deft_topk_baseline(const float* acc_d, int64_t n, int64_t k, float* val_d,
                               int64_t* idx_d, void* ws_d, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DEFT_H_ */
