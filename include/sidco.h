/*
 * sidco.h - C ABI of the B200 (sm_100a) SIDCo gradient sparsifier.
 *
 * The library implements one call of the paper's compressor (Algorithm 1,
 * function Sparsify, wrapped in error compensation) over a flattened model
 * gradient that is split into contiguous segments (layers).  Every step runs
 * in CUDA kernels of this library; there is no CPU fallback.
 *
 * Conventions
 *   - "device" pointers refer to memory of the CUDA device that is current
 *     when the function is called; "host" pointers are ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Functions return 0 on success, a negative SIDCO_E_* code for an argument
 *     error found on the host before anything was enqueued, or a positive
 *     cudaError_t value if a CUDA runtime call failed.
 *   - Device-side conditions never trap.  They set bits in a per-segment status
 *     word that sidco_get_debug() returns (SIDCO_ST_*).
 *   - The caller owns every buffer it passes in.  The library owns, per
 *     `residual` pointer (the persistent identity of one model's error
 *     compensation memory): the tile table derived from `seg_offsets`, a
 *     scratch workspace (sidco_workspace_bytes) and the stage-adaptation state.
 *   - One call per `residual` may be in flight at a time; calls for different
 *     `residual` pointers are independent.
 */
#ifndef SIDCO_H_
#define SIDCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Sparsity-inducing distribution of the first stage and the family of the
 * later stages (Section 2.4, paragraph after Corollary 2.1):
 * exponential -> exponential, gamma -> generalised Pareto, GPD -> GPD. */
#define SIDCO_SID_EXP   0
#define SIDCO_SID_GAMMA 1
#define SIDCO_SID_GPD   2

#define SIDCO_MAX_STAGES 8      /* hard upper limit on |max_stages| */

/* argument errors (returned before any work is enqueued) */
#define SIDCO_E_NULL        (-1)   /* a required pointer is NULL */
#define SIDCO_E_SEGMENTS    (-2)   /* n_segs < 1, offsets[0] != 0, offsets decreasing, or d too large */
#define SIDCO_E_DELTA       (-3)   /* delta not in (0, 1) */
#define SIDCO_E_SID         (-4)   /* unknown sid_type */
#define SIDCO_E_STAGES      (-5)   /* max_stages == 0 or |max_stages| > SIDCO_MAX_STAGES */
#define SIDCO_E_PARAMS      (-6)   /* sidco_set_params: value out of range */
#define SIDCO_E_UNKNOWN_KEY (-7)   /* no state exists for this residual pointer */
#define SIDCO_E_WORKSPACE   (-8)   /* caller-provided workspace too small or misaligned */
#define SIDCO_E_ALIAS       (-9)   /* grad and residual overlap */
#define SIDCO_E_SIZE        (-10)  /* size beyond the limit of this entry point */
#define SIDCO_E_CAPTURE     (-11)  /* the call would have to allocate or upload tables while `stream` is capturing */
#define SIDCO_E_UNSUPPORTED (-12)  /* the function needs a build of the library with another compile-time switch */

/* per-segment status bits */
#define SIDCO_ST_NONFINITE  1   /* a magnitude was NaN/Inf: nothing is selected in the segment */
#define SIDCO_ST_DEGENERATE 2   /* a fit took one of its degenerate-case rules */
#define SIDCO_ST_ALL_ZERO   4   /* every magnitude is zero: nothing is selected */
#define SIDCO_ST_TIMEOUT    8   /* a bounded wait inside the kernel ran out; results are invalid */
#define SIDCO_ST_BOUNDS     16  /* -DSIDCO_BOUNDS_CHECK builds only: an index fell outside its buffer and the access
                                   was skipped; results are invalid */

typedef struct sidco_seg_debug {
    int32_t M_used;                       /* stages used by the last call (after the cap for delta) */
    int32_t M_next;                       /* stage count the next adaptive call starts from */
    int32_t status;                       /* SIDCO_ST_* bits of the last call */
    int32_t calls;                        /* adaptive calls seen so far */
    int64_t k_sum;                        /* sum of k_hat since the last adaptation point */
    double  eta[SIDCO_MAX_STAGES];        /* eta_1 .. eta_{M_used} */
    int32_t k_stage[SIDCO_MAX_STAGES];    /* #{|x| > eta_m} for m < M_used, #{|x| >= eta_M} for the last */
} sidco_seg_debug;

/*
 * sidco_compress - one iteration of the sparsifier on device buffers.
 *
 * Computes, for every segment s = [seg_offsets[s], seg_offsets[s+1]) independently:
 *   1. error compensation  acc_j = grad_j + residual_j                    (one fp32 add; appendix on
 *      gradient distributions, memory-based compression);
 *   2. the threshold eta_M by multi-stage fitting (Section 2.4, Lemma 2, Corollary 2.1) with the first
 *      stage from Corollary 1.1 (EXP), 1.2 (GAMMA) or 1.3 (GPD); the first-stage ratio is delta_1 (0.25 by
 *      default), every non-final stage keeps delta_1 and the last stage takes delta / delta_1^(M-1);
 *   3. threshold sparsification (Section 2.3): K = { j : |acc_j| >= eta_M };
 *   4. residual_j <- +0.0f for j in K and acc_j otherwise;
 *   5. if max_stages > 0, stage adaptation (Algorithm 1, Adapt_Stages) every Q calls.
 *
 * grad        device, float[d], read only, d = seg_offsets[n_segs].
 * residual    device, float[d], in/out.  Must not overlap grad.
 * seg_offsets HOST, int64[n_segs + 1], seg_offsets[0] = 0, non-decreasing (empty segments allowed),
 *             d <= 2^31 - 2^16.  Read during the call only.
 * n_segs      >= 1.
 * delta       target ratio k/d, 0 < delta < 1 (the float value is used as is, widened to double).
 * sid_type    SIDCO_SID_*.
 * max_stages  > 0: adaptive, M starts at 1 and moves within [1, max_stages];
 *             < 0: fixed M = -max_stages, no adaptation.  M is additionally capped so that the last
 *             stage's ratio stays below one.
 * out_idx     device, int32, capacity >= d.  Flat indices of the survivors, strictly ascending.
 * out_val     device, float, capacity >= d.  out_val[t] = acc[out_idx[t]], bit exact.
 * out_k       device, int32[n_segs + 1].  out_k[s] = survivors of segment s, out_k[n_segs] = total;
 *             segment s occupies positions [sum_{t<s} out_k[t], +out_k[s]) of out_idx/out_val.
 * stream      all device work is enqueued here; the call does not synchronise, except that the first
 *             call for a residual pointer (or for a new segment table) allocates and uploads tables.
 *             Every later call enqueues one kernel whose arguments depend only on the arguments given
 *             here (the call counter and the "residual is empty" mark live in the workspace and are
 *             advanced by the kernel), so such calls may be recorded by stream capture and replayed as a
 *             CUDA graph.  A call that would have to allocate or upload while `stream` is capturing
 *             returns SIDCO_E_CAPTURE and enqueues nothing.
 *
 * 32-byte aligned grad and residual take the vectorised path; other alignments are handled with scalar
 * accesses.
 */
int sidco_compress(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs,
                   float delta, int sid_type, int max_stages,
                   int32_t* out_idx, float* out_val, int32_t* out_k, void* stream);

/*
 * sidco_compress_bf16 - sidco_compress with the gradient stored as bf16 (the error-compensation memory, the
 * thresholds and the outputs stay fp32).  Step 1 becomes acc_j = (float)grad_j + residual_j, the bf16 value
 * widened exactly; everything after it is unchanged.  This is the mixed-precision variant of the paper's
 * synthetic-tensor micro-benchmark (appendix, compression overhead on tensors of 0.26 to 260 million elements)
 * for frameworks that keep gradients in bf16: the call reads 2 bytes per gradient element instead of 4.
 * grad_bf16   device, uint16[d] holding bf16 bit patterns, read only; 16-byte alignment (together with a
 *             32-byte aligned residual) gives the vectorised path.
 * State is keyed by `residual` as in sidco_compress, and the two entry points may be mixed on one residual.
 */
int sidco_compress_bf16(const uint16_t* grad_bf16, float* residual, const int64_t* seg_offsets, int n_segs,
                        float delta, int sid_type, int max_stages,
                        int32_t* out_idx, float* out_val, int32_t* out_k, void* stream);

/*
 * sidco_compress_host - the same operation with HOST buffers (pinned memory gives full copy speed).
 * Copies grad and residual to device staging buffers owned by the library, runs sidco_compress,
 * copies residual, out_k and the first out_k[n_segs] entries of out_idx/out_val back, and
 * synchronises `stream` before returning.  State is keyed by the host `residual` pointer.
 * out_idx/out_val need capacity >= d on the host as well.
 */
int sidco_compress_host(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs,
                        float delta, int sid_type, int max_stages,
                        int32_t* out_idx, float* out_val, int32_t* out_k, void* stream);

/*
 * sidco_compress_static - sidco_compress for callers that must not allocate device memory.
 *
 * (The paper has no counterpart to this entry point; it exists for integration reasons only.)
 *
 * Some callers cannot tolerate a cudaMalloc: code running while a CUDA graph is being captured, code inside
 * a framework whose caching allocator owns all device memory and treats outside allocations as leaks or
 * fragmentation, and latency-critical loops where an allocation's implicit device synchronisation is
 * unacceptable.  sidco_compress allocates its scratch workspace on the first call for a residual pointer.
 * This variant never calls cudaMalloc, cudaFree or any allocating routine: its workspace is a fixed
 * 18 MiB array in device memory that is part of the library image, so every GPU on which the library is
 * loaded holds those 18 MiB until the process exits, whether or not this function is ever called.
 *
 * Same arguments, results and error codes as sidco_compress, with these differences:
 *   - limits: d = seg_offsets[n_segs] <= SIDCO_STATIC_MAX_ELEMS and n_segs <= SIDCO_STATIC_MAX_SEGS;
 *     larger inputs are rejected with SIDCO_E_SIZE before anything is enqueued;
 *   - there is one workspace per device, shared by every call: two calls that overlap on the GPU (for
 *     example on different streams) race on it and corrupt each other; serialise them;
 *   - the workspace keeps the contents the previous call left.  The counters and records that must start
 *     at zero are cleared on `stream` together with the table upload, i.e. on the first call for a
 *     (residual pointer, segment table) pair; after that they carry on from call to call.  The
 *     stage-adaptation state lives in the workspace too and
 *     belongs to the last (residual pointer, segment table) pair: calling with a different pair rebuilds
 *     the tables, resets M to 1 and synchronises `stream` once (while `stream` is capturing such a call
 *     returns SIDCO_E_CAPTURE and enqueues nothing).  The pair is recognised by the pointer's value: a
 *     residual buffer that is freed and allocated again at the same address, used with the same segment
 *     table, inherits the old M and counts; the only way to start over is a call with a different pair;
 *   - the first call on a device looks up the device address of the array (cudaGetSymbolAddress) and
 *     uploads tables; make that first call before any stream capture begins;
 *   - the debug, state and workspace helpers below do not see this workspace.
 */
#define SIDCO_STATIC_MAX_ELEMS 1048576
#define SIDCO_STATIC_MAX_SEGS  256
int sidco_compress_static(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs,
                          float delta, int sid_type, int max_stages,
                          int32_t* out_idx, float* out_val, int32_t* out_k, void* stream);

/*
 * sidco_aggregate - dense mean of N workers' sparse gradients.
 *
 * The step that follows the sparsifier in the paper's sparsified distributed synchronous SGD (appendix,
 * algorithm box "Sparsified Distributed Synchronous SGD", line "Collective-Comm"):
 *     G = (1/N) * sum_{n=1..N} Sparsify(g_n, delta).
 * The exchange itself (an all-gather of every worker's out_idx / out_val / count) is done by the caller;
 * this call turns the gathered lists, which lie in local device memory, into the dense vector.
 *
 * idx_all    device, int32[n_workers * stride]: worker n's indices at idx_all + n * stride, strictly
 *            ascending, each in [0, d); entries beyond counts[n] are padding and are not read.
 * val_all    device, float[n_workers * stride], same layout.
 * counts     device, int32[n_workers]: entries of each worker's list (what the worker's out_k[n_segs] said).
 * n_workers  1 .. SIDCO_AGG_MAX_WORKERS.
 * stride     elements between consecutive workers' lists (>= every count).
 * d          length of the dense vector, <= 2^31 - 2^16.
 * out_dense  device, float[d], written in full: out[j] = (float)((v_1[j] + ... + v_N[j]) / N), the sum taken
 *            in fp64 over the workers that sent position j, in worker order, and +0.0f where nobody did.
 *            32-byte alignment gives the vectorised path.
 * status     device, int32, optional (NULL to ignore): cleared on `stream`, then OR-ed with SIDCO_AGG_ST_COUNT
 *            if a count lay outside [0, stride] (it is clipped) and SIDCO_AGG_ST_ORDER if an index was met
 *            where an ascending list cannot have it (that entry is skipped; nothing is written outside
 *            out_dense either way).
 * stream     everything is enqueued here (one kernel, plus the 4-byte clear of `status`); no synchronisation,
 *            no allocation.
 */
#define SIDCO_AGG_MAX_WORKERS 64
#define SIDCO_AGG_ST_COUNT 1
#define SIDCO_AGG_ST_ORDER 2
int sidco_aggregate(const int32_t* idx_all, const float* val_all, const int32_t* counts, int n_workers,
                    int64_t stride, int64_t d, float* out_dense, int32_t* status, void* stream);

/*
 * Reference points: the two compressors the paper compares its method with (Section 1 and Fig. 1), on the same
 * inputs and with the same error-compensation wrapper, so that speed and achieved ratio can be compared on one
 * machine.  Whole-vector selection, as in the paper's micro-benchmark.  Both compute acc = grad + residual
 * (stored over residual), write the selected (index, value) pairs in ascending index order, set the selected
 * residual entries to +0.0f, and write the number selected to out_k[0].  Magnitudes are compared as the bit
 * patterns of |acc| (finite < infinite < NaN).
 *
 * sidco_topk - exact Top-k: the k largest magnitudes; among equal magnitudes the lower index wins.
 * sidco_dgc  - sampled threshold (Deep Gradient Compression style): the threshold is the ceil(delta * n_sample)-th
 *              largest magnitude (at least the largest) among acc[sample_idx[0 .. n_sample)]; every element of the
 *              vector whose magnitude reaches it is selected.  The sample positions are the caller's (any
 *              generator; a position outside [0, d) counts as a zero).
 *
 * grad, residual, out_idx, out_val   device, as in sidco_compress (capacity d).
 * out_k       device, int32[1].
 * sample_idx  device, int32[n_sample].
 * workspace   device, 256-byte aligned, at least sidco_reference_workspace_bytes(d, n_sample) bytes (n_sample = 0
 *             for sidco_topk); caller-owned, no state is kept in it between calls.
 * stream      everything is enqueued here (about ten kernels); no synchronisation, no allocation.
 */
size_t sidco_reference_workspace_bytes(int64_t d, int64_t n_sample);
int sidco_topk(const float* grad, float* residual, int64_t d, int64_t k, int32_t* out_idx, float* out_val,
               int32_t* out_k, void* workspace, size_t workspace_bytes, void* stream);
int sidco_dgc(const float* grad, float* residual, int64_t d, float delta, const int32_t* sample_idx,
              int64_t n_sample, int32_t* out_idx, float* out_val, int32_t* out_k, void* workspace,
              size_t workspace_bytes, void* stream);

/* Bytes of device scratch one residual key needs for a vector of d elements in n_segs segments. */
size_t sidco_workspace_bytes(int64_t d, int n_segs);

/* Optional: let the library use caller-owned device memory (256-byte aligned, at least
 * sidco_workspace_bytes) as the workspace of `residual` instead of allocating its own.  Must be called
 * before the first sidco_compress for that residual; the memory must outlive the state. */
int sidco_set_workspace(const float* residual, void* device_ptr, size_t bytes);

/* Constants of Algorithm 1 for subsequent calls (defaults: the paper's experimental settings,
 * delta_1 = 0.25, eps_H = eps_L = 0.2, Q = 5).  0 < delta1 < 1, 0 <= eps < 1, Q >= 1. */
int sidco_set_params(double delta1, double eps_H, double eps_L, int Q);

/* Variants the paper describes and then replaces or leaves open, for subsequent calls (all 0 by default: the
 * method as the paper evaluates it).  They exist to quantify what the shortcuts cost in achieved ratio.
 *   gamma_exact        Corollary 1.2 without its two shortcuts: the shape is the maximum-likelihood estimate (the
 *                      root of the digamma equation in the corollary's proof, Newton's method on the device) and
 *                      the first-stage threshold is beta * P^{-1}(alpha, 1 - delta), the exact gamma quantile,
 *                      instead of the closed-form bound.  Costs tens of microseconds of serial fp64 per call.
 *   ratio_from_counts  the last stage of a multi-stage fit aims at the target count itself: its ratio is
 *                      k / k_hat_{M-1} (delta * n over the exceedances the stage before it left, at most 1) instead
 *                      of the nominal delta / delta_1^(M-1) (Section 2.4 only fixes the product of the ratios).
 *   adapt_reversed     Adapt_Stages (Algorithm 1) with the opposite sign: too many selected -> one stage more.
 */
int sidco_set_policy(int gamma_exact, int ratio_from_counts, int adapt_reversed);

/* Start over for `residual`: the adaptation state is forgotten (M back to 1, counters to 0) and the error
 * compensation memory is declared empty - the next sidco_compress on it takes the residual as all zeros
 * without reading it (and overwrites it), so the caller need not clear the buffer.  Synchronises the device. */
int sidco_reset_state(const float* residual);

/* The same reset enqueued on `stream` (one tiny kernel, no synchronisation): for callers that restart a
 * run without stalling the stream.  The next sidco_compress for `residual` must be issued after this call
 * returns; the mark that tells it not to read the residual lives in the workspace on the device and is
 * consumed by the first compress kernel that runs after the reset kernel on `stream`. */
int sidco_reset_state_async(const float* residual, void* stream);

/* Copy per-segment thresholds, counts, stage counts and status of the last call to host memory
 * (`out` has room for n_segs entries).  Synchronises the device; meant for tests and logging. */
int sidco_get_debug(const float* residual, sidco_seg_debug* out, int n_segs);

/* (Only in a build with -DSIDCO_PROFILE, see sidco_build_flags; the default build takes no device timestamps
 * and both functions below return SIDCO_E_UNSUPPORTED.)
 * Phase breakdown of the last call in microseconds, from device timestamps taken by the first CTA as it
 * moves from phase to phase (the other CTAs move on their own): us_out[0] error compensation + stage-1 statistics and fit, [1] stage-2 side-buffer
 * compaction and fit, [2] stages 3..M, [3] survivor staging + residual zeroing, [4] final placement and
 * adaptation, [5] whole kernel; then finer marks of that CTA alone: [6] its first sweep, [7] its arrivals
 * and fits after it, [8] its stage-2 sweep, [9] arrivals and fits after it, [10] arrivals and fits of the
 * last refit stage, [11] its survivor staging sweep.  us_out has room for 12 values.  Entries of phases
 * the call did not run are meaningless.  Synchronises the device; for profiling. */
int sidco_get_phase_times(const float* residual, double* us_out);

/* Per-CTA view of the last call, for load-balance studies: us_out[4*i + p] is the time (microseconds
 * after the kernel's first CTA started) at which CTA i finished its sweep of phase p (0 first sweep,
 * 1 stage-2 sweep, 2 last refit sweep, 3 survivor staging).  Writes at most max_ctas rows and returns
 * the number of rows written (>= 0) or an error code (< 0).  Synchronises the device. */
int sidco_get_cta_sweep_times(const float* residual, double* us_out, int max_ctas);

/* (Profile builds only.)  How the final selection of the last call went, per CTA: out[8*i + 0] 1 if the run's
 * survivors went through the shared-memory list, [1] candidate slots recorded, [2] chunks read by the warps,
 * [3] survivors of the run, [4] chunks of acc read a second time in full, [5] chunks of the run.  Returns the
 * number of rows written or an error code (< 0).  Synchronises the device. */
int sidco_get_cta_selection_info(const float* residual, int32_t* out, int max_ctas);

/* Checkpointing of the adaptation state (Algorithm 1 keeps M and the running k_hat sum across
 * iterations): host blobs of 3 int64 per segment (M, calls, k_sum).  Both synchronise the device. */
int sidco_state_save(const float* residual, int64_t* host_blob, int n_segs);
int sidco_state_load(const float* residual, const int64_t* host_blob, int n_segs);

/* Free everything the library holds for `residual` / for all keys.  Synchronises the device. */
int sidco_release(const float* residual);
int sidco_release_all(void);

/* Switches for tests; production code has no reason to call this.
 *   grid                  > 0: launch with at most this many CTAs (contexts created afterwards); 0: all the device
 *                         holds.  Starts from the environment variable SIDCO_GRID, if set.
 *   spec_enable           0: the sweeps record no candidate slots and the final selection re-reads acc in full;
 *                         2: candidate thresholds are set too high on purpose, so that the final selection finds
 *                         most of them unusable and takes its other routes (results are the same in every mode).
 *                         Starts from SIDCO_SPEC, if set.
 *   spin_limit            polls after which a bounded wait inside the kernel gives up and raises SIDCO_ST_TIMEOUT;
 *                         0 restores the default (about one second).
 *   drop_publication_seg  >= 0: the kernel withholds the published threshold words of this segment, so that the
 *                         CTAs waiting for them run into spin_limit (to exercise the time-out path without
 *                         harming the device); -1: off. */
int sidco_set_test_hooks(int grid, int spec_enable, long long spin_limit, int drop_publication_seg);

/* Compile-time switches this library was built with. */
#define SIDCO_BUILD_PROFILE      1   /* -DSIDCO_PROFILE: device timestamps at phase boundaries */
#define SIDCO_BUILD_BOUNDS_CHECK 2   /* -DSIDCO_BOUNDS_CHECK: every index into a caller or workspace buffer is
                                        range-checked before use; a bad one is skipped and reported in the status */
int sidco_build_flags(void);

/* Number of kernel launches the library has enqueued since it was loaded. */
int64_t sidco_launch_count(void);

const char* sidco_error_string(int code);
int sidco_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SIDCO_H_ */
