// Device code of the SIDCo sparsifier for sm_100a.
//
// One persistent cooperative kernel runs the whole call.  The flat vector is cut
// into chunks that never straddle a segment or a 1024-element window.  Every CTA
// (one per SM, 32 warps) owns one contiguous run of chunks for the whole call, so
// what it wrote in one phase (acc, side buffers) it re-reads itself in the next.
// Inside a run the warps pull chunks from a shared-memory queue and work on them
// without any block-level synchronisation: a chunk is loaded and reduced with warp
// shuffles by one warp.  A CTA moves from one phase to
// the next on its own: a run that needs a segment's threshold waits (bounded) on
// that segment's published word {call number, stages fitted, threshold}, which
// the run completing the segment's statistics stores.  There is no grid-wide
// barrier: for the final placement every run publishes its survivor count as a
// tagged word that the runs above it poll, and a segment's total count comes out
// of the atomic by which the last of its runs reports.
//
//   P1  acc = grad + residual (stored over residual) and the stage-1 statistics
//       of every chunk; the CTA whose run completes a segment sums the per-chunk
//       partials in chunk order and fits eta_1 (Corollaries 1.1-1.3).  For
//       single-stage segments the sweep also notes, in shared memory, the place of
//       every 8-element slot of a lane in which some |x| >= tau, tau being 0.85
//       times the segment's final threshold of the previous call (without one --
//       the first call on a fresh residual -- 0.8 times the exponential-form
//       threshold of the chunk's own mean, remembered per window).  If the new
//       threshold turns out >= tau (checked per segment or window) the final
//       selection compares only the noted slots; otherwise it reads the chunks
//       concerned again, so the result never depends on tau
//   P3  (segments with M >= 2) statistics of the shifted peaks |x| - eta_1 over
//       the exceedances |x| > eta_1 (Lemma 2 / Corollary 2.1) and fit of eta_2.
//       Two-stage segments note candidate slots here (as P1 does for one stage);
//       segments with more stages copy their exceedances into the chunk's side
//       region, dense and in index order (positions from two packed warp scans,
//       one slot row at a time through a shared-memory staging row, 16-byte
//       stores), together with a 32-bit mask per lane that says which of its 32
//       elements they are
//   P4  (m = 3..M) statistics of side-region entries above eta_{m-1}; fit eta_m
//   P5a survivors |x| >= eta_M.  The usual way stays in shared memory: one thread
//       per noted slot compares it with the final threshold (the first noted slots
//       have their values in shared memory already, copied asynchronously behind
//       the fits), the few chunks without usable candidates are added slot by slot
//       or read by the warps (three or more stages: from the side region), and all
//       survivors of the run end up in one unordered list that is put in index
//       order by counting per 1024-element window and ranking inside a window.
//       Nothing is modified before the list is known to fit; otherwise (a large
//       fraction selected) the warps stage every chunk's survivors in order in the
//       chunk's staging region
//   P5b base of the run = published counts of the runs below; survivors copied
//       to their final ascending positions (from the ordered list, or from the
//       staging regions through a block scan of the chunk counts) and zeroed in
//       the residual; per-segment counts and stage adaptation (Algorithm 1,
//       Adapt_Stages) by the thread whose report completes the segment
//
// Reductions are deterministic and independent of the grid: per-lane sequential
// accumulation in a fixed order, a fixed shuffle tree per chunk, and a fixed-order
// sum of the per-chunk partials of a segment.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

// Device timestamps at phase boundaries (sidco_get_phase_times, sidco_get_cta_sweep_times) exist only in a
// build with -DSIDCO_PROFILE; the default build carries none of them.
#ifdef SIDCO_PROFILE
#define SIDCO_STAMP(...) do { __VA_ARGS__; } while (0)
#else
#define SIDCO_STAMP(...) do { } while (0)
#endif

namespace sidco {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kChunk = 1024;                      // window: elements per full chunk (one warp)
constexpr int kComp = 8;                          // elements per slot: one 32-byte access per lane
constexpr int kSlots = kChunk / (32 * kComp);     // slots per lane per chunk (4)
constexpr int kSmallSeg = 256;                    // segments of <= 256 chunks are summed by one warp
constexpr int kGiantSeg = 4096;                   // segments of more chunks are summed in two levels:
constexpr int kTile = 1024;                       // tiles of this many chunks first (by the run that completes a tile)
constexpr int kSegCache = 256;                    // segments of a CTA run whose table entries sit in shared memory
constexpr int kOutCache = 2048;                   // survivors of a run the shared-memory selection can hold
constexpr int kSlotCap = 3072;                    // candidate slots (8 elements of one lane) a run can note
constexpr int kSlotPre = 1280;                    // the first of them have their values copied to shared memory ahead
constexpr int kWinCap = 2048;                     // 1024-element windows of a run the shared-memory selection covers
constexpr int kScWin = 1024;                      // ... and the windows a run may have for warps to calibrate candidate thresholds themselves
constexpr float kScRatio = 0.8f;                  // a warp's own candidate threshold: this fraction of the exponential estimate from its last chunk
static_assert(kSlotPre * kComp >= 2 * kOutCache, "the ordered survivors reuse the candidate values' space");
constexpr float kSpecRatio = 0.85f;                // candidate threshold = this fraction of the last eta
constexpr int kMaxStages = 8;
constexpr unsigned kFull = 0xffffffffu;
constexpr long long kSpinLimit = 1ll << 22;       // default bound of the waits: ~1 s with the back-off below
static_assert(kWarps == 32, "block_tree and the scans assume 32 warps per CTA");

enum { kSidExp = 0, kSidGamma = 1, kSidGpd = 2 };
enum { kStNonFinite = 1, kStDegenerate = 2, kStAllZero = 4, kStTimeout = 8 };

struct SegDev {
    double eta[kMaxStages];
    int32_t k_stage[kMaxStages];
    float thr_gt;        // largest fp32 <= eta of the newest stage: (|x| > thr_gt) == (|x| > eta)
    float thr_ge;        // smallest fp32 >= eta_M:                  (|x| >= thr_ge) == (|x| >= eta_M)
    int32_t M_eff;       // stages used by this call
    int32_t status;
    int32_t arrived;     // CTA runs of this segment finished in the current phase (self-resetting)
    int32_t k_acc;       // survivors counted so far in this call by runs that keep no shared-memory count for the
                         // segment (integer atomics; self-resetting)
    int32_t M;           // adaptation state: stage count for the next adaptive call
    int32_t calls;
    long long k_sum;
    // Published with release semantics by the thread that fits a stage and polled with acquire semantics by
    // the runs that wait for it.  Low word: call_id * 16 + number of stages fitted so far in that call.  High
    // word: the fp32 compare threshold of the newest stage, thr_ge if that stage is the segment's last,
    // thr_gt otherwise, so that a waiting thread has it with the same load that tells it the stage is fitted.
    unsigned long long pub;
    // Survivor count of the call and the runs that have reported theirs: each run adds (count << 32) + 1 with one
    // atomic, and the run whose addition completes the arrivals has the segment's total in the value returned,
    // writes out_k and does the adaptation step (self-resetting).
    unsigned long long k_arr;
    float spec_thr;      // candidate threshold for the next call's first sweep (<= 0: none), see P1
    int32_t pad;
};

struct Control {
    unsigned count;      // CTAs that have finished, over all calls since the workspace was set up (never reset by
                         // the kernel): the one that brings it to (seq + 1) * G closes the call
    unsigned seq;        // calls completed since then: call number seq + 1 tags SegDev::pub and Args::cta_pub.
                         // Advanced by the kernel itself, so that a launch's arguments do not change from call to
                         // call (a recorded launch can be replayed)
    int timeout;         // set when a bounded wait ran out
    int residual_is_zero;  // the next call takes the residual's contents as zeros and does not read them
                         // (set by a state reset, cleared by the call)
    int bounds;          // -DSIDCO_BOUNDS_CHECK builds: an index fell outside its buffer (the access was skipped)
    int pad;
    unsigned long long t_ns[16];  // globaltimer at phase boundaries, written by CTA 0 (diagnostics)
};

struct Args {
    const float* grad;           // fp32 gradient, or bf16 (two bytes per element) if grad_bf16 is set
    float* residual;
    int32_t* out_idx;
    float* out_val;
    int32_t* out_k;
    // tables (read only during the call)
    const int32_t* chunk_start;  // [C + 1]
    const int32_t* chunk_seg;    // [C]
    const int32_t* seg_chunk0;   // [S + 1]
    const int32_t* seg_n;        // [S]
    const int32_t* seg_runs;     // [S] number of CTA runs that hold chunks of the segment
    const int32_t* seg_tile0;    // [S + 1] first tile of the segment (segments of more than kGiantSeg chunks have tiles)
    int32_t* tile_arr;           // [tiles] chunks of the tile whose partials are in (self-resetting)
    double* tile_part;           // [tiles][3] sums over the tile's chunk partials
    const int4* cta_desc;        // [G] {first chunk, one past last chunk, first segment, segments} of the run
    // scratch
    double* part;                // [C][3] per-chunk partial sums
    int32_t* part_n;             // [C] per-chunk partial counts
    int32_t* chunk_cnt;          // [C] final survivors staged for the chunk
    float* side_val;             // [C][kChunk] side regions: the kept values of chunk c, dense, in index order
    unsigned* side_mask;         // [C][32] per lane: which of its elements (bit 8 j + component) the side region holds
    int32_t* side_cnt;           // [C] entries in the chunk's side region
    int32_t* stage_idx;          // [d]
    float* stage_val;            // [d]
    unsigned long long* cta_pub; // [G] {call number, survivors of the run}: published once the run's selection is done
    int32_t* cta_dir;            // [G] 1: this CTA's next first sweep runs over descending chunks
    unsigned long long* cta_ns;  // [G][4] globaltimer when the CTA finished its P1, P3, last P4, P5a sweep
    int* cta_dbg;                // [G][8] profile builds: how the final selection of the run went
    int32_t* slot_spill_e;       // [d / 8 + G] candidate slots beyond what shared memory holds: first element ...
    unsigned char* slot_spill_seg;   // ... and segment of the run (a run's entries start at its first element / 8)
    SegDev* seg;                 // [S]
    Control* ctl;
    // scalars
    double delta, delta1, eps_H, eps_L;
    // log(ratio) and log(1 / ratio) of the stage ratios, from the host: slot 0 is delta_1 (every stage but the
    // last), slot M the ratio of the last stage of an M-stage schedule (delta for M = 1)
    double ln_ratio[kMaxStages + 1], ln_inv_ratio[kMaxStages + 1];
    int Q, sid, max_stages;
    int C, S, G;
    int d;                       // elements of the vector
    int vec_ok;                  // grad and residual are 32-byte aligned (256-bit accesses)
    int spec_enable;             // candidate pre-selection in the first sweep (see P1)
    int grad_bf16;               // grad points to bf16 values, widened exactly to fp32 before the add
    // variants the paper describes and replaces (sidco_set_policy; all zero: the method as evaluated)
    int pol_gamma_exact;         // Corollary 1.2 with the maximum-likelihood shape and the exact quantile
    int pol_ratio_counts;        // last stage's ratio = target count / exceedances the stage before it left
    int pol_adapt_rev;           // Adapt_Stages with the opposite sign
    long long spin_limit;        // polls after which a bounded wait gives up (kSpinLimit unless a test shortens it)
    int drop_pub_seg;            // test hook: the published words of this segment are withheld (-1: none), so that
                                 // the runs waiting for them run into the bound
};

// ----------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------

// Range check of an index into a caller or workspace buffer.  Only a build with -DSIDCO_BOUNDS_CHECK checks
// anything (the stand-in for an external memory checker): a bad index is recorded in the control block and the
// access is skipped.  In the product build this is the constant true.
#ifdef SIDCO_BOUNDS_CHECK
#define SIDCO_IN_RANGE(A, i, n) sidco::in_range_checked((A), (long long)(i), (long long)(n))
#else
#define SIDCO_IN_RANGE(A, i, n) true
#endif

__device__ __forceinline__ bool in_range_checked(const Args& A, long long i, long long n);

__device__ __forceinline__ int ld_cg(const int* p) { return __ldcg(p); }
__device__ __forceinline__ float ld_cg(const float* p) { return __ldcg(p); }
__device__ __forceinline__ double ld_cg(const double* p) { return __ldcg(p); }
__device__ __forceinline__ unsigned ld_cg(const unsigned* p) { return __ldcg(p); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ int ld_volatile(const int* p) {
    return *reinterpret_cast<const volatile int*>(p);
}

__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Arrival counter update whose returned value, if it shows that every other run has arrived, also makes
// their earlier (fenced) stores visible to this thread's later loads.
__device__ __forceinline__ int atom_add_acquire(int* p, int v) {
    int old;
    asm volatile("atom.acquire.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ bool in_range_checked(const Args& A, long long i, long long n) {
    if (i >= 0 && i < n) return true;
    atomicOr(&A.ctl->bounds, 1);
    return false;
}

// Single-thread wait until segment `sg` has `need` stages fitted in call `call_id` (bounded).  Returns the
// threshold published with that stage.  Only runs holding chunks of the segment wait for it, and the next
// stage cannot be fitted before they have swept those chunks, so the word read is the one of stage `need`.
__device__ __forceinline__ float wait_ready_thread(const Args& A, unsigned call_id, const SegDev* sg, int need) {
    const unsigned target = call_id * 16u + (unsigned)need;
    long long spins = 0;
    unsigned long long w;
    // (polled with plain strong loads: the word carries the threshold itself; a reader that goes on to load
    // eta, stored before a non-last stage's word and released with it, orders that load with a fence)
    while ((int)((unsigned)(w = ld_relaxed_u64(&sg->pub)) - target) < 0) {     // wrap-safe
        // (the time-out flag is looked at now and then only: a second dependent load in every round would
        // double the time it takes to notice the word)
        if ((++spins & 15) == 0 && ld_volatile(&A.ctl->timeout)) break;
        if (spins > A.spin_limit) { atomicExch(&A.ctl->timeout, 1); break; }
        __nanosleep(spins < 16 ? 20 : 100);
    }
    return __uint_as_float((unsigned)(w >> 32));
}

// Warp-level wait until segment `sg` has `need` stages fitted in call `call_id` (bounded).
__device__ __forceinline__ float wait_ready(const Args& A, unsigned call_id, const SegDev* sg, int need) {
    float thr = 0.0f;
    if ((threadIdx.x & 31) == 0) thr = wait_ready_thread(A, call_id, sg, need);
    return __shfl_sync(kFull, thr, 0);
}

struct Sums { double a, b; int n; };

__device__ __forceinline__ Sums warp_tree(double a, double b, int n) {
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_down_sync(kFull, a, o);
        b += __shfl_down_sync(kFull, b, o);
        n += __shfl_down_sync(kFull, n, o);
    }
    return Sums{a, b, n};
}

// The same tree over the sums a sweep of family SID needs: `b` only where a second moment (GPD) is kept, the
// count by a warp reduction (integer addition has no order to fix).  Result valid in lane 0.
template <bool WithB>
__device__ __forceinline__ Sums chunk_tree(double a, double b, int n) {
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_down_sync(kFull, a, o);
        if (WithB) b += __shfl_down_sync(kFull, b, o);
    }
    return Sums{a, WithB ? b : 0.0, (int)__reduce_add_sync(kFull, n)};
}

// Block-wide sums with a fixed tree (warp trees, then one warp over the 32 warp results);
// result valid in thread 0.
__device__ __forceinline__ Sums block_tree(double a, double b, int n, double (*sm)[3]) {
    Sums w = warp_tree(a, b, n);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();                       // previous use of sm is over
    if (lane == 0) { sm[warp][0] = w.a; sm[warp][1] = w.b; sm[warp][2] = (double)w.n; }
    __syncthreads();
    Sums r{0.0, 0.0, 0};
    if (warp == 0) {
        double x = sm[lane][0], y = sm[lane][1], z = sm[lane][2];
        #pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            x += __shfl_down_sync(kFull, x, o);
            y += __shfl_down_sync(kFull, y, o);
            z += __shfl_down_sync(kFull, z, o);
        }
        r.a = x; r.b = y; r.n = (int)z;
    }
    return r;
}

// Block-wide exclusive prefix sum of one int per thread (thread order); `total` is the block's sum.
// `sm` holds one int per warp and may be reused after the call returns.
__device__ __forceinline__ int block_exscan(int x, int* sm, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = x;
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                       // previous use of sm is over
    if (lane == 31) sm[warp] = incl;
    __syncthreads();
    int w = sm[lane];                      // every warp scans the 32 warp sums itself
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, w, o);
        if (lane >= o) w += t;
    }
    total = __shfl_sync(kFull, w, 31);
    const int warp_incl = __shfl_sync(kFull, w, warp);
    return warp_incl - sm[warp] + incl - x;
}

// The same for one group of kFitGroupWarps warps (warps g * kFitGroupWarps ...), the groups working
// independently: a group meets at named barrier 1 + g.  Result valid in the group's first thread.
constexpr int kFitGroupWarps = 12;
constexpr int kFitGroups = 2;            // the remaining warps fit small segments meanwhile
__device__ __forceinline__ Sums group_tree(double a, double b, int n, double (*sm)[3], int g) {
    Sums w = warp_tree(a, b, n);
    const int lane = threadIdx.x & 31, wg = (threadIdx.x >> 5) - g * kFitGroupWarps;
    asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(32 * kFitGroupWarps) : "memory");   // previous use of sm is over
    if (lane == 0) { sm[wg][0] = w.a; sm[wg][1] = w.b; sm[wg][2] = (double)w.n; }
    asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "r"(32 * kFitGroupWarps) : "memory");
    Sums r{0.0, 0.0, 0};
    if (wg == 0) {
        const bool in = lane < kFitGroupWarps;
        double x = in ? sm[lane][0] : 0.0, y = in ? sm[lane][1] : 0.0, z = in ? sm[lane][2] : 0.0;
        #pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            x += __shfl_down_sync(kFull, x, o);
            y += __shfl_down_sync(kFull, y, o);
            z += __shfl_down_sync(kFull, z, o);
        }
        r.a = x; r.b = y; r.n = (int)z;
    }
    return r;
}

// ----------------------------------------------------------------------------
// closed-form fits (one thread)
// ----------------------------------------------------------------------------

// Largest M with delta1^(M-1) > delta: more stages would leave the last ratio >= 1.
__device__ inline int stage_cap(double delta, double delta1) {
    int M = 1;
    double p = 1.0;
    for (;;) {
        p *= delta1;
        if (!(p > delta) || M >= 64) return M;
        ++M;
    }
}

// Stage count of a segment for this call: from the adaptation state the previous call left (or the
// fixed count), capped so that the last stage's ratio stays below one.  Stable during a call.
__device__ __forceinline__ int seg_stages(const Args& A, int seg, int cap) {
    int M;
    if (A.max_stages > 0) {
        M = A.seg[seg].M < 1 ? 1 : A.seg[seg].M;
        if (M > A.max_stages) M = A.max_stages;
    } else {
        M = -A.max_stages;
    }
    return M < cap ? M : cap;
}

// Tail ratio of stage m (0-based) out of M: delta_1 for every non-final stage, the rest for the last.
__host__ __device__ inline double stage_ratio(double delta, double delta1, int M, int m) {
    if (M == 1) return delta;
    if (m < M - 1) return delta1;
    double p = 1.0;
    for (int i = 0; i < M - 1; ++i) p *= delta1;
    return delta / p;
}

// Logarithms of the stage ratios (Args::ln_ratio, Args::ln_inv_ratio): slot 0 is delta_1 (every stage but the
// last), slot M the ratio of the last stage of an M-stage schedule (delta for M = 1).
struct LnTab {
    const double* ln;       // [kMaxStages + 1] log(ratio)
    const double* ln_inv;   // [kMaxStages + 1] log(1 / ratio)
    unsigned call_id;       // number of this call (tags the published words)
};
__device__ __forceinline__ int ratio_slot(int M, int m) { return (M == 1 || m == M - 1) ? M : 0; }

// Corollary 1.3 / Lemma 2: moment-matched generalised Pareto quantile at the tail probability whose
// logarithms are given.  A variance at rounding-noise level (raw-moment form) is treated as zero: the
// formula's limit is `mean`.
__device__ inline double gpd_step(double mean, double var, double ln_ratio, double ln_inv_ratio, int& status) {
    if (!(var > 1e-12 * mean * mean)) { status |= kStDegenerate; return mean; }
    const double R = mean * mean / var;
    const double alpha = 0.5 * (1.0 - R);
    const double beta = 0.5 * mean * (R + 1.0);
    const double t = -alpha * ln_ratio;
    if (fabs(t) < 1e-12) return beta * ln_inv_ratio;
    return (beta / alpha) * expm1(t);
}

// Corollary 1.1 / 2.1.
__device__ inline double exp_step(double mean, double ln_inv_ratio) { return mean * ln_inv_ratio; }

// ---- special functions for the exact forms of Corollary 1.2 (policy pol_gamma_exact; one thread, fp64)

// psi(x) and psi'(x), x > 0: recurrence up to x >= 8, then the asymptotic series.
__device__ inline void digamma_trigamma(double x, double& psi, double& psi1) {
    double a0 = 0.0, a1 = 0.0;
    while (x < 8.0) {
        const double r = 1.0 / x;
        a0 -= r;
        a1 += r * r;
        x += 1.0;
    }
    const double r = 1.0 / x, f = r * r;
    psi = a0 + log(x) - 0.5 * r - f * (1.0 / 12 - f * (1.0 / 120 - f * (1.0 / 252 - f * (1.0 / 240 - f / 132))));
    psi1 = a1 + r + 0.5 * f + r * f * (1.0 / 6 - f * (1.0 / 30 - f * (1.0 / 42 - f / 30)));
}

// Maximum-likelihood gamma shape: the root of log(alpha) - psi(alpha) = s, Newton from the closed form.
__device__ inline double gamma_shape_mle(double s, double alpha) {
    for (int it = 0; it < 100; ++it) {
        double psi, psi1;
        digamma_trigamma(alpha, psi, psi1);
        const double f = log(alpha) - psi - s;
        double nw = alpha - f / (1.0 / alpha - psi1);
        if (!(nw > 0.0)) nw = 0.5 * alpha;
        const bool done = fabs(nw - alpha) <= 1e-15 * alpha;
        alpha = nw;
        if (done) break;
    }
    return alpha;
}

// Q(a, x), the regularised upper incomplete gamma function: power series of P below a + 1, continued fraction
// of Q above.
__device__ inline double gamma_upper_q(double a, double x) {
    if (!(x > 0.0)) return 1.0;
    const double log_front = a * log(x) - x - lgamma(a);
    if (x < a + 1.0) {
        double term = 1.0 / a, total = term;
        for (int n = 1; n < 10000; ++n) {
            term *= x / (a + n);
            total += term;
            if (fabs(term) <= 1e-17 * fabs(total)) break;
        }
        return 1.0 - total * exp(log_front);
    }
    const double tiny = 1e-300;
    double b = x + 1.0 - a, c = 1.0 / tiny, d = 1.0 / b, h = d;
    for (int i = 1; i < 10000; ++i) {
        const double an = -(double)i * ((double)i - a);
        b += 2.0;
        d = an * d + b;
        if (fabs(d) < tiny) d = tiny;
        c = b + an / c;
        if (fabs(c) < tiny) c = tiny;
        d = 1.0 / d;
        const double del = d * c;
        h *= del;
        if (fabs(del - 1.0) < 1e-16) break;
    }
    return h * exp(log_front);
}

// x with Q(a, x) = q: bracket by doubling, then Newton on log Q kept inside the bracket (bisection otherwise).
__device__ inline double gamma_upper_quantile(double a, double q) {
    if (q >= 1.0) return 0.0;
    double lo = 0.0, hi = a > 1.0 ? a : 1.0;
    for (int it = 0; it < 2000 && gamma_upper_q(a, hi) > q; ++it) { lo = hi; hi = 2.0 * hi; }
    double x = 0.5 * (lo + hi);
    const double lq = log(q);
    for (int it = 0; it < 200; ++it) {
        const double qx = gamma_upper_q(a, x);
        if (qx > q) lo = x; else hi = x;
        const double dens = exp((a - 1.0) * log(x) - x - lgamma(a));
        double nw = (qx > 0.0 && dens > 0.0) ? x + (log(qx) - lq) * qx / dens : 0.5 * (lo + hi);
        if (!(lo < nw && nw < hi)) nw = 0.5 * (lo + hi);
        const bool done = fabs(nw - x) <= 1e-15 * x;
        x = nw;
        if (done) break;
    }
    return x;
}

// What the fitting thread hands to its own CTA (the other runs of the segment read SegDev::pub).
struct Fit {
    double eta;
    float thr;          // thr_ge(eta) if the stage is the segment's last, thr_gt(eta) otherwise
    int stages;         // stages fitted so far
    bool last;
    // for the record kept in SegDev (see record_stage)
    int M_eff, status, n_e;
    bool empty;         // segment without elements
};

__device__ __forceinline__ Fit warp_broadcast(const Fit& f) {
    Fit g;
    g.eta = __shfl_sync(kFull, f.eta, 0);
    g.thr = __shfl_sync(kFull, f.thr, 0);
    g.stages = __shfl_sync(kFull, f.stages, 0);
    g.last = __shfl_sync(kFull, (int)f.last, 0) != 0;
    g.M_eff = __shfl_sync(kFull, f.M_eff, 0);
    g.status = __shfl_sync(kFull, f.status, 0);
    g.n_e = __shfl_sync(kFull, f.n_e, 0);
    g.empty = __shfl_sync(kFull, (int)f.empty, 0) != 0;
    return g;
}

// The fields of SegDev that describe a fitted stage, other than the published word: written after it, by
// the threads first, first + step, ... of a group that all hold `f` (a warp, or one thread with step 1).
// `stage` = 0 writes the whole record of the call's first stage and clears the later stages' entries.
// These stores are ordered before any later fit of the segment by the fence and arrival atomic of this
// CTA's next phase.  Nothing else reads them during the call: the end of the call takes a segment's stage
// count and threshold from the run's own cache or from the published word, and writes only entries that
// this record leaves alone (k_stage[M_eff - 1], the adaptation state).
__device__ __forceinline__ void record_stage(SegDev* sg, int stage, const Fit& f, int first, int step) {
    if (stage == 0) {
        for (int q = first; q < 20; q += step) {
            if (q < 8) sg->eta[q] = (q == 0 || (f.empty && q < f.M_eff)) ? f.eta : 0.0;
            else if (q < 16) { if (q - 8 >= f.M_eff) sg->k_stage[q - 8] = 0; }   // the others are written by later fits / the count
            else if (q == 16) sg->M_eff = f.M_eff;
            else if (q == 17) sg->status = f.status;
            else if (q == 18) sg->thr_gt = __double2float_rd(f.eta);
            else sg->thr_ge = __double2float_ru(f.eta);
        }
    } else {
        for (int q = first; q < 5; q += step) {
            if (q == 0) sg->k_stage[stage - 1] = f.n_e;
            else if (q == 1) sg->eta[stage] = f.eta;
            else if (q == 2) sg->thr_gt = __double2float_rd(f.eta);
            else if (q == 3) sg->thr_ge = __double2float_ru(f.eta);
            else if (f.status) sg->status = ld_cg(&sg->status) | f.status;   // written by the previous stage's fit
        }
    }
}

// Publish a fitted stage: the tagged threshold word goes out first; everything else about the stage is
// stored afterwards (record_stage).  If another stage follows, its sweep shifts by eta, which is therefore
// stored before the word and released with it.  The word of a last stage carries all that its readers need
// (they go on to read only their own run's data), so it is a plain strong store with no fence to wait for.
__device__ inline Fit publish_stage(const Args& A, unsigned call_id, SegDev* sg, int stages, bool last, double eta) {
    Fit f{eta, last ? __double2float_ru(eta) : __double2float_rd(eta), stages, last, 0, 0, 0, false};
    const unsigned long long word = ((unsigned long long)__float_as_uint(f.thr) << 32) |
                                    (unsigned long long)(call_id * 16u + (unsigned)stages);
    if (A.drop_pub_seg >= 0 && sg == A.seg + A.drop_pub_seg) {
        // (test hook: nothing is published)
    } else if (last) {
        st_relaxed_u64(&sg->pub, word);
    } else {
        sg->eta[stages - 1] = eta;
        st_release_u64(&sg->pub, word);
    }
    return f;
}

// Stage 1 from the segment sums: S1 = sum|x|, and S2 = sum x^2 (GPD) or SL = sum log|x| over the
// n_nz nonzero magnitudes (gamma).
// EXACT: the exact forms of Corollary 1.2 are compiled in (a kernel instantiation of its own, so that the default
// one does not carry their code and registers).
template <int SID, bool EXACT>
__device__ inline Fit fit_stage1(const Args& A, SegDev* sg, int M_state, int n, double S1, double S2_or_SL,
                                 int n_nz, int cap, const LnTab& T) {
    int M;
    if (A.max_stages > 0) {
        M = M_state < 1 ? 1 : M_state;
        if (M > A.max_stages) M = A.max_stages;
    } else {
        M = -A.max_stages;
    }
    const int M_eff = M < cap ? M : cap;
    int status = 0;
    double eta;
    const int slot = ratio_slot(M_eff, 0);
    if (n == 0) {
        eta = __longlong_as_double(0x7ff0000000000000ll);
    } else if (!isfinite(S1) || !isfinite(S2_or_SL)) {
        status |= kStNonFinite;
        eta = __longlong_as_double(0x7ff8000000000000ll);
    } else if (S1 == 0.0) {
        status |= kStAllZero;
        eta = __longlong_as_double(0x7ff0000000000000ll);
    } else if (SID == kSidExp) {
        eta = exp_step(S1 / n, T.ln_inv[slot]);
    } else if (SID == kSidGpd) {
        const double mu = S1 / n;
        eta = gpd_step(mu, S2_or_SL / n - mu * mu, T.ln[slot], T.ln_inv[slot], status);
    } else {
        const double ratio = stage_ratio(A.delta, A.delta1, M_eff, 0);
        const double mu = S1 / n_nz;
        const double s = log(mu) - S2_or_SL / n_nz;
        double rz = ratio * n / n_nz;
        if (rz > 1.0) rz = 1.0;
        if (s <= 1e-12) {
            status |= kStDegenerate;
            eta = mu * log(1.0 / rz);
            if (!(eta > 0.0)) eta = 0.0;
        } else {
            double alpha = (3.0 - s + sqrt((s - 3.0) * (s - 3.0) + 24.0 * s)) / (12.0 * s);
            if (EXACT && A.pol_gamma_exact) {
                alpha = gamma_shape_mle(s, alpha);
                eta = (mu / alpha) * gamma_upper_quantile(alpha, rz);
            } else {
                const double beta = mu / alpha;
                eta = -beta * (log(rz) + lgamma(alpha));
                if (eta <= 0.0) { status |= kStDegenerate; eta = 0.0; }
            }
        }
    }
    // an empty segment takes part in no later phase: all its stages count as fitted here
    Fit f = publish_stage(A, T.call_id, sg, n == 0 ? M_eff : 1, n == 0 || M_eff == 1, eta);
    f.M_eff = M_eff;
    f.status = status;
    f.empty = n == 0;
    return f;
}

// Stage index m >= 1 (eta_{m+1} in the paper's numbering) of an M_eff-stage segment from the shifted peaks
// over prev = eta_m: n_e = #{|x| > eta_m}, Sy = sum(|x| - eta_m), Sy2 = sum(|x| - eta_m)^2.
template <int SID>
__device__ inline Fit fit_stage_m(const Args& A, SegDev* sg, int m, int M_eff, double prev, int n_e, double Sy,
                                  double Sy2, const LnTab& T, int n_seg) {
    double eta = prev;
    int status = 0;
    if (n_e > 0) {
        const int slot = ratio_slot(M_eff, m);
        double ln = T.ln[slot], ln_inv = T.ln_inv[slot];
        if (A.pol_ratio_counts && m + 1 == M_eff) {
            // the last stage keeps the target count out of what the stage before it left
            double ratio = A.delta * (double)n_seg / (double)n_e;
            if (ratio > 1.0) ratio = 1.0;
            ln = log(ratio);
            ln_inv = log(1.0 / ratio);
        }
        const double ybar = Sy / n_e;
        double inc;
        if (SID == kSidExp) inc = exp_step(ybar, ln_inv);
        else inc = gpd_step(ybar, Sy2 / n_e - ybar * ybar, ln, ln_inv, status);
        eta = prev + inc;
    }
    Fit f = publish_stage(A, T.call_id, sg, m + 1, m + 1 == M_eff, eta);
    f.M_eff = M_eff;
    f.status = status;
    f.n_e = n_e;
    return f;
}

// ----------------------------------------------------------------------------
// chunk access (one warp)
// ----------------------------------------------------------------------------

// 256-bit global accesses with an L2 eviction priority.  The error-compensation memory is read and
// rewritten by every call and nearly fits in L2: its lines are asked to stay (evict_last).  The gradient
// is read once: its lines are asked to leave first.  (Cache-policy operands on 128-bit accesses did not
// change what stays resident; these qualified 256-bit forms do.)
struct F8 { float v[kComp]; };

__device__ __forceinline__ F8 ld8_evict_first(const float* p) {
    F8 r;
    asm volatile("ld.global.L2::evict_first.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
__device__ __forceinline__ F8 ld8_evict_last(const float* p) {
    F8 r;
    asm volatile("ld.global.L2::evict_last.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ void st8_evict_last(float* p, const F8& r) {
    asm volatile("st.global.L2::evict_last.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
                 : "memory");
}

// Eight gradient elements starting at element e (read once: evict_first).  A bf16 gradient is widened exactly
// (bf16 is the upper half of an fp32).
__device__ __forceinline__ F8 ld8_grad(const float* grad, int e, bool bf16) {
    if (!bf16) return ld8_evict_first(grad + e);
    // (the eviction-priority qualifier exists for 256-bit accesses only: a streaming 128-bit load here)
    const uint4 w = __ldcs(reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned short*>(grad) + e));
    const unsigned w0 = w.x, w1 = w.y, w2 = w.z, w3 = w.w;
    F8 r;
    r.v[0] = __uint_as_float(w0 << 16); r.v[1] = __uint_as_float(w0 & 0xffff0000u);
    r.v[2] = __uint_as_float(w1 << 16); r.v[3] = __uint_as_float(w1 & 0xffff0000u);
    r.v[4] = __uint_as_float(w2 << 16); r.v[5] = __uint_as_float(w2 & 0xffff0000u);
    r.v[6] = __uint_as_float(w3 << 16); r.v[7] = __uint_as_float(w3 & 0xffff0000u);
    return r;
}
__device__ __forceinline__ float ld1_grad(const float* grad, int e, bool bf16) {
    if (!bf16) return __ldcs(grad + e);
    return __uint_as_float((unsigned)__ldcs(reinterpret_cast<const unsigned short*>(grad) + e) << 16);
}

// Asynchronous 16-byte copy from global to shared memory (completes in the background; see cp_async_wait_all).
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

// Error-compensation memory accesses: `keep` asks for L2 residency.  Segments with three or more stages
// go without it, because their side regions (re-read by every later stage) need the L2 more.
__device__ __forceinline__ F8 ld8_res(const float* p, bool keep) {
    if (keep) return ld8_evict_last(p);
    F8 r;
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p)), b = __ldcg(reinterpret_cast<const float4*>(p) + 1);
    r.v[0] = a.x; r.v[1] = a.y; r.v[2] = a.z; r.v[3] = a.w; r.v[4] = b.x; r.v[5] = b.y; r.v[6] = b.z; r.v[7] = b.w;
    return r;
}
__device__ __forceinline__ void st8_res(float* p, const F8& r, bool keep) {
    if (keep) { st8_evict_last(p, r); return; }
    reinterpret_cast<float4*>(p)[0] = make_float4(r.v[0], r.v[1], r.v[2], r.v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(r.v[4], r.v[5], r.v[6], r.v[7]);
}

// A chunk in registers: lane l holds, for slot j, the 8 elements at window offset 256 j + 8 l.
// Chunk order (= ascending index) is slot, lane, component; mask bit 8 j + c stands for v[j][c].

// Load the part [lo, hi) of the window starting at wb from `src` (the error-compensation memory).
// Returns the validity mask.
__device__ __forceinline__ unsigned load_chunk(const float* __restrict__ src, int lo, int hi, int wb, bool vec_ok,
                                               bool keep, float (&v)[kSlots][kComp]) {
    const int e0 = wb + (threadIdx.x & 31) * kComp;
    if (vec_ok && lo == wb && hi == wb + kChunk) {
        #pragma unroll
        for (int j = 0; j < kSlots; ++j) {
            const F8 q = ld8_res(src + e0 + j * 256, keep);
            #pragma unroll
            for (int c = 0; c < kComp; ++c) v[j][c] = q.v[c];
        }
        return kFull;
    }
    unsigned valid = 0;
    #pragma unroll
    for (int j = 0; j < kSlots; ++j) {
        const int e = e0 + j * 256;
        #pragma unroll
        for (int c = 0; c < kComp; ++c) v[j][c] = 0.0f;
        if (e + kComp <= lo || e >= hi) continue;
        if (vec_ok && e >= lo && e + kComp <= hi) {
            const F8 q = ld8_res(src + e, keep);
            #pragma unroll
            for (int c = 0; c < kComp; ++c) v[j][c] = q.v[c];
            valid |= 0xFFu << (8 * j);
        } else {
            #pragma unroll
            for (int c = 0; c < kComp; ++c)
                if (e + c >= lo && e + c < hi) { v[j][c] = __ldcg(src + e + c); valid |= 1u << (8 * j + c); }
        }
    }
    return valid;
}

// Warp-ordered emission: calls emit(position, j, c) for every set bit of `mask`, positions counted
// in chunk order starting at `base`.  Returns the number of set bits in the warp.
template <class Emit>
__device__ __forceinline__ int ordered_emit(unsigned mask, int base, Emit emit) {
    const unsigned lt = (1u << (threadIdx.x & 31)) - 1u;
    int run = base;
    #pragma unroll
    for (int j = 0; j < kSlots; ++j) {
        const unsigned byte = (mask >> (8 * j)) & 0xFFu;
        if (__ballot_sync(kFull, byte != 0) == 0) continue;
        const int n = __popc(byte);                       // 0..8 survivors of this lane in this slot
        const unsigned b0 = __ballot_sync(kFull, n & 1);
        const unsigned b1 = __ballot_sync(kFull, n & 2);
        const unsigned b2 = __ballot_sync(kFull, n & 4);
        const unsigned b3 = __ballot_sync(kFull, n & 8);
        int p = run + __popc(b0 & lt) + 2 * __popc(b1 & lt) + 4 * __popc(b2 & lt) + 8 * __popc(b3 & lt);
        run += __popc(b0) + 2 * __popc(b1) + 4 * __popc(b2) + 8 * __popc(b3);
        #pragma unroll
        for (int cc = 0; cc < kComp; ++cc)
            if (byte & (1u << cc)) { emit(p, j, cc); ++p; }
    }
    return run - base;
}

// Per-warp view of the segment a chunk belongs to, refreshed only when the segment changes.  The
// values come from the run's shared-memory cache; a warp that gets there first waits (bounded) for
// the thread that publishes them.
struct SegView {
    int seg = -1;
    int M_eff = 0;
    float thr_gt = 0.f, thr_ge = 0.f;   // both hold the one threshold of the phase (see RunSegs::thr)
    double eta_prev = 0.0;
};

// Dynamic chunk queue of a CTA run: warps take the next chunk index (ascending or descending).
struct ChunkQueue {
    int* sm_next;
    int c0, c1;
    __device__ __forceinline__ int next(bool descending) const {
        int k = 0;
        if ((threadIdx.x & 31) == 0) k = atomicAdd(sm_next, 1);
        k = __shfl_sync(kFull, k, 0);
        if (k >= c1 - c0) return -1;
        return descending ? c1 - 1 - k : c0 + k;
    }
    // The next entry of a list of n chunk numbers (relative to c0) instead.
    __device__ __forceinline__ int next_listed(const int* list, int n) const {
        int k = 0;
        if ((threadIdx.x & 31) == 0) k = atomicAdd(sm_next, 1);
        k = __shfl_sync(kFull, k, 0);
        return k < n ? c0 + list[k] : -1;
    }
};

constexpr int kSidePre = 1;                       // 16-byte pieces of a side region fetched with the descriptor
constexpr int kSidePre4 = 2;                      // the same in the sweeps that read nothing but side regions
// Dynamic shared memory: per-warp staging of one slot row of a chunk's side region (stage-2 sweep only; the
// survivor list and the window counters of the final selection lie over it), then the candidate slots.  (Kept
// small on purpose: what shared memory takes, the L1 loses, and the first sweep's bandwidth suffers.)
constexpr int kStageRow = kChunk / kSlots + 8;    // floats of staging per warp: one slot row plus the carried tail
constexpr int kStageBytes = kWarps * kStageRow * (int)sizeof(float);
constexpr int kDynSmemBytes = kStageBytes + kSlotPre * kComp * (int)sizeof(float) + kSlotCap * ((int)sizeof(int) + 1)
                            + kScWin * ((int)sizeof(float) + (int)sizeof(unsigned short) + 1);
static_assert(kStageBytes >= kOutCache * 8 + kWinCap * 8, "survivor list and window counters fit over the staging area");

// Positions of a lane's kept elements in the chunk's dense, index-ordered side region.  `mask` has bit
// 8 j + c set for component c of slot j; chunk order is slot, lane, component.  pos[j] is where this lane's
// first kept element of slot j goes, base[j] where slot j's elements begin; the return value is the number of
// kept elements in the whole chunk.
__device__ __forceinline__ int side_positions(unsigned mask, int (&pos)[kSlots], int (&base)[kSlots]) {
    static_assert(kSlots == 4, "two packed scans cover four slots");
    const int lane = threadIdx.x & 31;
    const unsigned c01 = __popc(mask & 0xFFu) | (__popc((mask >> 8) & 0xFFu) << 16);
    const unsigned c23 = __popc((mask >> 16) & 0xFFu) | (__popc(mask >> 24) << 16);
    unsigned i01 = c01, i23 = c23;                 // inclusive scans over the lanes (a field holds at most 256)
    #pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned a = __shfl_up_sync(kFull, i01, o), b = __shfl_up_sync(kFull, i23, o);
        if (lane >= o) { i01 += a; i23 += b; }
    }
    const unsigned t01 = __shfl_sync(kFull, i01, 31), t23 = __shfl_sync(kFull, i23, 31);
    const unsigned e01 = i01 - c01, e23 = i23 - c23;
    const int t0 = t01 & 0xFFFFu, t1 = t01 >> 16, t2 = t23 & 0xFFFFu, t3 = t23 >> 16;
    base[0] = 0; base[1] = t0; base[2] = t0 + t1; base[3] = t0 + t1 + t2;      // where each slot's entries begin
    pos[0] = e01 & 0xFFFFu;
    pos[1] = base[1] + (e01 >> 16);
    pos[2] = base[2] + (e23 & 0xFFFFu);
    pos[3] = base[3] + (e23 >> 16);
    return base[3] + t3;
}

// Chunk descriptor, fetched one chunk ahead so that its loads overlap the current chunk's work.
struct Desc {
    int c, seg, lo, hi;
    int side_n;          // entries in the chunk's side region (phases that read side regions)
    float4 pre[kSidePre];// entries 128 u + 4 lane .. + 3 of the side region, fetched with the descriptor and
                         // without waiting for the count (entries beyond it are ignored)
};

__device__ __forceinline__ Desc fetch_desc(const Args& A, int c, bool with_side) {
    Desc d;
    d.c = c; d.seg = 0; d.lo = 0; d.hi = 0; d.side_n = 0;
    if (c >= 0) {
        d.seg = __ldg(A.chunk_seg + c);
        d.lo = __ldg(A.chunk_start + c);
        d.hi = __ldg(A.chunk_start + c + 1);
        if (with_side) {
            d.side_n = ld_cg(A.side_cnt + c);
            const float4* side = reinterpret_cast<const float4*>(A.side_val + (size_t)c * kChunk) + (threadIdx.x & 31);
            #pragma unroll
            for (int u = 0; u < kSidePre; ++u) d.pre[u] = __ldcg(side + 32 * u);
        }
    }
    return d;
}

// Descriptor of the sweeps over side regions alone (stages 3..M).
struct SideDesc {
    int c, seg, side_n;
    float4 pre[kSidePre4];
};
__device__ __forceinline__ SideDesc fetch_side_desc(const Args& A, int c) {
    SideDesc d;
    d.c = c; d.seg = 0; d.side_n = 0;
    if (c >= 0) {
        d.seg = __ldg(A.chunk_seg + c);
        d.side_n = ld_cg(A.side_cnt + c);
        const float4* side = reinterpret_cast<const float4*>(A.side_val + (size_t)c * kChunk) + (threadIdx.x & 31);
        #pragma unroll
        for (int u = 0; u < kSidePre4; ++u) d.pre[u] = __ldcg(side + 32 * u);
    }
    return d;
}

// Sum of the per-chunk partials q = first, first + stride, ... < q1, added in that order.  Loads are
// issued eight chunks at a time so that a long segment costs few memory round trips.
__device__ __forceinline__ Sums strided_partials(const Args& A, int first, int q1, int stride) {
    double a = 0.0, b = 0.0;
    int n = 0;
    for (int q = first; q < q1; q += 8 * stride) {
        double xa[8], xb[8];
        int xn[8];
        #pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int qq = q + u * stride;
            const bool ok = qq < q1;
            xa[u] = ok ? ld_cg(A.part + 3 * (size_t)qq + 0) : 0.0;
            xb[u] = ok ? ld_cg(A.part + 3 * (size_t)qq + 1) : 0.0;
            xn[u] = ok ? ld_cg(A.part_n + qq) : 0;
        }
        #pragma unroll
        for (int u = 0; u < 8; ++u) { a += xa[u]; b += xb[u]; n += xn[u]; }
    }
    return Sums{a, b, n};
}

// Table entries of the segments of a CTA run, cached in shared memory at kernel start.
struct RunSegs {
    unsigned call_id;           // number of this call
    int seg_lo, n_seg;          // segments seg_lo .. seg_lo + n_seg - 1 have chunks in (or between) this run
    int* q0;                    // [kSegCache] first chunk
    int* q1;                    // [kSegCache] one past the last chunk
    int* runs;                  // [kSegCache] CTA runs holding chunks of the segment
    int* m_eff;                 // [kSegCache] stage count of the segment in this call
    int* n;                     // [kSegCache] elements of the segment
    float* tau;                 // [kSegCache] candidate threshold for the first sweep (< 0: none)
    // thresholds of the phase being swept, published by one thread per segment (see publish_params)
    float* thr;                 // [kSegCache] thr_gt of the stage the phase shifts by; thr_ge of the last stage in P5a
    double* eta_prev;           // [kSegCache]
    volatile int* ok;           // [kSegCache] == phase tag once the two values above are valid
    int c0, c1;                 // chunks of the run
    __device__ __forceinline__ void get(const Args& A, int i, int& a, int& b, int& r) const {
        if (i < kSegCache) { a = q0[i]; b = q1[i]; r = runs[i]; }
        else { a = A.seg_chunk0[seg_lo + i]; b = A.seg_chunk0[seg_lo + i + 1]; r = A.seg_runs[seg_lo + i]; }
    }
};

// One thread per segment of the run waits (bounded) until the segment has the stages this phase needs,
// then copies its thresholds into the shared-memory cache and marks them valid with the phase tag.
// need: stages that must be fitted (0: all of the segment's); m_prev: index of the eta the phase shifts by.
// A segment fitted by this CTA itself already has them (see arrive_and_fit).
__device__ __forceinline__ void publish_params(const Args& A, const RunSegs& R, int need, int m_prev, int tag) {
    const int i = threadIdx.x;
    if (i < R.n_seg && i < kSegCache && R.q1[i] > R.q0[i] && R.ok[i] != tag) {
        const SegDev* sg = &A.seg[R.seg_lo + i];
        const int M_eff = R.m_eff[i];
        R.thr[i] = wait_ready_thread(A, R.call_id, sg, need == 0 ? M_eff : (need < M_eff ? need : M_eff));
        // only a segment with a further stage is swept in this phase and needs the shift
        double eta_prev = 0.0;
        if (m_prev >= 0 && M_eff > need) {
            __threadfence();                       // acquire side of the stage's release
            eta_prev = ld_cg(&sg->eta[m_prev]);
        }
        R.eta_prev[i] = eta_prev;
        __threadfence_block();
        R.ok[i] = tag;
    }
}

// Refresh a warp's segment view when the chunk's segment changed.
__device__ __forceinline__ void view_load(const Args& A, const RunSegs& R, SegView& v, int seg, int need, int m_prev,
                                          int tag, int cap) {
    if (seg == v.seg) return;
    v.seg = seg;
    const int i = seg - R.seg_lo;
    if (i < kSegCache) {
        v.M_eff = R.m_eff[i];
        long long spins = 0;
        while (R.ok[i] != tag) {                       // published by a thread of this CTA
            if (++spins > A.spin_limit) { atomicExch(&A.ctl->timeout, 1); break; }
            __nanosleep(20);
        }
        __threadfence_block();
        v.thr_gt = v.thr_ge = R.thr[i];
        v.eta_prev = R.eta_prev[i];
    } else {
        // beyond the cache (a run spanning more than kSegCache segments): straight from global memory
        const SegDev* sg = &A.seg[seg];
        v.M_eff = seg_stages(A, seg, cap);
        v.thr_gt = v.thr_ge = wait_ready(A, R.call_id, sg, need == 0 ? v.M_eff : (need < v.M_eff ? need : v.M_eff));
        v.eta_prev = 0.0;
        if (m_prev >= 0 && v.M_eff > need) {
            __threadfence();                       // acquire side of the stage's release
            v.eta_prev = ld_cg(&sg->eta[m_prev]);
        }
    }
}

// `stage` = 0 for the first stage, m >= 1 for the refits.  Every CTA calls this after its warps
// have written the partials of all chunks of its run.  A segment that lies inside this run alone is
// fitted at once; one shared with other runs is fitted by the run that arrives last.
// The fitting thread also puts the result into this CTA's own parameter cache, tagged for the phase that
// uses it next, so that the CTA does not wait for its own publication to come back through L2.
// One warp: its first lane fits segment i2 of the run from its sums (M_state and r are that lane's), publishes, and
// fills the CTA's own cache entry; all lanes then write the stage's record.
template <int SID, bool EXACT>
__device__ __forceinline__ void fit_and_cache(const Args& A, const RunSegs& R, int stage, int cap, const LnTab& T,
                                              SegDev* sg, int i2, int M_state, const Sums& r) {
    const int lane = threadIdx.x & 31;
    {
        const bool cached = i2 < kSegCache;
        Fit f{};
        if (lane == 0) {
            if (stage == 0) {
                f = fit_stage1<SID, EXACT>(A, sg, M_state, cached ? R.n[i2] : A.seg_n[R.seg_lo + i2], r.a, r.b, r.n, cap, T);
            } else {
                // this run swept the segment in the phase that just ended, so its cache holds eta_{stage}
                const int M_eff = cached ? R.m_eff[i2] : seg_stages(A, R.seg_lo + i2, cap);
                const double prev = cached ? R.eta_prev[i2] : ld_cg(&sg->eta[stage - 1]);
                f = fit_stage_m<SID>(A, sg, stage, M_eff, prev, r.n, r.a, r.b, T, cached ? R.n[i2] : A.seg_n[R.seg_lo + i2]);
            }
            if (cached) {
                R.thr[i2] = f.thr;
                R.eta_prev[i2] = f.eta;
                __threadfence_block();
                R.ok[i2] = f.last ? 100 : f.stages;        // tag of the phase that uses these values next
            }
        }
        record_stage(sg, stage, warp_broadcast(f), lane, 32);
    }
}

template <int SID, bool EXACT>
__device__ __forceinline__ void fit_phase(const Args& A, const RunSegs& R, int stage, int cap, const LnTab& T,
                                          int* sm_small, int* sm_large, int* sm_count, double (*sm_red)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto fit_and_cache = [&](SegDev* sg, int i2, int M_state, const Sums& r) {
        sidco::fit_and_cache<SID, EXACT>(A, R, stage, cap, T, sg, i2, M_state, r);
    };
    for (int base = 0; base < R.n_seg; base += kThreads) {
        const int i = base + (int)threadIdx.x;
        if (i < R.n_seg) {
            int q0, q1, runs;
            R.get(A, i, q0, q1, runs);
            if (q1 > q0) {
                SegDev* sg = &A.seg[R.seg_lo + i];
                const bool takes_part = stage == 0 || (i < kSegCache ? R.m_eff[i] : seg_stages(A, R.seg_lo + i, cap)) > stage;
                const bool giant = q1 - q0 > kGiantSeg;
                bool complete = takes_part && runs == 1 && !giant;
                if (takes_part && runs > 1 && !giant) {
                    complete = atom_add_acquire(&sg->arrived, 1) == runs - 1;
                    if (complete) sg->arrived = 0;     // (the other runs' partials, read next, came with the acquire)
                }
                if (complete) {
                    if (q1 - q0 <= kSmallSeg) sm_small[atomicAdd(&sm_count[0], 1)] = i;
                    else sm_large[atomicAdd(&sm_count[1], 1)] = i;
                }
                if (takes_part && giant) {
                    // A giant segment is summed in two levels, so that no single CTA has to read all its chunk
                    // partials: tiles of kTile chunks (counted from the segment's first chunk, whatever the grid)
                    // are summed by the run whose arrival completes the tile; the run that completes the last
                    // tile adds the tile sums up and fits.
                    const int ca = max(q0, R.c0), cb = min(q1, R.c1);
                    const int t0 = A.seg_tile0[R.seg_lo + i];
                    for (int t = (ca - q0) / kTile; t * kTile + q0 < cb; ++t) {
                        const int ta = q0 + t * kTile, tb = min(ta + kTile, q1);
                        const int mine = min(cb, tb) - max(ca, ta);
                        const int old = atom_add_acquire(&A.tile_arr[t0 + t], mine);
                        if (old + mine == tb - ta) {
                            A.tile_arr[t0 + t] = 0;
                            const int slot = atomicAdd(&sm_count[1], 1);
                            if (slot < kThreads) sm_large[slot] = i | ((t + 1) << 20);      // (tile number + 1 above the segment)
                        }
                    }
                }
            }
        }
        __syncthreads();
        const int n_small = sm_count[0], n_large = min(sm_count[1], kThreads);
        // Large segments (other runs wait for them) are fitted by two groups of twelve warps, two segments at
        // a time: threads stride over the chunk partials, fixed tree over the group.  The other eight warps
        // take the small segments meanwhile (all warps do if there is no large one).
        const int g = warp / kFitGroupWarps;
        if (g < kFitGroups) {
            const int tg = threadIdx.x - g * 32 * kFitGroupWarps;
            for (int k = g; k < n_large; k += kFitGroups) {
                const int i2 = sm_large[k] & 0xFFFFF, tile = (sm_large[k] >> 20) - 1;
                int q0, q1, runs;
                R.get(A, i2, q0, q1, runs);
                SegDev* sg = &A.seg[R.seg_lo + i2];
                const int M_state = (stage == 0 && tg == 0) ? (i2 < kSegCache ? R.m_eff[i2] : sg->M) : 0;
                if (tile < 0) {
                    const Sums t = strided_partials(A, q0 + tg, q1, 32 * kFitGroupWarps);
                    Sums r = group_tree(t.a, t.b, t.n, sm_red + kFitGroupWarps * g, g);
                    if (tg < 32) fit_and_cache(sg, i2, M_state, r);
                } else {
                    // one tile of a giant segment; if it is the segment's last, the tile sums and the fit
                    const int t0 = A.seg_tile0[R.seg_lo + i2], n_tiles = (q1 - q0 + kTile - 1) / kTile;
                    const int ta = q0 + tile * kTile, tb = min(ta + kTile, q1);
                    const Sums t = strided_partials(A, ta + tg, tb, 32 * kFitGroupWarps);
                    Sums r = group_tree(t.a, t.b, t.n, sm_red + kFitGroupWarps * g, g);
                    if (tg < 32) {
                        int last = 0;
                        if (lane == 0) {
                            double* tp = A.tile_part + 3 * (size_t)(t0 + tile);
                            tp[0] = r.a; tp[1] = r.b; tp[2] = (double)r.n;
                            __threadfence();
                            last = atom_add_acquire(&sg->arrived, 1) == n_tiles - 1;
                            if (last) sg->arrived = 0;
                        }
                        if (__shfl_sync(kFull, last, 0)) {
                            double a = 0.0, b = 0.0, c = 0.0;
                            for (int u = lane; u < n_tiles; u += 32) {             // lanes stride over the tiles
                                const double* tp = A.tile_part + 3 * (size_t)(t0 + u);
                                a += ld_cg(tp); b += ld_cg(tp + 1); c += ld_cg(tp + 2);
                            }
                            #pragma unroll
                            for (int o = 16; o > 0; o >>= 1) {
                                a += __shfl_down_sync(kFull, a, o);
                                b += __shfl_down_sync(kFull, b, o);
                                c += __shfl_down_sync(kFull, c, o);
                            }
                            fit_and_cache(sg, i2, M_state, Sums{a, b, (int)c});
                        }
                    }
                }
            }
        }
        // small segments: one warp each, lanes stride over the chunk partials, fixed shuffle tree
        const int small_first = n_large ? kFitGroups * kFitGroupWarps : 0;       // warps that take them
        for (int k = warp - small_first; k >= 0 && k < n_small; k += kWarps - small_first) {
            const int i2 = sm_small[k];
            int q0, q1, runs;
            R.get(A, i2, q0, q1, runs);
            SegDev* sg = &A.seg[R.seg_lo + i2];
            // (a cached stage count reproduces itself through fit_stage1's clamps; otherwise the state is
            // loaded, in flight with the partials)
            const int M_state = (stage == 0 && lane == 0) ? (i2 < kSegCache ? R.m_eff[i2] : sg->M) : 0;
            const Sums t = strided_partials(A, q0 + lane, q1, 32);
            Sums r = warp_tree(t.a, t.b, t.n);
            fit_and_cache(sg, i2, M_state, r);
        }
        __syncthreads();
        if (threadIdx.x < 2) sm_count[threadIdx.x] = 0;
        __syncthreads();
    }
}

template <int SID, bool EXACT, class AfterSweep>
__device__ __forceinline__ void arrive_and_fit(const Args& A, const RunSegs& R, int stage, int cap, const LnTab& T,
                                               int* sm_small, int* sm_large, int* sm_count, double (*sm_red)[3],
                                               int stamp_slot, const AfterSweep& after_sweep) {
    __threadfence();
    __syncthreads();
    after_sweep();       // (the CTA's sweep is over and its stores are fenced)
    SIDCO_STAMP(if (threadIdx.x == 0) {                       // this CTA's sweep is over
        const unsigned long long now = global_ns();
        A.cta_ns[4 * blockIdx.x + (stage < 2 ? stage : 2)] = now;
        if (blockIdx.x == 0) A.ctl->t_ns[stamp_slot] = now;
    });
    fit_phase<SID, EXACT>(A, R, stage, cap, T, sm_small, sm_large, sm_count, sm_red);
}

// ----------------------------------------------------------------------------
// the kernel
// ----------------------------------------------------------------------------

template <int SID, bool EXACT = false>
__global__ void __launch_bounds__(kThreads, 1) sidco_persistent_kernel(const __grid_constant__ Args A) {
    extern __shared__ __align__(16) float sm_stage[];        // [kWarps][kChunk] (kDynSmemBytes)
    __shared__ double sm_red[kWarps][3];
    __shared__ int sm_list[kThreads];
    __shared__ int sm_scan[kThreads];
    __shared__ int sm_warp[kWarps];
    __shared__ int sm_count[2];
    __shared__ int sm_next;
    __shared__ int sm_base;
    __shared__ int sm_resweep;
    __shared__ int sm_mloc;
    __shared__ int sm_q0[kSegCache], sm_q1[kSegCache], sm_runs[kSegCache], sm_meff[kSegCache], sm_segn[kSegCache];
    __shared__ float sm_tau[kSegCache], sm_thr[kSegCache];
    __shared__ double sm_eta[kSegCache];
    __shared__ int sm_ok[kSegCache];
    __shared__ int sm_segk[kSegCache];      // survivors of the run per cached segment
    __shared__ int sm_rest[kThreads];       // chunks (relative to c0) whose survivors the candidates do not cover
    __shared__ int sm_nrest, sm_nslot, sm_nfetched, sm_nsurv;
    __shared__ int sm_run_e[2];             // first element of the run and one past its last
    // over the staging area (used after the last sweep that stages): the run's unordered survivor list and the
    // per-window counters that put it in order
    int* const sm_oidx = reinterpret_cast<int*>(sm_stage);
    float* const sm_oval = sm_stage + kOutCache;
    int* const sm_wcnt = reinterpret_cast<int*>(sm_stage) + 2 * kOutCache;
    int* const sm_wfill = sm_wcnt + kWinCap;
    // behind it: the candidate slots (their 8 values, first element, segment of the run); once the survivors are
    // known, the space of the values takes the ordered list
    float* const sm_slot_val = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(sm_stage) + kStageBytes);
    int* const sm_slot_e = reinterpret_cast<int*>(sm_slot_val + kSlotPre * kComp);
    unsigned char* const sm_slot_seg = reinterpret_cast<unsigned char*>(sm_slot_e + kSlotCap);
    // A segment without a candidate threshold from the previous call (the first call on a fresh residual): a warp
    // derives one from the chunk of the segment it read last.  Per window: the threshold used (0: none), the chunk
    // (relative to the run) and the cached segment, for the check against the fitted threshold.
    float* const sm_wtau = reinterpret_cast<float*>(sm_slot_seg + kSlotCap);
    unsigned short* const sm_wchunk = reinterpret_cast<unsigned short*>(sm_wtau + kScWin);
    unsigned char* const sm_wseg = reinterpret_cast<unsigned char*>(sm_wchunk + kScWin);
    int* const sm_cidx = reinterpret_cast<int*>(sm_slot_val);
    float* const sm_cval = sm_slot_val + kOutCache;
    __shared__ unsigned sm_call;
    __shared__ int sm_reszero;

    const int cta = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int4 run = __ldg(A.cta_desc + cta);          // {first chunk, end chunk, first segment, segments}
    const int c0 = run.x, c1 = run.y;
    const bool vec_ok = A.vec_ok != 0;
    const bool g_bf16 = A.grad_bf16 != 0;
    const ChunkQueue queue{&sm_next, c0, c1};
    // Sweep directions.  Every full sweep over acc starts where the previous one (of this call or
    // of the last call) ended, so that it begins on the lines most recently left in L2.
    const bool p1_desc = A.cta_dir[cta] != 0;
    // The first chunk of every warp is fixed (chunk number `warp` of the sweep; the queue starts behind
    // these), so that its descriptor can be fetched now, under the set-up that follows.
    const int first_chunk = warp < c1 - c0 ? (p1_desc ? c1 - 1 - warp : c0 + warp) : -1;
    const Desc first_desc = fetch_desc(A, first_chunk, false);
    const int cap = stage_cap(A.delta, A.delta1);
    [[maybe_unused]] const bool stamper = (cta == 0 && threadIdx.x == 0);
    SIDCO_STAMP(if (stamper) A.ctl->t_ns[0] = global_ns());
    if (threadIdx.x == 0) sm_mloc = 1;
    if (threadIdx.x == 0) { sm_next = kWarps; sm_resweep = 0; sm_nrest = 0; sm_nslot = 0; sm_nfetched = 0; sm_nsurv = 0; }
    if (threadIdx.x < 2) sm_count[threadIdx.x] = 0;
    if (threadIdx.x < kScWin) sm_wtau[threadIdx.x] = 0.0f;
    if (threadIdx.x < 2) sm_run_e[threadIdx.x] = __ldg(A.chunk_start + (threadIdx.x ? c1 : c0));
    // What changes from call to call lives in the workspace (and is advanced by the CTA that finishes the call
    // last, long after every CTA has read it here).  The loads are issued now and their values handed to the
    // CTA after the table loop, whose own loads they overlap.
    unsigned seq_loaded = 0u;
    int reszero_loaded = 0;
    if (threadIdx.x == 0) {
        seq_loaded = ld_cg(&A.ctl->seq);
        reszero_loaded = ld_cg(&A.ctl->residual_is_zero);
    }
    __syncthreads();
    auto stages_of = [&](int seg) -> int { return seg_stages(A, seg, cap); };
    // cache the run's segment table; find the largest stage count among the run's segments, which
    // is the number of statistics phases this CTA takes part in
    const int run_seg_lo = run.z, run_n_seg = run.w;
    for (int i = threadIdx.x; i < run_n_seg; i += kThreads) {
        const int q0 = A.seg_chunk0[run_seg_lo + i], q1 = A.seg_chunk0[run_seg_lo + i + 1];
        const int m = stages_of(run_seg_lo + i);
        if (i < kSegCache) {
            sm_q0[i] = q0; sm_q1[i] = q1; sm_runs[i] = A.seg_runs[run_seg_lo + i];
            sm_meff[i] = m;
            sm_segn[i] = A.seg_n[run_seg_lo + i];
            // (a segment of one window at most records every slot that is not all zero: its threshold moves too
            // much from call to call for a fraction of the last one to hold)
            const float tau = A.seg_n[run_seg_lo + i] <= kChunk ? 1.17549435e-38f : A.seg[run_seg_lo + i].spec_thr;
            sm_tau[i] = (A.spec_enable && m <= 2 && tau > 0.0f) ? tau : -1.0f;
            sm_ok[i] = 0;
            sm_segk[i] = 0;
        }
        if (q1 > q0) atomicMax(&sm_mloc, m);
    }
    int resweep = 0;             // chunks of acc this warp read a second time in full

    if (threadIdx.x == 0) { sm_call = seq_loaded + 1u; sm_reszero = reszero_loaded; }
    __syncthreads();
    const unsigned call_id = sm_call;
    const bool res_zero = sm_reszero != 0;
    RunSegs R{call_id, run_seg_lo, run_n_seg, sm_q0, sm_q1, sm_runs, sm_meff, sm_segn, sm_tau, sm_thr, sm_eta, sm_ok, c0, c1};
    const LnTab T{A.ln_ratio, A.ln_inv_ratio, call_id};
    const int sc_win0 = sm_run_e[0] >> 10;
    const bool sc_on = A.spec_enable && vec_ok && c1 > c0 && run_n_seg <= kSegCache && c1 - c0 < 65536 &&
                       ((sm_run_e[1] - 1) >> 10) - sc_win0 + 1 <= kScWin;
    auto sc_note = [&](int wb, float t, int c, int seg_i) {
        const int w = (wb >> 10) - sc_win0;
        if (SIDCO_IN_RANGE(A, w, kScWin)) { sm_wtau[w] = t; sm_wchunk[w] = (unsigned short)(c - c0); sm_wseg[w] = (unsigned char)seg_i; }
    };

    // Candidate threshold of a segment for this call (segments with one or two stages use one: the sweep
    // that precedes their last fit records which slots may hold survivors).  It depends on state the
    // previous call left behind, so every warp and every phase derives the same value.
    auto spec_tau = [&](int seg) -> float {
        return seg - R.seg_lo < kSegCache ? sm_tau[seg - R.seg_lo] : -1.0f;     // (candidates carry a cache index)
    };
    // A slot (8 elements of one lane) that may hold a survivor: only its place is noted here, inside the sweep;
    // its values are fetched into shared memory in one asynchronous wave when the CTA's sweep is over (for the
    // first kSlotPre slots; a run with more reads the others from acc when it compares them).
    auto list_slot = [&](int e, int seg_i) {
        const int q = atomicAdd(&sm_nslot, 1);
        if (!SIDCO_IN_RANGE(A, e + kComp - 1, A.d) || !SIDCO_IN_RANGE(A, seg_i, kSegCache)) return;
        if (q < kSlotCap) {
            sm_slot_e[q] = e;
            sm_slot_seg[q] = (unsigned char)seg_i;
        } else {
            // beyond what shared memory holds: to the run's part of the spill arrays (a run has at most one slot
            // per 8 elements, and its part starts at its first element / 8, so it cannot run out)
            const size_t at = (size_t)(sm_run_e[0] >> 3) + blockIdx.x + (size_t)(q - kSlotCap);
            if (SIDCO_IN_RANGE(A, at, (size_t)(A.d >> 3) + A.G)) { A.slot_spill_e[at] = e; A.slot_spill_seg[at] = (unsigned char)seg_i; }
        }
    };
    // Start the copies of the slots listed since the last call (all threads; after the sweep's stores are
    // fenced and the CTA has met).  They complete in the background, behind the fits.
    auto fetch_slots = [&]() {
        const int from = sm_nfetched, to = min(sm_nslot, kSlotPre);
        for (int q = from + (int)threadIdx.x; q < to; q += kThreads) {
            if (!SIDCO_IN_RANGE(A, sm_slot_e[q] + kComp - 1, A.d)) continue;
            const float* src = A.residual + sm_slot_e[q];
            cp_async_16(sm_slot_val + q * kComp, src);
            cp_async_16(sm_slot_val + q * kComp + 4, src + 4);
        }
        __syncthreads();
        if (threadIdx.x == 0) sm_nfetched = to;
    };
    // A chunk whose survivors no candidate list will hold: the final selection reads it.
    auto list_chunk = [&](int c) {
        if (lane == 0) {
            const int q = atomicAdd(&sm_nrest, 1);
            if (q < kThreads) sm_rest[q] = c - c0;
        }
    };

    // ------------------------------------------------------------------ P1
    {
        int tau_seg = -1, seg_m = 1;
        float tau = 3.4e38f;       // candidate threshold of the chunk's segment (huge: none)
        const float sc_ln = sc_on ? (A.spec_enable == 2 ? 2.0f : kScRatio) * (float)T.ln_inv[1] : 0.0f;
        const bool keep = true;    // ask for L2 residency of the acc lines
        Desc cur = first_desc;
        while (cur.c >= 0) {
            const Desc nxt = fetch_desc(A, queue.next(p1_desc), false);
            const int c = cur.c, lo = cur.lo, hi = cur.hi;
            const int wb = lo & ~(kChunk - 1);
            const int e0 = wb + lane * kComp;
            if (cur.seg != tau_seg) {
                tau_seg = cur.seg;
                seg_m = stages_of(cur.seg);
                const float t = seg_m == 1 ? spec_tau(cur.seg) : -1.0f;    // two-stage segments record in P3
                tau = t > 0.0f ? t : 3.4e38f;
            }

            double s1 = 0.0, s2 = 0.0, prod = 1.0;
            int esum = 0, nnz = 0;
            // `cc` is the element's place in its slot.  Sum of log|x| = (sum of exponents) * ln 2 + log(product of
            // mantissas): the magnitudes are multiplied in fp64 as they are, and after every fourth place of a slot
            // the product's exponent moves to an integer sum (four fp32 magnitudes cannot leave the fp64 range);
            // one log per chunk.
            auto accumulate = [&](float x, int cc) {
                const float a = fabsf(x);
                const double ad = (double)a;
                s1 += ad;
                if (SID == kSidGpd) s2 = fma(ad, ad, s2);
                if (SID == kSidGamma) {
                    if (a > 0.0f) {
                        prod *= ad;
                        ++nnz;
                    }
                    if ((cc & 3) == 3) {
                        const long long bits = __double_as_longlong(prod);
                        esum += (int)(bits >> 52) - 1023;
                        prod = __longlong_as_double((bits & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
                    }
                }
            };

            bool sc_chunk = false;
            float bigs[kSlots];
            if (vec_ok && lo == wb && hi == wb + kChunk && SIDCO_IN_RANGE(A, wb + kChunk - 1, A.d) && SIDCO_IN_RANGE(A, c, A.C)) {
                // no threshold from the previous call: the candidates are chosen below, by an estimate from the chunk itself
                sc_chunk = sc_on && seg_m == 1 && !(tau < 3.0e38f);
                #pragma unroll
                for (int b = 0; b < kSlots; b += 2) {
                    F8 g8[2], r8[2];
                    #pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        g8[j] = ld8_grad(A.grad, e0 + (b + j) * 256, g_bf16);
                        if (!res_zero) r8[j] = ld8_res(A.residual + e0 + (b + j) * 256, keep);
                    }
                    #pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        float big = 0.0f;
                        #pragma unroll
                        for (int cc = 0; cc < kComp; ++cc) {
                            const float a = res_zero ? g8[j].v[cc] : g8[j].v[cc] + r8[j].v[cc];
                            r8[j].v[cc] = a;
                            accumulate(a, cc);
                            big = fmaxf(big, fabsf(a));
                        }
                        st8_res(A.residual + e0 + (b + j) * 256, r8[j], keep);
                        bigs[b + j] = big;
                        if (big >= tau) list_slot(e0 + (b + j) * 256, cur.seg - R.seg_lo);
                    }
                }
                if (seg_m == 1 && !(tau < 3.0e38f) && !sc_chunk) list_chunk(c);      // single stage, no candidates recorded
            } else {
                // a ragged chunk made of whole slots records candidates like a full one
                const bool whole_slots = vec_ok && ((lo | hi) & (kComp - 1)) == 0;
                if (seg_m == 1 && !(whole_slots && tau < 3.0e38f)) list_chunk(c);
                #pragma unroll 1
                for (int j = 0; j < kSlots; ++j) {
                    const int e = e0 + j * 256;
                    if (e + kComp <= lo || e >= hi) continue;
                    if (!SIDCO_IN_RANGE(A, hi - 1, A.d) || !SIDCO_IN_RANGE(A, lo, A.d)) continue;
                    if (vec_ok && e >= lo && e + kComp <= hi) {
                        const F8 g = ld8_grad(A.grad, e, g_bf16);
                        F8 r;
                        if (!res_zero) r = ld8_res(A.residual + e, keep);
                        float big = 0.0f;
                        #pragma unroll
                        for (int cc = 0; cc < kComp; ++cc) {
                            r.v[cc] = res_zero ? g.v[cc] : g.v[cc] + r.v[cc];
                            accumulate(r.v[cc], cc);
                            big = fmaxf(big, fabsf(r.v[cc]));
                        }
                        st8_res(A.residual + e, r, keep);
                        if (whole_slots && big >= tau) list_slot(e, cur.seg - R.seg_lo);
                    } else {
                        for (int cc = 0; cc < kComp; ++cc) {
                            if (e + cc >= lo && e + cc < hi) {
                                const float a = ld1_grad(A.grad, e + cc, g_bf16) + (res_zero ? 0.0f : A.residual[e + cc]);
                                A.residual[e + cc] = a;
                                accumulate(a, cc);
                            }
                        }
                    }
                }
            }

            // per-chunk partials with a fixed shuffle tree
            double second = s2;
            if (SID == kSidGamma) {
                // normalise the per-lane product, multiply the mantissas across the warp, one log:
                // SL_chunk = (sum of exponents) * ln 2 + log(product of mantissas)
                const long long bits = __double_as_longlong(prod);
                esum += (int)(bits >> 52) - 1023;
                double m = __longlong_as_double((bits & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
                #pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    m *= __shfl_down_sync(kFull, m, o);
                    esum += __shfl_down_sync(kFull, esum, o);
                }
                second = (double)esum * 0.693147180559945309417232121458 + log(m);   // used from lane 0 only
            }
            Sums r = chunk_tree<SID == kSidGpd>(s1, second, nnz);
            if (lane == 0 && SIDCO_IN_RANGE(A, c, A.C)) {
                A.part[3 * (size_t)c + 0] = r.a;
                A.part[3 * (size_t)c + 1] = SID == kSidGamma ? second : r.b;
                A.part_n[c] = r.n;
            }
            if (sc_chunk) {
                // (the exponential form of the threshold, on this chunk's mean, scaled down; whether it was low
                // enough is checked against the fitted threshold before its candidates are used)
                const float mean = __shfl_sync(kFull, (float)r.a, 0) * (1.0f / kChunk);
                const float tau_c = mean > 0.0f ? mean * sc_ln : 1.17549435e-38f;
                #pragma unroll
                for (int j = 0; j < kSlots; ++j)
                    if (bigs[j] >= tau_c) list_slot(e0 + j * 256, cur.seg - R.seg_lo);
                if (lane == 0) sc_note(wb, tau_c, c, cur.seg - R.seg_lo);
            }
            cur = nxt;
        }
    }
    arrive_and_fit<SID, EXACT>(A, R, 0, cap, T, sm_list, sm_scan, sm_count, sm_red, 6, fetch_slots);
    if (threadIdx.x == 0) sm_next = 0;
    __syncthreads();
    const int M_max_eff = sm_mloc;       // phases this CTA runs; other CTAs may run more or fewer
    SIDCO_STAMP(if (stamper) A.ctl->t_ns[7] = A.ctl->t_ns[1] = A.ctl->t_ns[2] = A.ctl->t_ns[3] = global_ns());

    // ------------------------------------------------------------------ P3: stage 2 from acc
    if (M_max_eff >= 2) {
        publish_params(A, R, 1, 0, 1);
        {
            SegView sv;
            const float sc_ln = sc_on ? (A.spec_enable == 2 ? 2.0f : kScRatio) * (float)T.ln_inv[2] : 0.0f;
            Desc cur = fetch_desc(A, queue.next(!p1_desc), false);
            while (cur.c >= 0) {
                const Desc nxt = fetch_desc(A, queue.next(!p1_desc), false);
                view_load(A, R, sv, cur.seg, 1, 0, 1, cap);
                if (sv.M_eff >= 2) {
                    ++resweep;
                    const int c = cur.c, lo = cur.lo, hi = cur.hi;
                    const int wb = lo & ~(kChunk - 1);
                    float v[kSlots][kComp];
                    if (!SIDCO_IN_RANGE(A, hi - 1, A.d) || !SIDCO_IN_RANGE(A, lo, A.d) || !SIDCO_IN_RANGE(A, c, A.C)) { cur = nxt; continue; }
                    const unsigned valid = load_chunk(A.residual, lo, hi, wb, vec_ok, true, v);
                    // Stage 2 is the last stage of a two-stage segment: nothing reads its exceedances again except
                    // the final selection, which can work from the noted candidate slots (as after P1 for one stage).
                    const float tau2 = sv.M_eff == 2 ? spec_tau(cur.seg) : -1.0f;
                    // (without one from the previous call: by an estimate from the chunk itself, below)
                    const bool sc_chunk = sc_on && sv.M_eff == 2 && !(tau2 > 0.0f) && lo == wb && hi == wb + kChunk;
                    const bool flag_chunk = sc_chunk || (tau2 > 0.0f && vec_ok && ((lo | hi) & (kComp - 1)) == 0);
                    float bigs[kSlots];
                    // (elements outside the chunk read as zero and the threshold is never negative, so they
                    // pass no strict compare)
                    unsigned mask = 0;
                    double sy = 0.0, sy2 = 0.0;
                    #pragma unroll
                    for (int j = 0; j < kSlots; ++j) {
                        float big = 0.0f;
                        double sj = 0.0, sj2 = 0.0;        // (one short chain per slot, added up in slot order)
                        #pragma unroll
                        for (int cc = 0; cc < kComp; ++cc) {
                            const float a = fabsf(v[j][cc]);
                            big = fmaxf(big, a);
                            if (a > sv.thr_gt) {
                                const double y = (double)a - sv.eta_prev;
                                sj += y;
                                if (SID != kSidExp) sj2 = fma(y, y, sj2);
                                mask |= 1u << (8 * j + cc);
                            }
                        }
                        sy += sj;
                        if (SID != kSidExp) sy2 += sj2;
                        bigs[j] = big;
                        if (flag_chunk && !sc_chunk && big >= tau2) list_slot(wb + lane * kComp + j * 256, cur.seg - R.seg_lo);
                    }
                    if (!flag_chunk) {
                        list_chunk(c);
                        // The side region also takes the entries equal to eta_1: they are no exceedances (the
                        // statistics above leave them out), but if no later stage raises the threshold
                        // (eta_M = eta_1, e.g. a segment of equal magnitudes) the final rule |x| >= eta_M selects them.
                        // (An fp32 magnitude can equal eta_1 only if eta_1 is an fp32 value, which then is thr_gt.)
                        unsigned keep_mask = mask;
                        if ((double)sv.thr_gt == sv.eta_prev) {
                            #pragma unroll
                            for (int j = 0; j < kSlots; ++j)
                                #pragma unroll
                                for (int cc = 0; cc < kComp; ++cc)
                                    if (fabsf(v[j][cc]) == sv.thr_gt) keep_mask |= 1u << (8 * j + cc);
                            keep_mask &= valid;
                        }
                        // The kept values go to the chunk's side region dense and in index order, one slot row at a
                        // time: every lane puts its own at their positions in the warp's shared-memory staging area,
                        // and the warp copies the area out with 16-byte stores.  A row rarely ends on a 16-byte
                        // boundary: its last few values are carried to the front of the next row's staging.
                        int pos[kSlots], base[kSlots];
                        const int kept = side_positions(keep_mask, pos, base);
                        float* stage = sm_stage + warp * kStageRow;
                        float4* side = reinterpret_cast<float4*>(A.side_val + (size_t)c * kChunk);
                        #pragma unroll
                        for (int j = 0; j < kSlots; ++j) {
                            const int a0 = base[j] & ~3;                   // first position this round writes
                            const int end = j + 1 < kSlots ? base[j + 1] : kept;
                            int q = pos[j] - a0;
                            #pragma unroll
                            for (int cc = 0; cc < kComp; ++cc)
                                if ((keep_mask >> (8 * j + cc)) & 1u) { if (SIDCO_IN_RANGE(A, q, kStageRow)) stage[q] = v[j][cc]; ++q; }
                            __syncwarp();
                            const int n4 = (end - a0 + 3) >> 2;
                            for (int q4 = lane; q4 < n4; q4 += 32)
                                if (SIDCO_IN_RANGE(A, (a0 >> 2) + q4, kChunk / 4))
                                    side[(a0 >> 2) + q4] = reinterpret_cast<const float4*>(stage)[q4];
                            const int tail = end & 3;
                            const float carry = lane < tail ? stage[(end & ~3) - a0 + lane] : 0.0f;
                            __syncwarp();
                            if (lane < tail) stage[lane] = carry;
                        }
                        __syncwarp();
                        if (lane == 0) A.side_cnt[c] = kept;
                        A.side_mask[(size_t)c * 32 + lane] = keep_mask;
                    }
                    Sums r = chunk_tree<SID != kSidExp>(sy, sy2, __popc(mask));
                    if (lane == 0) {
                        A.part[3 * (size_t)c + 0] = r.a;
                        A.part[3 * (size_t)c + 1] = r.b;
                        A.part_n[c] = r.n;              // exceedances (the next fit's count)
                    }
                    if (sc_chunk) {
                        // (the exponential form of the stage's increment on this chunk's mean exceedance, scaled down)
                        const float sum_y = __shfl_sync(kFull, (float)r.a, 0);
                        const int n_y = __shfl_sync(kFull, r.n, 0);
                        float tau_c = n_y > 0 ? (float)sv.eta_prev + sum_y / (float)n_y * sc_ln : sv.thr_gt;
                        if (!(tau_c > 0.0f)) tau_c = 1.17549435e-38f;
                        #pragma unroll
                        for (int j = 0; j < kSlots; ++j)
                            if (bigs[j] >= tau_c) list_slot(wb + lane * kComp + j * 256, cur.seg - R.seg_lo);
                        if (lane == 0) sc_note(wb, tau_c, c, cur.seg - R.seg_lo);
                    }
                }
                cur = nxt;
            }
        }
        arrive_and_fit<SID, EXACT>(A, R, 1, cap, T, sm_list, sm_scan, sm_count, sm_red, 8, fetch_slots);
        if (threadIdx.x == 0) sm_next = 0;
        __syncthreads();
        SIDCO_STAMP(if (stamper) A.ctl->t_ns[9] = A.ctl->t_ns[2] = A.ctl->t_ns[3] = global_ns());

        // -------------------------------------------------------------- P4: stages 3..M from the side regions
        for (int m = 2; m < M_max_eff; ++m) {
            publish_params(A, R, m, m - 1, m);
            {
                SegView sw;
                SideDesc cur = fetch_side_desc(A, queue.next(false));
                while (cur.c >= 0) {
                    const SideDesc nxt = fetch_side_desc(A, queue.next(false));
                    view_load(A, R, sw, cur.seg, m, m - 1, m, cap);
                    if (sw.M_eff > m) {
                        // the side region is a dense list: 16 bytes per lane and step, the first steps fetched
                        // with the descriptor
                        const int c = cur.c, n = SIDCO_IN_RANGE(A, cur.side_n, kChunk + 1) && SIDCO_IN_RANGE(A, cur.c, A.C) ? cur.side_n : 0;
                        const float4* side = reinterpret_cast<const float4*>(A.side_val + (size_t)c * kChunk) + lane;
                        double sy = 0.0, sy2 = 0.0;
                        int cnt = 0;
                        auto take = [&](const float4& x, int first) {
                            const float a[4] = {fabsf(x.x), fabsf(x.y), fabsf(x.z), fabsf(x.w)};
                            #pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (first + u < n && a[u] > sw.thr_gt) {
                                    const double y = (double)a[u] - sw.eta_prev;
                                    sy += y;
                                    if (SID != kSidExp) sy2 = fma(y, y, sy2);
                                    ++cnt;
                                }
                        };
                        #pragma unroll
                        for (int u = 0; u < kSidePre4; ++u) take(cur.pre[u], 128 * u + 4 * lane);
                        for (int t = kSidePre4; 128 * t < n; t += 2) {
                            const float4 x0 = __ldcg(side + 32 * t);
                            const float4 x1 = 128 * (t + 1) < n ? __ldcg(side + 32 * (t + 1)) : make_float4(0.f, 0.f, 0.f, 0.f);
                            take(x0, 128 * t + 4 * lane);
                            take(x1, 128 * (t + 1) + 4 * lane);
                        }
                        Sums r = chunk_tree<SID != kSidExp>(sy, sy2, cnt);
                        if (lane == 0) {
                            A.part[3 * (size_t)c + 0] = r.a;
                            A.part[3 * (size_t)c + 1] = r.b;
                            A.part_n[c] = r.n;
                        }
                    }
                    cur = nxt;
                }
            }
            arrive_and_fit<SID, EXACT>(A, R, m, cap, T, sm_list, sm_scan, sm_count, sm_red, 10, [] {});
            if (threadIdx.x == 0) sm_next = 0;
            __syncthreads();
            SIDCO_STAMP(if (stamper) A.ctl->t_ns[11] = A.ctl->t_ns[3] = global_ns());
        }
    }

    // ------------------------------------------------------------------ P5: the final selection
    // Two ways.  (A) The usual one keeps everything in shared memory: the candidates recorded by the sweeps
    // are compared with the final thresholds, the few chunks without candidates (ragged chunks, segments with
    // three or more stages, segments whose candidate threshold turned out too high) are read by the warps, and
    // all survivors of the run end up in one unordered shared-memory list that is then put in index order
    // (grouped by 1024-element window with a counting pass, ranked inside a window by comparison), written to
    // its final place and zeroed in the residual.  Nothing is modified before the list is known to fit.
    // (B) Otherwise (many survivors per run, e.g. delta = 0.1) the warps go through all chunks of the run,
    // stage each chunk's survivors in order in the chunk's staging region, and the placement goes through a
    // block scan over the chunk counts.
    publish_params(A, R, 0, -1, 100);          // one thread per segment waits (bounded) for its last threshold
    cp_async_wait_all();                       // this thread's share of the candidate slots has arrived
    __syncthreads();
    SIDCO_STAMP(if (threadIdx.x == 0 && M_max_eff == 1) A.cta_ns[4 * cta + 1] = global_ns());     // (single-stage runs: thresholds known)
    // the recorded candidates of cached segment i contain all its survivors among the chunks that recorded some
    auto seg_cand_ok = [&](int i) -> bool { return sm_tau[i] > 0.0f && R.thr[i] >= sm_tau[i]; };
    // the same for a full chunk whose warp used its own estimate (0 if it used none)
    auto sc_tau_of = [&](int e) -> float { return sc_on ? sm_wtau[(e >> 10) - sc_win0] : 0.0f; };
    const int run_e0 = sm_run_e[0], run_e1 = sm_run_e[1];
    const int win0 = run_e0 >> 10;
    const int n_win = c1 > c0 ? ((run_e1 - 1) >> 10) - win0 + 1 : 0;
    bool path_a = run_n_seg <= kSegCache && n_win <= kWinCap;
    int cta_count = 0;
    // Lists longer than shared memory holds continue in the run's own part of the staging buffers (one entry per
    // element of the run at most; the first half takes the unordered list, the second the ordered one).
    const int run_n = run_e1 - run_e0;
    int* const g_uidx = A.stage_idx + run_e0;
    float* const g_uval = A.stage_val + run_e0;
    int* const g_oidx = A.stage_idx + run_e0 + run_n / 2;
    float* const g_oval = A.stage_val + run_e0 + run_n / 2;
    const int list_cap = max(kOutCache, run_n / 2 - 8);           // denser selections go the other way

    // Survivors into the run's unordered list (path A).  reserve(): room for n survivors that lie in one
    // 1024-element window and one segment (one atomic each on the list, the window and the segment counter,
    // whatever n); put(): one of them at its reserved place.
    auto reserve = [&](int n, int e_any, int seg_i) -> int {
        if (SIDCO_IN_RANGE(A, (e_any >> 10) - win0, n_win)) atomicAdd(&sm_wcnt[(e_any >> 10) - win0], n);
        if (SIDCO_IN_RANGE(A, seg_i, kSegCache)) atomicAdd(&sm_segk[seg_i], n);
        return atomicAdd(&sm_nsurv, n);
    };
    auto put = [&](int sp, int e, float val) {
        if (sp < kOutCache) { sm_oidx[sp] = e; sm_oval[sp] = val; }
        else if (sp < list_cap) { g_uidx[sp - kOutCache] = e; g_uval[sp - kOutCache] = val; }
    };

    // The warps' pass over chunks.  list_n >= 0: the chunks sm_rest[0 .. list_n); < 0: all chunks of the run,
    // skipping (if skip_covered) those whose survivors the candidates already gave.  to_list: survivors go to the
    // shared-memory list and nothing is modified; otherwise they are staged per chunk and zeroed in the residual.
    auto warp_pass = [&](int list_n, bool skip_covered, bool to_list) -> int {
        int total = 0;
        SegView sv;
        bool seg_from_side = false, seg_cand = false, seg_covered = false;
        int seg_count = 0;       // survivors of sv.seg not yet added to its counter (staging mode)
        const bool any_side = M_max_eff >= 2;      // some chunk of this run may have a side region
        auto next_chunk = [&]() -> int { return list_n >= 0 ? queue.next_listed(sm_rest, list_n) : queue.next(!p1_desc); };
        auto add_seg_count = [&](int seg, int n) {
            const int i = seg - R.seg_lo;
            if (i < kSegCache) atomicAdd(&sm_segk[i], n);
            else atomicAdd(&A.seg[seg].k_acc, n);
        };
        Desc cur = fetch_desc(A, list_n == 0 ? -1 : next_chunk(), any_side);
        while (cur.c >= 0) {
            const Desc nxt = fetch_desc(A, next_chunk(), any_side);
            if (cur.seg != sv.seg) {
                if (seg_count && lane == 0) add_seg_count(sv.seg, seg_count);
                seg_count = 0;
                view_load(A, R, sv, cur.seg, 0, -1, 100, cap);
                const int i = cur.seg - R.seg_lo;
                seg_cand = spec_tau(cur.seg) > 0.0f;               // its full chunks recorded candidates
                seg_from_side = sv.M_eff >= 2;
                seg_covered = i < kSegCache && seg_cand && seg_cand_ok(i);
            }
            const int c = cur.c, lo = cur.lo, hi = cur.hi;
            const int wb = lo & ~(kChunk - 1);
            const float wt = (lo == wb && hi == wb + kChunk) ? sc_tau_of(wb) : 0.0f;
            const bool cand_chunk = (seg_cand && vec_ok && ((lo | hi) & (kComp - 1)) == 0) || wt > 0.0f;
            int cnt = 0;
            const bool chunk_ok = SIDCO_IN_RANGE(A, c, A.C) && SIDCO_IN_RANGE(A, lo, A.d) && SIDCO_IN_RANGE(A, hi - 1, A.d);
            const bool covered = wt > 0.0f ? sv.thr_ge >= wt : seg_covered;
            if (chunk_ok && !(skip_covered && cand_chunk && covered)) {
                unsigned surv = 0;
                float v[kSlots][kComp];
                // a whole-slot chunk of a candidate-recording two-stage segment has no side region: it is read from acc
                const bool from_side = seg_from_side && !cand_chunk;
                if (from_side) {
                    // The side region is a dense list in index order.  Lanes read it 16 bytes at a time; a survivor
                    // is known by its position in the list, and the lane that holds the element at that position
                    // (found through the per-lane masks, only for chunks that have a survivor at all) marks it
                    // in a mask of the chunk's own layout, which gives the survivors their indices and order.
                    const int n = SIDCO_IN_RANGE(A, cur.side_n, kChunk + 1) ? cur.side_n : 0;
                    const float4* side = reinterpret_cast<const float4*>(A.side_val + (size_t)c * kChunk) + lane;
                    int pos[kSlots], base[kSlots];
                    unsigned smask = 0;
                    bool have_pos = false;
                    auto take = [&](const float4& x, int first) {
                        const float a[4] = {fabsf(x.x), fabsf(x.y), fabsf(x.z), fabsf(x.w)};
                        unsigned hit = 0;
                        #pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (first + u < n && a[u] >= sv.thr_ge) hit |= 1u << u;
                        unsigned any = __ballot_sync(kFull, hit != 0);
                        if (any == 0) return;
                        if (!have_pos) {
                            smask = __ldcg(A.side_mask + (size_t)c * 32 + lane);
                            side_positions(smask, pos, base);
                            have_pos = true;
                        }
                        while (any) {
                            const int src = __ffs(any) - 1;
                            any &= any - 1u;
                            unsigned h = __shfl_sync(kFull, hit, src);
                            const int base = __shfl_sync(kFull, first, src);
                            while (h) {
                                const int p = base + __ffs(h) - 1;         // position in the list
                                h &= h - 1u;
                                // the lane whose elements of some slot cover position p
                                #pragma unroll
                                for (int j = 0; j < kSlots; ++j) {
                                    const unsigned byte = (smask >> (8 * j)) & 0xFFu;
                                    const int r = p - pos[j];
                                    if (r >= 0 && r < __popc(byte)) surv |= (1u << (8 * j)) << (__fns(byte, 0, r + 1));
                                }
                            }
                        }
                    };
                    #pragma unroll
                    for (int u = 0; u < kSidePre; ++u) take(cur.pre[u], 128 * u + 4 * lane);
                    for (int t = kSidePre; 128 * t < n; ++t) take(__ldcg(side + 32 * t), 128 * t + 4 * lane);
                } else {
                    ++resweep;
                    const unsigned valid = load_chunk(A.residual, lo, hi, wb, vec_ok, true, v);
                    #pragma unroll
                    for (int j = 0; j < kSlots; ++j)
                        #pragma unroll
                        for (int cc = 0; cc < kComp; ++cc)
                            if (fabsf(v[j][cc]) >= sv.thr_ge) surv |= 1u << (8 * j + cc);
                    surv &= valid;
                }
                if (__ballot_sync(kFull, surv != 0)) {
                    const int e0 = wb + lane * kComp;
                    if (to_list) {
                        const int seg_i = cur.seg - R.seg_lo;
                        unsigned m = surv;
                        int sp = m ? reserve(__popc(m), wb, seg_i) : 0;       // (a chunk lies in one window)
                        while (m) {
                            const int bit = __ffs(m) - 1;
                            m &= m - 1u;
                            const int e = e0 + (bit >> 3) * 256 + (bit & 7);
                            if (SIDCO_IN_RANGE(A, e, A.d)) put(sp, e, __ldcg(A.residual + e));
                            ++sp;
                        }
                    } else {
                        cnt = ordered_emit(surv, lo, [&](int p, int j, int cc) {
                            const int e = e0 + j * 256 + cc;
                            if (!SIDCO_IN_RANGE(A, p, A.d) || !SIDCO_IN_RANGE(A, e, A.d)) return;
                            A.stage_idx[p] = e;
                            A.stage_val[p] = from_side ? __ldcg(A.residual + e) : v[j][cc];
                            A.residual[e] = 0.0f;
                        });
                    }
                }
            }
            if (!to_list) {
                if (lane == 0) A.chunk_cnt[c] = cnt;
                seg_count += cnt;
                total += cnt;
            }
            cur = nxt;
        }
        if (seg_count && lane == 0) add_seg_count(sv.seg, seg_count);
        return total;
    };

    if (path_a) {
        for (int w = threadIdx.x; w < n_win; w += kThreads) { sm_wcnt[w] = 0; sm_wfill[w] = 0; }
        // A segment that recorded candidates which turned out unusable (its threshold fell below the candidate
        // threshold): its chunks made of whole slots are in no list yet.  (A first or last chunk that is not
        // recorded no candidates and was listed by the sweep.)
        if (vec_ok) {
            // (such segments are rare: they are collected first, then all threads list their chunks)
            for (int i = threadIdx.x; i < R.n_seg; i += kThreads)
                if (sm_q1[i] > sm_q0[i] && sm_tau[i] > 0.0f && !seg_cand_ok(i)) sm_list[atomicAdd(&sm_count[0], 1)] = i;
            __syncthreads();
            const int n_bad = sm_count[0];
            for (int k = 0; k < n_bad; ++k) {
                const int i = sm_list[k];
                const int qa = max(sm_q0[i], c0), qb = min(sm_q1[i], c1);
                for (int c = qa + (int)threadIdx.x; c < qb; c += kThreads) {
                    const int lo = __ldg(A.chunk_start + c), hi = __ldg(A.chunk_start + c + 1);
                    if (((lo | hi) & (kComp - 1)) == 0) {
                        const int q = atomicAdd(&sm_nrest, 1);
                        if (q < kThreads) sm_rest[q] = c - c0;
                    }
                }
            }
            // likewise a full chunk whose warp estimated too high
            if (sc_on)
                for (int w = threadIdx.x; w < n_win; w += kThreads) {
                    const float t = sm_wtau[w];
                    if (t > 0.0f && !(R.thr[sm_wseg[w]] >= t)) {
                        const int q = atomicAdd(&sm_nrest, 1);
                        if (q < kThreads) sm_rest[q] = sm_wchunk[w];
                    }
                }
            __syncthreads();
            if (threadIdx.x == 0) sm_count[0] = 0;
        }
        __syncthreads();
        // The few listed chunks that are made of whole slots join the candidates, slot by slot and without
        // condition (this keeps them out of the warps' pass, whose set-up costs more than the comparisons here).
        const int n_cand = sm_nslot, n_rest0 = sm_nrest;
        const int n_pre = sm_nfetched;          // candidates whose values were copied to shared memory
        __syncthreads();
        if (vec_ok && n_rest0 > 0 && n_rest0 <= kThreads && n_cand + (kChunk / kComp) * n_rest0 <= kSlotCap) {
            for (int r = warp; r < n_rest0; r += kWarps) {
                const int c = c0 + sm_rest[r];
                const int lo = __ldg(A.chunk_start + c), hi = __ldg(A.chunk_start + c + 1);
                if (((lo | hi) & (kComp - 1)) == 0) {
                    const int seg_i = __ldg(A.chunk_seg + c) - R.seg_lo;
                    #pragma unroll
                    for (int j = 0; j < kSlots; ++j) {
                        const int e = (lo & ~(kChunk - 1)) + lane * kComp + j * 256;
                        if (e >= lo && e + kComp <= hi) list_slot(e, seg_i);
                    }
                } else if (lane == 0) {
                    sm_list[atomicAdd(&sm_count[0], 1)] = sm_rest[r];
                }
            }
            __syncthreads();
            const int n_keep = sm_count[0];
            if ((int)threadIdx.x < n_keep) sm_rest[threadIdx.x] = sm_list[threadIdx.x];
            __syncthreads();
            if (threadIdx.x == 0) { sm_nrest = n_keep; sm_count[0] = 0; }
            __syncthreads();
        }
        const int n_slot = sm_nslot;
        const size_t spill0 = (size_t)(run_e0 >> 3) + blockIdx.x;
        for (int q = threadIdx.x; q < n_slot; q += kThreads) {
            const int i = q < kSlotCap ? sm_slot_seg[q] : A.slot_spill_seg[spill0 + (q - kSlotCap)];
            const int e = q < kSlotCap ? sm_slot_e[q] : __ldcg(A.slot_spill_e + spill0 + (q - kSlotCap));
            const float thr = R.thr[i];
            const float wt = sm_tau[i] > 0.0f ? 0.0f : sc_tau_of(e);
            if (q >= n_cand || seg_cand_ok(i) || (wt > 0.0f && thr >= wt)) {
                float x[kComp];
                if (q < n_pre) {
                    #pragma unroll
                    for (int cc = 0; cc < kComp; ++cc) x[cc] = sm_slot_val[q * kComp + cc];
                } else {
                    const float4 a = __ldcg(reinterpret_cast<const float4*>(A.residual + e));
                    const float4 b = __ldcg(reinterpret_cast<const float4*>(A.residual + e) + 1);
                    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
                }
                unsigned m = 0;
                #pragma unroll
                for (int cc = 0; cc < kComp; ++cc)
                    if (fabsf(x[cc]) >= thr) m |= 1u << cc;
                if (m) {
                    int sp = reserve(__popc(m), e, i);                       // (a slot lies in one window)
                    #pragma unroll
                    for (int cc = 0; cc < kComp; ++cc)
                        if ((m >> cc) & 1u) put(sp++, e + cc, x[cc]);
                }
            }
        }
        SIDCO_STAMP(if (threadIdx.x == 0 && M_max_eff == 1) A.cta_ns[4 * cta + 2] = global_ns());     // (... and candidates compared)
        const bool scan_all = sm_nrest > kThreads;
        warp_pass(scan_all ? -1 : sm_nrest, true, true);
        __syncthreads();
        cta_count = sm_nsurv;
        if (cta_count > list_cap) {
            // too many for the list: start over the other way (nothing has been modified yet)
            path_a = false;
            for (int i = threadIdx.x; i < kSegCache; i += kThreads) sm_segk[i] = 0;
            if (threadIdx.x == 0) sm_next = 0;
            __syncthreads();
        }
    }
    if (!path_a) {
        const int warp_total = warp_pass(-1, false, false);
        if (lane == 0) sm_warp[warp] = warp_total;
        __syncthreads();
        if (warp == 0) {
            int x = sm_warp[lane];
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(kFull, x, o);
            if (lane == 0) sm_base = x;
        }
        __syncthreads();
        cta_count = sm_base;
    }
    if (lane == 0 && resweep) atomicAdd(&sm_resweep, resweep);
    __syncthreads();
    SIDCO_STAMP(if (threadIdx.x == 0) {
        int* dbg = A.cta_dbg + 8 * cta;
        dbg[0] = path_a; dbg[1] = sm_nslot; dbg[2] = sm_nrest; dbg[3] = cta_count; dbg[4] = sm_resweep + resweep; dbg[5] = c1 - c0;
    });
    SIDCO_STAMP(if (threadIdx.x == 0) A.cta_ns[4 * cta + 3] = global_ns());
    SIDCO_STAMP(if (stamper) A.ctl->t_ns[12] = global_ns());
    // next call: start the first sweep where this call's last full sweep over acc ended
    if (threadIdx.x == 0) A.cta_dir[cta] = (2 * sm_resweep >= c1 - c0) ? (p1_desc ? 1 : 0) : (p1_desc ? 0 : 1);

    // No grid-wide barrier follows.  The run's survivor count is published as one tagged word, which the runs
    // above it poll for their output base; a segment's total count comes out of the atomic by which the last of
    // its runs reports (SegDev::k_arr).  Neither needs a fence: the words carry everything their readers use,
    // and what this CTA stored for its own placement it reads back itself.
    if (threadIdx.x == 0) st_relaxed_u64(&A.cta_pub[cta], ((unsigned long long)call_id << 32) | (unsigned)cta_count);

    // Per-segment end of call: counts, last stage count, adaptation (Algorithm 1, Adapt_Stages), next call's
    // candidate threshold.  Done by the thread whose report completes the segment; reads nothing that another
    // CTA wrote during this call except through that report.
    const bool timed_out = ld_volatile(&A.ctl->timeout) != 0;
    auto seg_finish = [&](int s, int M_eff, int k_hat, float thr) {
        SegDev* sg = &A.seg[s];
        A.out_k[s] = k_hat;
        sg->k_stage[M_eff - 1] = k_hat;
        if (timed_out) atomicOr(&sg->status, (int)kStTimeout);
        if (A.max_stages > 0) {
            const int calls = sg->calls + 1;
            long long k_sum = sg->k_sum + k_hat;
            if (calls % A.Q == 0) {
                const double k_avg = (double)k_sum / (double)A.Q;
                const double k_target = A.delta * (double)A.seg_n[s];
                int M = sg->M;
                const int step = A.pol_adapt_rev ? -1 : 1;
                if (k_avg > k_target * (1.0 + A.eps_H)) M = M - step;
                if (k_avg < k_target * (1.0 - A.eps_L)) M = M + step;
                if (M < 1) M = 1;
                if (M > A.max_stages) M = A.max_stages;
                sg->M = M;
                k_sum = 0;
            }
            sg->calls = calls;
            sg->k_sum = k_sum;
        }
        // (test mode 2 sets it too high on purpose, so that the next call finds its candidates unusable)
        sg->spec_thr = (thr > 0.0f && thr < 3.0e38f) ? (A.spec_enable == 2 ? 1.25f : kSpecRatio) * thr : -1.0f;
    };
    for (int ib = 0; ib < R.n_seg; ib += kThreads) {
        const int i = ib + (int)threadIdx.x;
        if (i < R.n_seg) {
            int q0, q1, runs;
            R.get(A, i, q0, q1, runs);
            if (q1 > q0) {
                const int s = R.seg_lo + i;
                SegDev* sg = &A.seg[s];
                if (i < kSegCache) {
                    const int cnt = sm_segk[i];
                    unsigned long long old = 0ull;
                    if (runs > 1) old = atomicAdd(&sg->k_arr, ((unsigned long long)(unsigned)cnt << 32) | 1ull);
                    if (runs == 1 || (int)(old & 0xFFFFFFFFull) == runs - 1) {
                        if (runs > 1) sg->k_arr = 0ull;
                        seg_finish(s, R.m_eff[i], (int)(old >> 32) + cnt, R.thr[i]);
                    }
                } else {
                    // no shared-memory count: the warps added to k_acc; report (arrival only) after those additions
                    __threadfence();
                    bool last = runs == 1;
                    if (!last) {
                        last = (int)(atomicAdd(&sg->k_arr, 1ull) & 0xFFFFFFFFull) == runs - 1;
                        __threadfence();                   // acquire side: the other runs' additions to k_acc
                    }
                    if (last) {
                        const int k_hat = ld_cg(&sg->k_acc);
                        sg->k_acc = 0;
                        if (runs > 1) sg->k_arr = 0ull;
                        const float thr = __uint_as_float((unsigned)(ld_acquire_u64(&sg->pub) >> 32));
                        seg_finish(s, seg_stages(A, s, cap), k_hat, thr);
                    }
                }
            }
        }
    }

    // Segments without chunks (n = 0) never see an arrival or a report: their defaults and their end of call
    // are done here, spread over the grid.
    for (int s = cta * kThreads + (int)threadIdx.x; s < A.S; s += A.G * kThreads)
        if (A.seg_chunk0[s + 1] == A.seg_chunk0[s]) {
            const Fit f = fit_stage1<SID, EXACT>(A, &A.seg[s], A.seg[s].M, 0, 0.0, 0.0, 0, cap, T);
            record_stage(&A.seg[s], 0, f, 0, 1);
            seg_finish(s, f.M_eff, 0, f.thr);
        }

    // ------------------------------------------------------------------ placement
    {
        // In path A the list is put in index order while the counts of the runs below are on their way: a
        // counting pass groups the survivors by window, then every survivor is ranked inside its window.
        if (path_a && cta_count > 0) {
            // window bases: exclusive prefix sums of the window counts, two windows per thread
            const int w2 = 2 * (int)threadIdx.x;
            const int a0 = w2 < n_win ? sm_wcnt[w2] : 0, a1 = w2 + 1 < n_win ? sm_wcnt[w2 + 1] : 0;
            int total = 0;
            const int ex = block_exscan(a0 + a1, sm_warp, total);
            __syncthreads();
            if (w2 < n_win) sm_wcnt[w2] = ex;
            if (w2 + 1 < n_win) sm_wcnt[w2 + 1] = ex + a0;
            __syncthreads();
            const bool in_smem = cta_count <= kOutCache;
            for (int q0 = 0; q0 < cta_count; q0 += kThreads) {
                const int q = q0 + (int)threadIdx.x;
                const bool on = q < cta_count;
                const int e = on ? (q < kOutCache ? sm_oidx[q] : g_uidx[q - kOutCache]) : 0;
                const int w = on ? (e >> 10) - win0 : -1;
                const float val = on ? (q < kOutCache ? sm_oval[q] : g_uval[q - kOutCache]) : 0.0f;
                // (neighbours in the list mostly share a window: one atomic per window and warp)
                const unsigned peers = __match_any_sync(kFull, w);
                const int leader = __ffs(peers) - 1;
                int first = 0;
                if (on && lane == leader) first = atomicAdd(&sm_wfill[w], __popc(peers));
                first = __shfl_sync(kFull, first, leader);
                if (!on) continue;
                const int slot = sm_wcnt[w] + first + __popc(peers & ((1u << lane) - 1u));
                if (!SIDCO_IN_RANGE(A, slot, in_smem ? kOutCache : run_n - run_n / 2)) continue;
                if (in_smem) { sm_cidx[slot] = e; sm_cval[slot] = val; }      // (the candidate values' space is free by now)
                else { g_oidx[slot] = e; g_oval[slot] = val; }
            }
            __syncthreads();
        }
        // survivors of the runs below this one: each run's word is polled (bounded) until it carries this
        // call's number; summed by one warp (a grid has a few hundred CTAs at most)
        if (warp == 0) {
            int below = 0;
            for (int c = lane; c < cta; c += 32) {
                unsigned long long w;
                long long spins = 0;
                while ((unsigned)((w = ld_relaxed_u64(&A.cta_pub[c])) >> 32) != call_id) {
                    if ((++spins & 15) == 0 && ld_volatile(&A.ctl->timeout)) break;
                    if (spins > A.spin_limit) { atomicExch(&A.ctl->timeout, 1); break; }
                    __nanosleep(spins < 64 ? 20 : 100);
                }
                below += (int)(unsigned)w;
            }
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) below += __shfl_down_sync(kFull, below, o);
            if (lane == 0) sm_base = below;
        }
        __syncthreads();
        SIDCO_STAMP(if (stamper) A.ctl->t_ns[4] = global_ns());
        int run_base = sm_base;
        if (cta == A.G - 1 && threadIdx.x == 0) A.out_k[A.S] = run_base + cta_count;
        if (path_a) {
            const bool in_smem = cta_count <= kOutCache;
            const int* oidx = in_smem ? sm_cidx : g_oidx;
            const float* oval = in_smem ? sm_cval : g_oval;
            constexpr int kDenseWin = 32;       // windows with more survivors are ranked through a bitmap, by one warp
            for (int q = threadIdx.x; q < cta_count; q += kThreads) {
                const int e = oidx[q], w = (e >> 10) - win0;
                const int g0 = sm_wcnt[w], n_w = sm_wfill[w];
                if (n_w > kDenseWin) continue;
                int rank = 0;
                for (int t = g0; t < g0 + n_w; ++t) rank += oidx[t] < e;
                if (!SIDCO_IN_RANGE(A, run_base + g0 + rank, A.d) || !SIDCO_IN_RANGE(A, e, A.d)) continue;
                A.out_idx[run_base + g0 + rank] = e;
                A.out_val[run_base + g0 + rank] = oval[q];
                A.residual[e] = 0.0f;
            }
            // A window with many survivors: its 1024 positions as a bitmap (one word per lane), prefix counts over
            // the words, and every survivor's rank is the number of set bits below its own.
            {
                unsigned* bm = reinterpret_cast<unsigned*>(sm_scan) + warp * 32;
                int* pf = sm_list + warp * 32;
                for (int w = warp; w < n_win; w += kWarps) {
                    const int n_w = sm_wfill[w];
                    if (n_w <= kDenseWin) continue;
                    const int g0 = sm_wcnt[w];
                    bm[lane] = 0u;
                    __syncwarp();
                    for (int t = lane; t < n_w; t += 32) {
                        const int o = oidx[g0 + t] & (kChunk - 1);
                        atomicOr(&bm[o >> 5], 1u << (o & 31));
                    }
                    __syncwarp();
                    const int mine = __popc(bm[lane]);
                    int incl = mine;
                    #pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int t = __shfl_up_sync(kFull, incl, o);
                        if (lane >= o) incl += t;
                    }
                    pf[lane] = incl - mine;
                    __syncwarp();
                    for (int t = lane; t < n_w; t += 32) {
                        const int e = oidx[g0 + t], o = e & (kChunk - 1);
                        const int rank = pf[o >> 5] + __popc(bm[o >> 5] & ((1u << (o & 31)) - 1u));
                        if (!SIDCO_IN_RANGE(A, run_base + g0 + rank, A.d) || !SIDCO_IN_RANGE(A, e, A.d)) continue;
                        A.out_idx[run_base + g0 + rank] = e;
                        A.out_val[run_base + g0 + rank] = oval[g0 + t];
                        A.residual[e] = 0.0f;
                    }
                    __syncwarp();
                }
            }
        }
        // path B: chunk bases by a block-wide exclusive scan, kThreads chunks at a time
        for (int pass = c0; pass < c1 && cta_count > 0 && !path_a; pass += kThreads) {
            const int c = pass + (int)threadIdx.x;
            const int cnt = c < c1 ? ld_cg(A.chunk_cnt + c) : 0;
            int incl = cnt;
            #pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += t;
            }
            __syncthreads();
            if (lane == 31) sm_warp[warp] = incl;
            __syncthreads();
            if (warp == 0) {
                int w = sm_warp[lane];
                #pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFull, w, o);
                    if (lane >= o) w += t;
                }
                sm_warp[lane] = w;          // inclusive over warps
            }
            __syncthreads();
            const int warp_off = warp ? sm_warp[warp - 1] : 0;
            const int pass_total = sm_warp[kWarps - 1];
            sm_scan[threadIdx.x] = run_base + warp_off + incl - cnt;     // exclusive base of chunk c
            __syncthreads();
            // one thread per survivor: the owning chunk is the last one whose base is <= the position
            const int n_here = min(kThreads, c1 - pass);
            for (int p = threadIdx.x; p < pass_total; p += kThreads) {
                const int pos = run_base + p;
                int a = 0, b = n_here;
                while (a < b) {
                    const int mid = (a + b) >> 1;
                    if (sm_scan[mid] <= pos) a = mid + 1; else b = mid;
                }
                const int i = a - 1;
                const int src = __ldg(A.chunk_start + pass + i) + (pos - sm_scan[i]);
                if (!SIDCO_IN_RANGE(A, pos, A.d) || !SIDCO_IN_RANGE(A, src, A.d)) continue;
                A.out_idx[pos] = ld_cg(A.stage_idx + src);
                A.out_val[pos] = ld_cg(A.stage_val + src);
            }
            run_base += pass_total;
            __syncthreads();
        }
    }
    // The CTA that finishes last closes the call: from then on the next call's number is in force.  (Every CTA
    // read the current one at its start, long before it could get here.)
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned done = atomicAdd(&A.ctl->count, 1u) + 1u;
        if (done == call_id * (unsigned)A.G) {
            A.ctl->seq = call_id;
            A.ctl->residual_is_zero = 0;
        }
    }

    SIDCO_STAMP(if (stamper) A.ctl->t_ns[5] = global_ns());
}

// Back to the state of a fresh residual: M = 1, counters and candidate thresholds cleared, the residual
// declared empty.  The published words keep their call tags.
__global__ void sidco_reset_state_kernel(SegDev* seg, int S, Control* ctl) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s == 0) ctl->residual_is_zero = 1;
    if (s < S) {
        seg[s].M = 1;
        seg[s].calls = 0;
        seg[s].k_sum = 0;
        seg[s].spec_thr = -1.0f;
    }
}

}  // namespace sidco
