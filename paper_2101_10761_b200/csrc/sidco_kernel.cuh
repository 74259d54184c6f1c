// Device code of the SIDCo sparsifier for sm_100a.
//
// One persistent cooperative kernel runs the whole call.  The flat vector is cut
// into tiles that never straddle a segment or an 8192-element window; every CTA
// owns one contiguous run of tiles for the whole call, so data a CTA wrote in one
// phase (acc, side buffers) is re-read by the same CTA in the next one.  Phases
// are separated by grid-wide barriers with bounded waits:
//
//   P1  acc = grad + residual (stored over residual) and stage-1 statistics per
//       tile; the CTA that completes a segment's last tile sums the per-tile
//       partials in tile order and fits eta_1 (Corollaries 1.1-1.3)
//   P3  (only if some segment uses M >= 2) exceedances |x| > eta_1 compacted, in
//       order, into the segment's side buffer together with the statistics of the
//       shifted peaks (Lemma 2 / Corollary 2.1); last arriver fits eta_2
//   P4  (m = 3..M) statistics of side-buffer entries above eta_{m-1}; fit eta_m
//   P5a survivors |x| >= eta_M staged per tile in ascending order (from acc for
//       M = 1, from the side buffer otherwise), selected residual entries zeroed
//   P5b CTA bases from the per-CTA totals, staged survivors copied to their final
//       ascending positions, per-segment counts and stage adaptation
//
// Reductions are deterministic: per-thread sequential accumulation, a fixed
// shuffle tree per tile, and a fixed-order sum of per-tile partials, so thresholds
// do not depend on the grid size or on which CTA performs a fit.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sidco {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 8192;                       // window: elements per full tile
constexpr int kSlots = kTile / 4 / kThreads;      // float4 slots per thread per tile (8)
constexpr int kWarpElems = kTile / kWarps;        // contiguous elements per warp (1024)
constexpr int kMaxStages = 8;
constexpr unsigned kFull = 0xffffffffu;
constexpr long long kSpinLimit = 1ll << 22;       // bounded waits: ~1 s with the back-off below

enum { kSidExp = 0, kSidGamma = 1, kSidGpd = 2 };
enum { kStNonFinite = 1, kStDegenerate = 2, kStAllZero = 4, kStTimeout = 8 };

struct SegDev {
    double eta[kMaxStages];
    int32_t k_stage[kMaxStages];
    float thr_gt;        // largest fp32 <= eta of the newest stage: (|x| > thr_gt) == (|x| > eta)
    float thr_ge;        // smallest fp32 >= eta_M:                  (|x| >= thr_ge) == (|x| >= eta_M)
    int32_t M_eff;       // stages used by this call
    int32_t status;
    int32_t arrived;     // tiles of this segment finished in the current phase (self-resetting)
    int32_t M;           // adaptation state: stage count for the next adaptive call
    int32_t calls;
    int32_t pad;
    long long k_sum;
};

struct Control {
    unsigned bar;        // grid barrier arrivals (reset by the last CTA to finish)
    unsigned finished;
    int timeout;         // set when a bounded wait ran out
    int M_max_eff;       // max over segments of M_eff for this call
};

struct Args {
    const float* grad;
    float* residual;
    int32_t* out_idx;
    float* out_val;
    int32_t* out_k;
    // tables (read only during the call)
    const int32_t* tile_start;   // [T + 1]
    const int32_t* tile_seg;     // [T]
    const int32_t* seg_tile0;    // [S + 1]
    const int32_t* seg_n;        // [S]
    const int32_t* cta_tile0;    // [G + 1]
    // scratch
    double* part;                // [T][3] per-tile partial sums
    int32_t* part_n;             // [T] per-tile partial counts
    int32_t* side_cnt;           // [T] stage-2 exceedances stored for the tile
    int32_t* tile_cnt;           // [T] final survivors staged for the tile
    int32_t* side_idx;           // [d]
    float* side_val;             // [d]
    int32_t* stage_idx;          // [d]
    float* stage_val;            // [d]
    int32_t* cta_total;          // [G]
    SegDev* seg;                 // [S]
    Control* ctl;
    // scalars
    double delta, delta1, eps_H, eps_L;
    int Q, sid, max_stages;
    int T, S, G;
    int vec_ok;                  // grad and residual are 16-byte aligned
};

// ----------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------

__device__ __forceinline__ int ld_cg(const int* p) { return __ldcg(p); }
__device__ __forceinline__ float ld_cg(const float* p) { return __ldcg(p); }
__device__ __forceinline__ double ld_cg(const double* p) { return __ldcg(p); }

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ int ld_volatile(const int* p) {
    return *reinterpret_cast<const volatile int*>(p);
}

// Grid-wide barrier number `which` (1-based within the call).  All CTAs of the
// cooperative launch are resident, so the wait normally ends within microseconds;
// it is nevertheless bounded, and a time-out raises Control::timeout, after which
// every later wait returns at once.
__device__ __forceinline__ void grid_barrier(Control* ctl, int G, int which) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&ctl->bar, 1u);
        const unsigned target = (unsigned)which * (unsigned)G;
        long long spins = 0;
        while (ld_acquire(&ctl->bar) < target) {
            if (ld_volatile(&ctl->timeout)) break;
            if (++spins > kSpinLimit) { atomicExch(&ctl->timeout, 1); break; }
            __nanosleep(spins < 64 ? 32 : 200);
        }
        __threadfence();
    }
    __syncthreads();
}

struct RedOut { double a, b, c; int n; };

// Block-wide sums of three doubles and one int with a fixed tree; result valid in thread 0.
__device__ __forceinline__ RedOut block_sum(double a, double b, double c, int n, double (*sm)[4]) {
    #pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_down_sync(kFull, a, o);
        b += __shfl_down_sync(kFull, b, o);
        c += __shfl_down_sync(kFull, c, o);
        n += __shfl_down_sync(kFull, n, o);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();                       // previous use of sm is over
    if (lane == 0) { sm[warp][0] = a; sm[warp][1] = b; sm[warp][2] = c; sm[warp][3] = (double)n; }
    __syncthreads();
    RedOut r{0.0, 0.0, 0.0, 0};
    if (warp == 0) {
        double x = lane < kWarps ? sm[lane][0] : 0.0;
        double y = lane < kWarps ? sm[lane][1] : 0.0;
        double z = lane < kWarps ? sm[lane][2] : 0.0;
        double w = lane < kWarps ? sm[lane][3] : 0.0;
        #pragma unroll
        for (int o = kWarps / 2; o > 0; o >>= 1) {
            x += __shfl_down_sync(kFull, x, o);
            y += __shfl_down_sync(kFull, y, o);
            z += __shfl_down_sync(kFull, z, o);
            w += __shfl_down_sync(kFull, w, o);
        }
        r.a = x; r.b = y; r.c = z; r.n = (int)w;
    }
    return r;
}

// ----------------------------------------------------------------------------
// closed-form fits (thread 0 of the CTA that completed the segment)
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

// Tail ratio of stage m (0-based) out of M: delta_1 for every non-final stage, the rest for the last.
__device__ inline double stage_ratio(double delta, double delta1, int M, int m) {
    if (M == 1) return delta;
    if (m < M - 1) return delta1;
    double p = 1.0;
    for (int i = 0; i < M - 1; ++i) p *= delta1;
    return delta / p;
}

// Corollary 1.3 / Lemma 2: moment-matched generalised Pareto quantile at tail probability `ratio`.
// A variance at rounding-noise level (raw-moment form) is treated as zero: the formula's limit is `mean`.
__device__ inline double gpd_step(double mean, double var, double ratio, int& status) {
    if (!(var > 1e-12 * mean * mean)) { status |= kStDegenerate; return mean; }
    const double R = mean * mean / var;
    const double alpha = 0.5 * (1.0 - R);
    const double beta = 0.5 * mean * (R + 1.0);
    const double t = -alpha * log(ratio);
    if (fabs(t) < 1e-12) return beta * log(1.0 / ratio);
    return (beta / alpha) * expm1(t);
}

// Corollary 1.1 / 2.1.
__device__ inline double exp_step(double mean, double ratio) { return mean * log(1.0 / ratio); }

__device__ inline void publish_eta(SegDev* sg, int m, double eta) {
    sg->eta[m] = eta;
    sg->thr_gt = __double2float_rd(eta);
    sg->thr_ge = __double2float_ru(eta);
}

// Stage 1 from the segment sums: S1 = sum|x|, S2 = sum x^2 (GPD), SL = sum log|x| over the n_nz
// nonzero magnitudes (gamma).
__device__ inline void fit_stage1(const Args& A, SegDev* sg, int n, double S1, double S2_or_SL, int n_nz) {
    int M;
    if (A.max_stages > 0) {
        M = sg->M < 1 ? 1 : sg->M;
        if (M > A.max_stages) M = A.max_stages;
    } else {
        M = -A.max_stages;
    }
    const int cap = stage_cap(A.delta, A.delta1);
    const int M_eff = M < cap ? M : cap;
    int status = 0;
    double eta;
    const double ratio = stage_ratio(A.delta, A.delta1, M_eff, 0);
    if (n == 0) {
        eta = __longlong_as_double(0x7ff0000000000000ll);
    } else if (!isfinite(S1) || !isfinite(S2_or_SL)) {
        status |= kStNonFinite;
        eta = __longlong_as_double(0x7ff8000000000000ll);
    } else if (S1 == 0.0) {
        status |= kStAllZero;
        eta = __longlong_as_double(0x7ff0000000000000ll);
    } else if (A.sid == kSidExp) {
        eta = exp_step(S1 / n, ratio);
    } else if (A.sid == kSidGpd) {
        const double mu = S1 / n;
        eta = gpd_step(mu, S2_or_SL / n - mu * mu, ratio, status);
    } else {
        const double mu = S1 / n_nz;
        const double s = log(mu) - S2_or_SL / n_nz;
        double rz = ratio * n / n_nz;
        if (rz > 1.0) rz = 1.0;
        if (s <= 1e-12) {
            status |= kStDegenerate;
            eta = exp_step(mu, rz);
            if (!(eta > 0.0)) eta = 0.0;
        } else {
            const double alpha = (3.0 - s + sqrt((s - 3.0) * (s - 3.0) + 24.0 * s)) / (12.0 * s);
            const double beta = mu / alpha;
            eta = -beta * (log(rz) + lgamma(alpha));
            if (eta <= 0.0) { status |= kStDegenerate; eta = 0.0; }
        }
    }
    sg->M_eff = M_eff;
    sg->status = status;
    for (int m = 0; m < kMaxStages; ++m) { sg->eta[m] = 0.0; sg->k_stage[m] = 0; }
    // an empty segment takes part in no later phase: all its stage thresholds are set here
    if (n == 0)
        for (int m = 1; m < M_eff; ++m) sg->eta[m] = eta;
    publish_eta(sg, 0, eta);
    atomicMax(&A.ctl->M_max_eff, M_eff);
}

// Stage m (1-based index m >= 1 means eta_{m+1}) from the shifted peaks over eta_m:
// n_e = #{|x| > eta_m}, Sy = sum(|x| - eta_m), Sy2 = sum(|x| - eta_m)^2.
__device__ inline void fit_stage_m(const Args& A, SegDev* sg, int m, int n_e, double Sy, double Sy2) {
    // fields another SM may have written during this call are read through L2
    const double prev = ld_cg(&sg->eta[m - 1]);
    sg->k_stage[m - 1] = n_e;
    double eta = prev;
    if (n_e > 0) {
        const double ratio = stage_ratio(A.delta, A.delta1, ld_cg(&sg->M_eff), m);
        const double ybar = Sy / n_e;
        int status = ld_cg(&sg->status);
        double inc;
        if (A.sid == kSidExp) inc = exp_step(ybar, ratio);
        else inc = gpd_step(ybar, Sy2 / n_e - ybar * ybar, ratio, status);
        sg->status = status;
        eta = prev + inc;
    }
    publish_eta(sg, m, eta);
}

// ----------------------------------------------------------------------------
// tile access
// ----------------------------------------------------------------------------

// Streaming load for data that is read exactly once (the gradient).
__device__ __forceinline__ float4 ld_stream4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float ld_stream1(const float* p) { return __ldcs(p); }

// Load the part [lo, hi) of the window starting at wb from `src` into registers in tile order
// (warp-major, then slot, lane, component).  Returns the validity mask: bit 4*j + c.
__device__ __forceinline__ unsigned load_tile(const float* __restrict__ src, int lo, int hi, int wb, bool vec_ok,
                                              float (&v)[kSlots][4]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int e0 = wb + warp * kWarpElems + lane * 4;
    unsigned valid = 0;
    if (vec_ok && lo == wb && hi == wb + kTile) {
        #pragma unroll
        for (int j = 0; j < kSlots; ++j) {
            const float4 q = *reinterpret_cast<const float4*>(src + e0 + j * 128);
            v[j][0] = q.x; v[j][1] = q.y; v[j][2] = q.z; v[j][3] = q.w;
        }
        return kFull;
    }
    #pragma unroll
    for (int j = 0; j < kSlots; ++j) {
        const int e = e0 + j * 128;
        v[j][0] = v[j][1] = v[j][2] = v[j][3] = 0.0f;
        if (e + 4 <= lo || e >= hi) continue;
        if (vec_ok && e >= lo && e + 4 <= hi) {
            const float4 q = *reinterpret_cast<const float4*>(src + e);
            v[j][0] = q.x; v[j][1] = q.y; v[j][2] = q.z; v[j][3] = q.w;
            valid |= 0xFu << (4 * j);
        } else {
            #pragma unroll
            for (int c = 0; c < 4; ++c)
                if (e + c >= lo && e + c < hi) { v[j][c] = src[e + c]; valid |= 1u << (4 * j + c); }
        }
    }
    return valid;
}

// Warp-ordered emission: calls emit(position, j, c) for every set bit of `mask`, positions counted
// in tile order starting at `base` for this warp.
template <class Emit>
__device__ __forceinline__ void ordered_emit(unsigned mask, int base, Emit emit) {
    const unsigned lt = (1u << (threadIdx.x & 31)) - 1u;
    int run = base;
    #pragma unroll
    for (int j = 0; j < kSlots; ++j) {
        const unsigned nib = (mask >> (4 * j)) & 0xFu;
        if (__ballot_sync(kFull, nib != 0) == 0) continue;
        const int c = __popc(nib);
        const unsigned b0 = __ballot_sync(kFull, c & 1);
        const unsigned b1 = __ballot_sync(kFull, c & 2);
        const unsigned b2 = __ballot_sync(kFull, c & 4);
        int p = run + __popc(b0 & lt) + 2 * __popc(b1 & lt) + 4 * __popc(b2 & lt);
        run += __popc(b0) + 2 * __popc(b1) + 4 * __popc(b2);
        #pragma unroll
        for (int cc = 0; cc < 4; ++cc)
            if (nib & (1u << cc)) { emit(p, j, cc); ++p; }
    }
}

// Exclusive position of this warp among the CTA's warps and the CTA total, from per-warp counts.
__device__ __forceinline__ int warp_bases(int warp_count, int* sm_cnt, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sm_cnt[warp] = warp_count;
    __syncthreads();
    int base = 0, tot = 0;
    #pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const int c = sm_cnt[w];
        if (w < warp) base += c;
        tot += c;
    }
    total = tot;
    return base;
}

// Arrival of one tile of segment `seg`.  Returns true (to the whole CTA) when this was the segment's
// last tile of the phase; the caller then reduces the segment's partials and fits.
__device__ __forceinline__ bool segment_arrive(const Args& A, int seg, int* sm_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const int ntiles = A.seg_tile0[seg + 1] - A.seg_tile0[seg];
        const int old = atomicAdd(&A.seg[seg].arrived, 1);
        const int last = (old == ntiles - 1);
        if (last) { A.seg[seg].arrived = 0; __threadfence(); }
        *sm_flag = last;
    }
    __syncthreads();
    return *sm_flag != 0;
}

// Fixed-order sum of the per-tile partials of a segment (whole CTA); result in thread 0.
__device__ __forceinline__ RedOut segment_sum(const Args& A, int seg, double (*sm)[4]) {
    const int t0 = A.seg_tile0[seg], t1 = A.seg_tile0[seg + 1];
    double a = 0.0, b = 0.0, c = 0.0;
    int n = 0;
    for (int t = t0 + (int)threadIdx.x; t < t1; t += kThreads) {
        a += ld_cg(A.part + 3 * (size_t)t + 0);
        b += ld_cg(A.part + 3 * (size_t)t + 1);
        c += ld_cg(A.part + 3 * (size_t)t + 2);
        n += ld_cg(A.part_n + t);
    }
    return block_sum(a, b, c, n, sm);
}

// ----------------------------------------------------------------------------
// the kernel
// ----------------------------------------------------------------------------

template <int SID>
__global__ void __launch_bounds__(kThreads, 4) sidco_persistent_kernel(const Args A) {
    __shared__ double sm_red[kWarps][4];
    __shared__ int sm_cnt[kWarps];
    __shared__ int sm_flag;
    __shared__ int sm_base;

    const int cta = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t_begin = A.cta_tile0[cta], t_end = A.cta_tile0[cta + 1];
    const bool vec_ok = A.vec_ok != 0;
    int barrier_no = 0;

    // Segments without tiles (n = 0) never see an arrival: give them their defaults here.
    for (int s = cta; s < A.S; s += A.G)
        if (A.seg_tile0[s + 1] == A.seg_tile0[s] && threadIdx.x == 0) fit_stage1(A, &A.seg[s], 0, 0.0, 0.0, 0);

    // ------------------------------------------------------------------ P1
    // Descending tile order: the tiles touched last are the ones P3/P5a read first, which
    // raises the share of acc that is still in L2 when it is read again.
    for (int t = t_end - 1; t >= t_begin; --t) {
        const int lo = A.tile_start[t], hi = A.tile_start[t + 1];
        const int wb = lo & ~(kTile - 1);
        const int seg = A.tile_seg[t];
        const int e0 = wb + warp * kWarpElems + lane * 4;

        double s1 = 0.0, s2 = 0.0, prod = 1.0;
        int esum = 0, nnz = 0;
        auto accumulate = [&](float x) {
            const float a = fabsf(x);
            const double ad = (double)a;
            s1 += ad;
            if (SID == kSidGpd) s2 = fma(ad, ad, s2);
            if (SID == kSidGamma) {
                if (a > 0.0f) {
                    // log|x| = exponent * ln 2 + log(mantissa): exponents are summed as integers,
                    // mantissas multiplied in fp64, one log per tile.
                    const long long bits = __double_as_longlong(ad);
                    esum += (int)(bits >> 52) - 1023;
                    prod *= __longlong_as_double((bits & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
                    ++nnz;
                }
            }
        };

        if (vec_ok && lo == wb && hi == wb + kTile) {
            #pragma unroll
            for (int b = 0; b < kSlots; b += 4) {
                float4 g4[4], r4[4];
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    g4[j] = ld_stream4(A.grad + e0 + (b + j) * 128);
                    r4[j] = *reinterpret_cast<const float4*>(A.residual + e0 + (b + j) * 128);
                }
                #pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float4 a4;
                    a4.x = g4[j].x + r4[j].x; a4.y = g4[j].y + r4[j].y;
                    a4.z = g4[j].z + r4[j].z; a4.w = g4[j].w + r4[j].w;
                    *reinterpret_cast<float4*>(A.residual + e0 + (b + j) * 128) = a4;
                    accumulate(a4.x); accumulate(a4.y); accumulate(a4.z); accumulate(a4.w);
                }
            }
        } else {
            #pragma unroll 1
            for (int j = 0; j < kSlots; ++j) {
                const int e = e0 + j * 128;
                if (e + 4 <= lo || e >= hi) continue;
                if (vec_ok && e >= lo && e + 4 <= hi) {
                    const float4 g = ld_stream4(A.grad + e);
                    const float4 r = *reinterpret_cast<const float4*>(A.residual + e);
                    float4 a4;
                    a4.x = g.x + r.x; a4.y = g.y + r.y; a4.z = g.z + r.z; a4.w = g.w + r.w;
                    *reinterpret_cast<float4*>(A.residual + e) = a4;
                    accumulate(a4.x); accumulate(a4.y); accumulate(a4.z); accumulate(a4.w);
                } else {
                    for (int c = 0; c < 4; ++c) {
                        if (e + c >= lo && e + c < hi) {
                            const float a = ld_stream1(A.grad + e + c) + A.residual[e + c];
                            A.residual[e + c] = a;
                            accumulate(a);
                        }
                    }
                }
            }
        }

        // per-tile partials
        double pb = s2;
        if (SID == kSidGamma) {
            // normalise the per-thread product, multiply mantissas across the CTA (fixed tree),
            // then one log: SL_tile = esum * ln2 + log(product)
            long long bits = __double_as_longlong(prod);
            esum += (int)(bits >> 52) - 1023;
            double m = __longlong_as_double((bits & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
            #pragma unroll
            for (int o = 16; o > 0; o >>= 1) m *= __shfl_down_sync(kFull, m, o);
            __syncthreads();
            if (lane == 0) sm_red[warp][0] = m;
            __syncthreads();
            double mm = 1.0;
            if (threadIdx.x == 0) {
                #pragma unroll
                for (int w = 0; w < kWarps; ++w) mm *= sm_red[w][0];
            }
            pb = mm;     // thread 0 only; converted after the integer sum below
        }
        RedOut r = block_sum(s1, SID == kSidGamma ? 0.0 : pb, (double)esum, nnz, sm_red);
        if (threadIdx.x == 0) {
            double second = r.b;
            if (SID == kSidGamma) second = r.c * 0.693147180559945309417232121458 + log(pb);
            A.part[3 * (size_t)t + 0] = r.a;
            A.part[3 * (size_t)t + 1] = second;
            A.part[3 * (size_t)t + 2] = 0.0;
            A.part_n[t] = r.n;
        }
        if (segment_arrive(A, seg, &sm_flag)) {
            RedOut sres = segment_sum(A, seg, sm_red);
            if (threadIdx.x == 0) fit_stage1(A, &A.seg[seg], A.seg_n[seg], sres.a, sres.b, sres.n);
        }
    }
    grid_barrier(A.ctl, A.G, ++barrier_no);
    const int M_max_eff = ld_volatile(&A.ctl->M_max_eff);

    // ------------------------------------------------------------------ P3: stage 2 from acc
    if (M_max_eff >= 2) {
        for (int t = t_begin; t < t_end; ++t) {
            const int seg = A.tile_seg[t];
            const SegDev* sg = &A.seg[seg];
            if (ld_cg(&sg->M_eff) < 2) continue;
            const int lo = A.tile_start[t], hi = A.tile_start[t + 1];
            const int wb = lo & ~(kTile - 1);
            const float thr = ld_cg(&sg->thr_gt);
            const double eta_prev = ld_cg(&sg->eta[0]);
            float v[kSlots][4];
            const unsigned valid = load_tile(A.residual, lo, hi, wb, vec_ok, v);
            unsigned mask = 0;
            double sy = 0.0, sy2 = 0.0;
            #pragma unroll
            for (int j = 0; j < kSlots; ++j)
                #pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (fabsf(v[j][c]) > thr) mask |= 1u << (4 * j + c);
            mask &= valid;
            #pragma unroll
            for (int j = 0; j < kSlots; ++j)
                #pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (mask & (1u << (4 * j + c))) {
                        const double y = (double)fabsf(v[j][c]) - eta_prev;
                        sy += y;
                        if (SID != kSidExp) sy2 = fma(y, y, sy2);
                    }
            const int wcnt = __reduce_add_sync(kFull, __popc(mask));
            int total;
            const int wbase = warp_bases(wcnt, sm_cnt, total);
            const int e0 = wb + warp * kWarpElems + lane * 4;
            ordered_emit(mask, lo + wbase, [&](int p, int j, int c) {
                A.side_idx[p] = e0 + j * 128 + c;
                A.side_val[p] = v[j][c];
            });
            RedOut r = block_sum(sy, sy2, 0.0, 0, sm_red);
            if (threadIdx.x == 0) {
                A.part[3 * (size_t)t + 0] = r.a;
                A.part[3 * (size_t)t + 1] = r.b;
                A.part_n[t] = total;
                A.side_cnt[t] = total;
            }
            if (segment_arrive(A, seg, &sm_flag)) {
                RedOut sres = segment_sum(A, seg, sm_red);
                if (threadIdx.x == 0) fit_stage_m(A, &A.seg[seg], 1, sres.n, sres.a, sres.b);
            }
        }
        grid_barrier(A.ctl, A.G, ++barrier_no);

        // -------------------------------------------------------------- P4: stages 3..M from the side buffer
        for (int m = 2; m < M_max_eff; ++m) {
            for (int t = t_begin; t < t_end; ++t) {
                const int seg = A.tile_seg[t];
                const SegDev* sg = &A.seg[seg];
                if (ld_cg(&sg->M_eff) <= m) continue;
                const int lo = A.tile_start[t];
                const int wb = lo & ~(kTile - 1);
                const int hi = lo + A.side_cnt[t];
                const float thr = ld_cg(&sg->thr_gt);
                const double eta_prev = ld_cg(&sg->eta[m - 1]);
                float v[kSlots][4];
                const unsigned valid = load_tile(A.side_val, lo, hi, wb, vec_ok, v);
                double sy = 0.0, sy2 = 0.0;
                int cnt = 0;
                #pragma unroll
                for (int j = 0; j < kSlots; ++j)
                    #pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if ((valid & (1u << (4 * j + c))) && fabsf(v[j][c]) > thr) {
                            const double y = (double)fabsf(v[j][c]) - eta_prev;
                            sy += y;
                            if (SID != kSidExp) sy2 = fma(y, y, sy2);
                            ++cnt;
                        }
                RedOut r = block_sum(sy, sy2, 0.0, cnt, sm_red);
                if (threadIdx.x == 0) {
                    A.part[3 * (size_t)t + 0] = r.a;
                    A.part[3 * (size_t)t + 1] = r.b;
                    A.part_n[t] = r.n;
                }
                if (segment_arrive(A, seg, &sm_flag)) {
                    RedOut sres = segment_sum(A, seg, sm_red);
                    if (threadIdx.x == 0) fit_stage_m(A, &A.seg[seg], m, sres.n, sres.a, sres.b);
                }
            }
            grid_barrier(A.ctl, A.G, ++barrier_no);
        }
    }

    // ------------------------------------------------------------------ P5a: stage survivors per tile
    int cta_count = 0;
    for (int t = t_begin; t < t_end; ++t) {
        const int seg = A.tile_seg[t];
        const SegDev* sg = &A.seg[seg];
        const bool from_side = ld_cg(&sg->M_eff) >= 2;
        const int lo = A.tile_start[t];
        const int wb = lo & ~(kTile - 1);
        const int hi = from_side ? lo + A.side_cnt[t] : A.tile_start[t + 1];
        const float thr = ld_cg(&sg->thr_ge);
        float v[kSlots][4];
        const unsigned valid = load_tile(from_side ? A.side_val : A.residual, lo, hi, wb, vec_ok, v);
        unsigned mask = 0;
        #pragma unroll
        for (int j = 0; j < kSlots; ++j)
            #pragma unroll
            for (int c = 0; c < 4; ++c)
                if (fabsf(v[j][c]) >= thr) mask |= 1u << (4 * j + c);
        mask &= valid;
        const int wcnt = __reduce_add_sync(kFull, __popc(mask));
        int total;
        const int wbase = warp_bases(wcnt, sm_cnt, total);
        if (total > 0) {
            const int e0 = wb + warp * kWarpElems + lane * 4;
            ordered_emit(mask, lo + wbase, [&](int p, int j, int c) {
                const int e = e0 + j * 128 + c;
                const int idx = from_side ? A.side_idx[e] : e;
                A.stage_idx[p] = idx;
                A.stage_val[p] = v[j][c];
                A.residual[idx] = 0.0f;
            });
        }
        if (threadIdx.x == 0) A.tile_cnt[t] = total;
        cta_count += total;
    }
    if (threadIdx.x == 0) A.cta_total[cta] = cta_count;
    grid_barrier(A.ctl, A.G, ++barrier_no);

    // ------------------------------------------------------------------ P5b: final positions
    {
        int below = 0;
        for (int c = threadIdx.x; c < cta; c += kThreads) below += ld_cg(A.cta_total + c);
        RedOut r = block_sum(0.0, 0.0, 0.0, below, sm_red);
        if (threadIdx.x == 0) sm_base = r.n;
        __syncthreads();
        int pos = sm_base;
        if (cta == A.G - 1 && threadIdx.x == 0) A.out_k[A.S] = pos + cta_count;
        for (int t = t_begin; t < t_end; ++t) {
            const int cnt = A.tile_cnt[t];
            const int lo = A.tile_start[t];
            for (int i = threadIdx.x; i < cnt; i += kThreads) {
                A.out_idx[pos + i] = A.stage_idx[lo + i];
                A.out_val[pos + i] = A.stage_val[lo + i];
            }
            pos += cnt;
        }
    }
    // per-segment counts, last stage count, adaptation (Algorithm 1, Adapt_Stages)
    for (int s = cta; s < A.S; s += A.G) {
        const int t0 = A.seg_tile0[s], t1 = A.seg_tile0[s + 1];
        int k = 0;
        for (int t = t0 + (int)threadIdx.x; t < t1; t += kThreads) k += ld_cg(A.tile_cnt + t);
        RedOut r = block_sum(0.0, 0.0, 0.0, k, sm_red);
        if (threadIdx.x == 0) {
            SegDev* sg = &A.seg[s];
            const int k_hat = r.n;
            A.out_k[s] = k_hat;
            sg->k_stage[ld_cg(&sg->M_eff) - 1] = k_hat;
            if (ld_volatile(&A.ctl->timeout)) sg->status = ld_cg(&sg->status) | kStTimeout;
            if (A.max_stages > 0) {
                int calls = sg->calls + 1;
                long long k_sum = sg->k_sum + k_hat;
                if (calls % A.Q == 0) {
                    const double k_avg = (double)k_sum / (double)A.Q;
                    const double k_target = A.delta * (double)A.seg_n[s];
                    int M = sg->M;
                    if (k_avg > k_target * (1.0 + A.eps_H)) M = M - 1;
                    if (k_avg < k_target * (1.0 - A.eps_L)) M = M + 1;
                    if (M < 1) M = 1;
                    if (M > A.max_stages) M = A.max_stages;
                    sg->M = M;
                    k_sum = 0;
                }
                sg->calls = calls;
                sg->k_sum = k_sum;
            }
        }
    }

    // last CTA out resets the control block for the next call
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned done = atomicAdd(&A.ctl->finished, 1u);
        if (done == (unsigned)A.G - 1u) {
            A.ctl->bar = 0u;
            A.ctl->finished = 0u;
            A.ctl->M_max_eff = 0;
            __threadfence();
        }
    }
}

}  // namespace sidco
