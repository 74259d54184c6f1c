// The two compressors the paper measures its own against, on the same inputs and behind the same kind of
// call (Section 1 and Fig. 1: exact Top-k selection, and the sampled threshold of Deep Gradient Compression),
// written for sm_100a so that the comparison can be made on one machine.  They are reference points, not the
// product: plain multi-kernel implementations, each pass a bandwidth-bound sweep.
//
// Both start with the error-compensation add acc = grad + residual (stored over the residual), select on the
// magnitudes compared as the bit patterns of |acc| (finite < infinite < NaN), emit ascending (index, value)
// pairs and zero the selected residual entries.
//
//   Top-k: the k-th largest key is found by a three-level radix select (11 + 11 + 9 bits; the first
//   histogram is fused with the add), then everything above it and the first few equal to it (lowest index
//   first) are written in order through per-block counts, one scan and a block-ordered write.
//   Sampled threshold: the keys at the caller's sample positions are gathered, the same radix select finds the
//   ceil(delta n_s)-th largest of them, and every element of the vector reaching that key is written.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sidco.h"
#include "sidco_internal.h"

namespace sidco_ref {

constexpr int kThreads = 256;
constexpr int kBlockElems = 4096;                 // elements per block of the counting and writing passes
constexpr int kPerThread = kBlockElems / kThreads;
constexpr int kBins = 2048;
constexpr unsigned kFull = 0xffffffffu;

struct State {
    unsigned prefix;        // bits of the k-th largest key fixed so far (aligned to the key's top)
    unsigned long long k;   // rank still to find among the keys matching the prefix (1-based from the top)
    unsigned key;           // the threshold key once all levels are done
    unsigned long long take_eq;   // how many elements equal to the key are selected (lowest index first)
    int level;
};

__device__ __forceinline__ unsigned key_of(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// Level l looks at `bits` bits starting `shift` bits from the bottom, among keys whose higher bits equal the prefix.
__device__ __forceinline__ void level_bits(int level, int& shift, int& bits) {
    if (level == 0) { shift = 20; bits = 11; }
    else if (level == 1) { shift = 9; bits = 11; }
    else { shift = 0; bits = 9; }
}

// acc = grad + residual over the residual, optionally with the level-0 histogram of the keys.
__global__ void __launch_bounds__(kThreads) ec_add_kernel(const float* __restrict__ grad, float* __restrict__ residual,
                                                         long long d, unsigned* hist) {
    __shared__ unsigned sh[kBins];
    if (hist) for (int i = threadIdx.x; i < kBins; i += kThreads) sh[i] = 0u;
    __syncthreads();
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < d; i += stride) {
        const float a = __ldcs(grad + i) + residual[i];
        residual[i] = a;
        if (hist) atomicAdd(&sh[key_of(a) >> 20], 1u);
    }
    __syncthreads();
    if (hist) for (int i = threadIdx.x; i < kBins; i += kThreads) if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// keys[i] = |x[pos[i]]| for the sample, with the level-0 histogram.
__global__ void __launch_bounds__(kThreads) gather_kernel(const float* __restrict__ x, const int32_t* __restrict__ pos,
                                                          long long n, long long d, float* out, unsigned* hist) {
    __shared__ unsigned sh[kBins];
    for (int i = threadIdx.x; i < kBins; i += kThreads) sh[i] = 0u;
    __syncthreads();
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
        const long long p = pos[i];
        const float a = (p >= 0 && p < d) ? x[p] : 0.0f;          // a position outside the vector counts as a zero
        out[i] = a;
        atomicAdd(&sh[key_of(a) >> 20], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += kThreads) if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// Histogram of the next digit among the keys that match the prefix found so far.
__global__ void __launch_bounds__(kThreads) hist_kernel(const float* __restrict__ x, long long n, const State* st,
                                                        unsigned* hist) {
    __shared__ unsigned sh[kBins];
    for (int i = threadIdx.x; i < kBins; i += kThreads) sh[i] = 0u;
    __syncthreads();
    int shift, bits;
    level_bits(st->level, shift, bits);
    const unsigned prefix = st->prefix, mask = (1u << bits) - 1u;
    const int above = shift + bits;                   // bits above this digit are fixed (above < 32)
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
        const unsigned key = key_of(x[i]);
        if ((key >> above) == (prefix >> above)) atomicAdd(&sh[(key >> shift) & mask], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += kThreads) if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// One block: walk the histogram from the top to the bin that holds the rank still sought; fix that digit.
__global__ void __launch_bounds__(kBins / 2) pick_kernel(State* st, unsigned* hist) {
    __shared__ unsigned long long above[kBins / 2];
    __shared__ int found;
    int shift, bits;
    level_bits(st->level, shift, bits);
    const int n_bins = 1 << bits;
    const int t = threadIdx.x;                         // pairs of bins, from the top: pair t = bins n-1-2t, n-2-2t
    const int b_hi = n_bins - 1 - 2 * t, b_lo = b_hi - 1;
    const unsigned long long h_hi = b_hi >= 0 ? hist[b_hi] : 0ull, h_lo = b_lo >= 0 ? hist[b_lo] : 0ull;
    // inclusive prefix sums over the pairs (Hillis-Steele in shared memory)
    above[t] = h_hi + h_lo;
    if (t == 0) found = -1;
    __syncthreads();
    for (int o = 1; o < kBins / 2; o <<= 1) {
        const unsigned long long add = t >= o ? above[t - o] : 0ull;
        __syncthreads();
        above[t] += add;
        __syncthreads();
    }
    const unsigned long long k = st->k;
    const int level = st->level;
    __syncthreads();                                                  // (everybody has read the state)
    const unsigned long long before = above[t] - (h_hi + h_lo);      // keys in bins above this pair
    if (before < k && k <= above[t]) {
        const bool in_hi = k <= before + h_hi;
        const int bin = in_hi ? b_hi : b_lo;
        const unsigned long long k_rem = in_hi ? k - before : k - before - h_hi;
        st->prefix |= (unsigned)bin << shift;
        st->k = k_rem;
        found = bin;
        if (level == 2) { st->key = st->prefix; st->take_eq = k_rem; }
    }
    __syncthreads();
    for (int i = t; i < kBins; i += kBins / 2) hist[i] = 0u;       // ready for the next level
    if (t == 0) {
        if (found < 0) { st->key = 0xffffffffu; st->take_eq = 0ull; }      // fewer keys than the rank: nothing qualifies
        st->level = level + 1;
    }
}

// Per block of kBlockElems elements: how many keys lie above the threshold key and how many equal it.
__global__ void __launch_bounds__(kThreads) count_kernel(const float* __restrict__ acc, long long d, const State* st,
                                                         unsigned* cnt_gt, unsigned* cnt_eq) {
    const unsigned T = st->key;
    const long long base = (long long)blockIdx.x * kBlockElems;
    unsigned gt = 0, eq = 0;
    #pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
        const long long i = base + u * kThreads + threadIdx.x;
        if (i < d) {
            const unsigned key = key_of(acc[i]);
            gt += key > T;
            eq += key == T;
        }
    }
    gt = __reduce_add_sync(kFull, gt);
    eq = __reduce_add_sync(kFull, eq);
    __shared__ unsigned s_gt[kThreads / 32], s_eq[kThreads / 32];
    if ((threadIdx.x & 31) == 0) { s_gt[threadIdx.x >> 5] = gt; s_eq[threadIdx.x >> 5] = eq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned a = 0, b = 0;
        for (int w = 0; w < kThreads / 32; ++w) { a += s_gt[w]; b += s_eq[w]; }
        cnt_gt[blockIdx.x] = a;
        cnt_eq[blockIdx.x] = b;
    }
}

// One block: output base of every block and the equal keys that lie before it; the total count.
__global__ void __launch_bounds__(1024) scan_kernel(const unsigned* cnt_gt, const unsigned* cnt_eq, int n_blocks,
                                                    const State* st, unsigned long long* base_out,
                                                    unsigned long long* base_eq, int32_t* out_k) {
    __shared__ unsigned long long s_a[1024], s_b[1024];
    __shared__ unsigned long long carry_a, carry_b;
    const unsigned long long take = st->take_eq;
    if (threadIdx.x == 0) { carry_a = 0ull; carry_b = 0ull; }
    __syncthreads();
    for (int b0 = 0; b0 < n_blocks; b0 += 1024) {
        const int b = b0 + threadIdx.x;
        const unsigned long long g = b < n_blocks ? cnt_gt[b] : 0ull, e = b < n_blocks ? cnt_eq[b] : 0ull;
        s_a[threadIdx.x] = g;
        s_b[threadIdx.x] = e;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const unsigned long long xa = threadIdx.x >= o ? s_a[threadIdx.x - o] : 0ull;
            const unsigned long long xb = threadIdx.x >= o ? s_b[threadIdx.x - o] : 0ull;
            __syncthreads();
            s_a[threadIdx.x] += xa;
            s_b[threadIdx.x] += xb;
            __syncthreads();
        }
        if (b < n_blocks) {
            const unsigned long long gt_before = carry_a + s_a[threadIdx.x] - g;
            const unsigned long long eq_before = carry_b + s_b[threadIdx.x] - e;
            base_eq[b] = eq_before;
            base_out[b] = gt_before + (eq_before < take ? eq_before : take);
        }
        __syncthreads();
        if (threadIdx.x == 1023) { carry_a += s_a[1023]; carry_b += s_b[1023]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const unsigned long long total = carry_a + (carry_b < take ? carry_b : take);
        out_k[0] = (int32_t)total;
    }
}

// Per block, in index order: the selected elements to their places, their residual entries to zero.
__global__ void __launch_bounds__(kThreads) write_kernel(float* __restrict__ acc, long long d, const State* st,
                                                         const unsigned long long* base_out,
                                                         const unsigned long long* base_eq, int32_t* out_idx,
                                                         float* out_val) {
    __shared__ unsigned s_w[kThreads / 32];
    const unsigned T = st->key;
    const unsigned long long take = st->take_eq;
    const long long first = (long long)blockIdx.x * kBlockElems + (long long)threadIdx.x * kPerThread;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // every thread owns kPerThread consecutive elements, so thread order is index order
    float v[kPerThread];
    unsigned eq_mask = 0, gt_mask = 0;
    #pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
        const long long i = first + u;
        v[u] = i < d ? acc[i] : 0.0f;
        const unsigned key = key_of(v[u]);
        if (i < d && key > T) gt_mask |= 1u << u;
        if (i < d && key == T) eq_mask |= 1u << u;
    }
    auto block_exscan = [&](unsigned x) -> unsigned {
        unsigned incl = x;
        #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += t;
        }
        __syncthreads();
        if (lane == 31) s_w[warp] = incl;
        __syncthreads();
        unsigned off = 0;
        for (int w = 0; w < warp; ++w) off += s_w[w];
        return off + incl - x;
    };
    // which of the equal keys are taken: those whose rank among all equal keys of the vector is below `take`
    const unsigned long long eq_rank0 = base_eq[blockIdx.x] + block_exscan(__popc(eq_mask));
    unsigned sel = gt_mask;
    {
        unsigned long long r = eq_rank0;
        #pragma unroll
        for (int u = 0; u < kPerThread; ++u)
            if ((eq_mask >> u) & 1u) { if (r < take) sel |= 1u << u; ++r; }
    }
    unsigned long long pos = base_out[blockIdx.x] + block_exscan(__popc(sel));
    #pragma unroll
    for (int u = 0; u < kPerThread; ++u)
        if ((sel >> u) & 1u) {
            out_idx[pos] = (int32_t)(first + u);
            out_val[pos] = v[u];
            acc[first + u] = 0.0f;
            ++pos;
        }
}

struct Ws {
    State* st;
    unsigned* hist;
    unsigned* cnt_gt;
    unsigned* cnt_eq;
    unsigned long long* base_out;
    unsigned long long* base_eq;
    float* sample;
    size_t total;
};

Ws layout(void* base, long long d, long long n_sample) {
    const long long n_blocks = (d + kBlockElems - 1) / kBlockElems;
    char* p = (char*)base;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 255) / 256 * 256; return p + at; };
    Ws w;
    w.st = (State*)take(sizeof(State));
    w.hist = (unsigned*)take(sizeof(unsigned) * kBins);
    w.cnt_gt = (unsigned*)take(sizeof(unsigned) * (size_t)(n_blocks + 1));
    w.cnt_eq = (unsigned*)take(sizeof(unsigned) * (size_t)(n_blocks + 1));
    w.base_out = (unsigned long long*)take(sizeof(unsigned long long) * (size_t)(n_blocks + 1));
    w.base_eq = (unsigned long long*)take(sizeof(unsigned long long) * (size_t)(n_blocks + 1));
    w.sample = (float*)take(sizeof(float) * (size_t)(n_sample + 1));
    w.total = o;
    return w;
}

int sweep_grid() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            sms = 148;
    }
    return sms * 8;
}

// Radix select of the rank-th largest key of x[0..n), result left in *st (levels 1 and 2 here; the level-0
// histogram is already in `hist`).
cudaError_t select_rest(const float* x, long long n, const Ws& w, cudaStream_t s, int* launches) {
    pick_kernel<<<1, kBins / 2, 0, s>>>(w.st, w.hist);
    for (int level = 1; level <= 2; ++level) {
        long long g = (n + kThreads - 1) / kThreads;
        if (g > sweep_grid()) g = sweep_grid();
        if (g < 1) g = 1;
        hist_kernel<<<(unsigned)g, kThreads, 0, s>>>(x, n, w.st, w.hist);
        pick_kernel<<<1, kBins / 2, 0, s>>>(w.st, w.hist);
    }
    *launches += 5;
    return cudaGetLastError();
}

// The ordered write of everything above the threshold key and the first take_eq equal to it.
cudaError_t write_selected(float* acc, long long d, const Ws& w, int32_t* out_idx, float* out_val, int32_t* out_k,
                           cudaStream_t s, int* launches) {
    const int n_blocks = (int)((d + kBlockElems - 1) / kBlockElems);
    count_kernel<<<n_blocks, kThreads, 0, s>>>(acc, d, w.st, w.cnt_gt, w.cnt_eq);
    scan_kernel<<<1, 1024, 0, s>>>(w.cnt_gt, w.cnt_eq, n_blocks, w.st, w.base_out, w.base_eq, out_k);
    write_kernel<<<n_blocks, kThreads, 0, s>>>(acc, d, w.st, w.base_out, w.base_eq, out_idx, out_val);
    *launches += 3;
    return cudaGetLastError();
}

int common_checks(const void* grad, const void* residual, int64_t d, const void* out_idx, const void* out_val,
                  const void* out_k, const void* ws, size_t ws_bytes, int64_t n_sample) {
    if (!grad || !residual || !out_idx || !out_val || !out_k || !ws) return SIDCO_E_NULL;
    if (d < 0 || d > (int64_t)2147483647 - 65536 || n_sample < 0) return SIDCO_E_SIZE;
    if (((uintptr_t)ws & 255u) != 0 || ws_bytes < layout(nullptr, d, n_sample).total) return SIDCO_E_WORKSPACE;
    return 0;
}

}  // namespace sidco_ref

extern "C" {

size_t sidco_reference_workspace_bytes(int64_t d, int64_t n_sample) {
    if (d < 0 || n_sample < 0) return 0;
    return sidco_ref::layout(nullptr, d, n_sample).total;
}

int sidco_topk(const float* grad, float* residual, int64_t d, int64_t k, int32_t* out_idx, float* out_val,
               int32_t* out_k, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace sidco_ref;
    int rc = common_checks(grad, residual, d, out_idx, out_val, out_k, workspace, workspace_bytes, 0);
    if (rc) return rc;
    if (k < 0) return SIDCO_E_PARAMS;
    if (k > d) k = d;
    cudaStream_t s = (cudaStream_t)stream;
    const Ws w = layout(workspace, d, 0);
    cudaError_t e;
    State init{0u, (unsigned long long)k, 0xffffffffu, 0ull, 0};
    if ((e = cudaMemsetAsync(w.hist, 0, sizeof(unsigned) * kBins, s)) != cudaSuccess) return (int)e;
    if ((e = cudaMemcpyAsync(w.st, &init, sizeof(State), cudaMemcpyHostToDevice, s)) != cudaSuccess) return (int)e;
    int launches = 0;
    if (d > 0) {
        long long g = (d + kThreads - 1) / kThreads;
        if (g > sweep_grid()) g = sweep_grid();
        ec_add_kernel<<<(unsigned)g, kThreads, 0, s>>>(grad, residual, d, w.hist);
        ++launches;
    }
    if (k == 0 || d == 0) {
        // nothing to select: the key stays above every magnitude
        if ((e = cudaMemsetAsync(out_k, 0, sizeof(int32_t), s)) != cudaSuccess) return (int)e;
    } else {
        if ((e = select_rest(residual, d, w, s, &launches)) != cudaSuccess) return (int)e;
        if ((e = write_selected(residual, d, w, out_idx, out_val, out_k, s, &launches)) != cudaSuccess) return (int)e;
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return (int)e;
    for (int i = 0; i < launches; ++i) sidco_internal::note_launch();
    return 0;
}

int sidco_dgc(const float* grad, float* residual, int64_t d, float delta, const int32_t* sample_idx, int64_t n_sample,
              int32_t* out_idx, float* out_val, int32_t* out_k, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace sidco_ref;
    int rc = common_checks(grad, residual, d, out_idx, out_val, out_k, workspace, workspace_bytes, n_sample);
    if (rc) return rc;
    if (!(delta > 0.0f && delta <= 1.0f)) return SIDCO_E_DELTA;
    if (n_sample > 0 && !sample_idx) return SIDCO_E_NULL;
    cudaStream_t s = (cudaStream_t)stream;
    const Ws w = layout(workspace, d, n_sample);
    cudaError_t e;
    // rank within the sample: ceil(delta * n_s), at least one (the float delta widened to double, as everywhere)
    long long k_s = (long long)((double)delta * (double)n_sample);
    if ((double)k_s < (double)delta * (double)n_sample) ++k_s;
    if (k_s < 1) k_s = 1;
    if (k_s > n_sample) k_s = n_sample;
    // every element reaching the key is taken
    State init{0u, (unsigned long long)k_s, 0xffffffffu, ~0ull, 0};
    if ((e = cudaMemsetAsync(w.hist, 0, sizeof(unsigned) * kBins, s)) != cudaSuccess) return (int)e;
    if ((e = cudaMemcpyAsync(w.st, &init, sizeof(State), cudaMemcpyHostToDevice, s)) != cudaSuccess) return (int)e;
    int launches = 0;
    if (d > 0) {
        long long g = (d + kThreads - 1) / kThreads;
        if (g > sweep_grid()) g = sweep_grid();
        ec_add_kernel<<<(unsigned)g, kThreads, 0, s>>>(grad, residual, d, nullptr);
        ++launches;
    }
    if (n_sample == 0 || d == 0) {
        if ((e = cudaMemsetAsync(out_k, 0, sizeof(int32_t), s)) != cudaSuccess) return (int)e;
    } else {
        long long g = (n_sample + kThreads - 1) / kThreads;
        if (g > sweep_grid()) g = sweep_grid();
        gather_kernel<<<(unsigned)g, kThreads, 0, s>>>(residual, sample_idx, n_sample, d, w.sample, w.hist);
        ++launches;
        if ((e = select_rest(w.sample, n_sample, w, s, &launches)) != cudaSuccess) return (int)e;
        // (select_rest leaves take_eq = the rank inside the last bin: here all equal keys are taken)
        if ((e = cudaMemsetAsync(&w.st->take_eq, 0xff, sizeof(unsigned long long), s)) != cudaSuccess) return (int)e;
        if ((e = write_selected(residual, d, w, out_idx, out_val, out_k, s, &launches)) != cudaSuccess) return (int)e;
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return (int)e;
    for (int i = 0; i < launches; ++i) sidco_internal::note_launch();
    return 0;
}

}  // extern "C"
