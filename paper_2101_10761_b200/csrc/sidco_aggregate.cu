// Aggregation of N workers' sparse gradients into the dense mean (the collective step of the paper's
// sparsified distributed synchronous SGD: G = (1/N) * sum_n Sparsify(g_n, delta)), for sm_100a.
//
// The lists have been gathered into local memory already (padded to a common stride); this kernel turns
// them into the dense vector.  Almost all of the output is zeros, so the kernel is a store stream with a
// sparse correction: every CTA owns a contiguous range of the output; a few of its warps locate the range in
// each worker's ascending index list (warp-wide 32-ary search, both ends at once) while the other warps already
// write zeros over the range; after one CTA barrier the range's entries are copied into shared memory, a bitmap
// over the range finds the positions that more than one worker sent, and the entries are put in place.  Such a
// shared position is written once, by the entry of the first worker that has it: that thread looks the position
// up in the later workers' lists (binary search) and adds their values in worker order in fp64, so the result
// does not depend on scheduling.  (Two CTAs per SM: one CTA's search and merge overlap the other's stores.)
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/sidco.h"
#include "sidco_internal.h"

namespace sidco_agg {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxWorkers = SIDCO_AGG_MAX_WORKERS;
constexpr int kSmemEntries = 6144;             // (index, value) pairs of one CTA range kept in shared memory: 48 KB
constexpr int kMaxRange = 131072;              // elements of one CTA range: two bitmaps of that many bits, 32 KB
constexpr int kDupList = 2048;                 // entries at shared positions worked off as a dense list
constexpr int kFillBlock = 2048;               // elements one warp zero-fills per turn (8 KB)
constexpr unsigned kFull = 0xffffffffu;

struct Args {
    const int32_t* idx_all;      // [n_workers][stride]
    const float* val_all;        // [n_workers][stride]
    const int32_t* counts;       // [n_workers]
    float* out;                  // [d]
    int32_t* status;             // optional
    long long stride, d;
    long long per_cta;           // elements per CTA range (a multiple of kFillBlock, at most kMaxRange)
    int n_workers;
    int vec_ok;                  // out is 16-byte aligned
};

// First position in [a, b) of the ascending list whose index is >= target (b if none), found by the whole
// warp: 32 probes per round.
__device__ __forceinline__ long long warp_lower_bound(const int32_t* __restrict__ list, long long a, long long b,
                                                      long long target) {
    const int lane = threadIdx.x & 31;
    while (b - a > 32) {
        const long long step = (b - a + 31) / 32;
        const long long p = a + lane * step;
        const bool less = p < b && (long long)__ldg(list + p) < target;
        const int m = __popc(__ballot_sync(kFull, less));          // probes below the target: a prefix of the lanes
        if (m == 0) { b = a; break; }
        const long long na = a + (long long)(m - 1) * step + 1;
        const long long nb = a + (long long)m * step;
        a = na;
        b = nb < b ? nb : b;
    }
    const bool less = a + lane < b && (long long)__ldg(list + a + lane) < target;
    return a + __popc(__ballot_sync(kFull, less));
}

// Both ends of a range at once: first positions in [0, n) whose index is >= lo (-> b) and >= hi (-> e).  The two
// searches advance round by round with their probes in flight together.
__device__ __forceinline__ void warp_lower_bound2(const int32_t* __restrict__ list, long long n, long long lo,
                                                  long long hi, long long& b, long long& e) {
    const int lane = threadIdx.x & 31;
    long long a0 = 0, b0 = n, a1 = 0, b1 = n;
    while (b0 - a0 > 32 || b1 - a1 > 32) {
        const bool go0 = b0 - a0 > 32, go1 = b1 - a1 > 32;
        const long long s0 = (b0 - a0 + 31) / 32, s1 = (b1 - a1 + 31) / 32;
        const long long p0 = a0 + lane * s0, p1 = a1 + lane * s1;
        const int v0 = go0 && p0 < b0 ? __ldg(list + p0) : 0x7fffffff;
        const int v1 = go1 && p1 < b1 ? __ldg(list + p1) : 0x7fffffff;
        const int m0 = __popc(__ballot_sync(kFull, go0 && p0 < b0 && (long long)v0 < lo));
        const int m1 = __popc(__ballot_sync(kFull, go1 && p1 < b1 && (long long)v1 < hi));
        if (go0) {
            if (m0 == 0) b0 = a0;
            else { const long long nb = a0 + (long long)m0 * s0; a0 = a0 + (long long)(m0 - 1) * s0 + 1; b0 = nb < b0 ? nb : b0; }
        }
        if (go1) {
            if (m1 == 0) b1 = a1;
            else { const long long nb = a1 + (long long)m1 * s1; a1 = a1 + (long long)(m1 - 1) * s1 + 1; b1 = nb < b1 ? nb : b1; }
        }
    }
    const bool l0 = a0 + lane < b0 && (long long)__ldg(list + a0 + lane) < lo;
    const bool l1 = a1 + lane < b1 && (long long)__ldg(list + a1 + lane) < hi;
    b = a0 + __popc(__ballot_sync(kFull, l0));
    e = a1 + __popc(__ballot_sync(kFull, l1));
    if (e < b) e = b;          // (only a list that is not ascending can get here)
}

// Position of `target` in the ascending list [0, n), or -1.
template <class Ptr>
__device__ __forceinline__ int find_index(Ptr list, int n, int target) {
    int a = 0, b = n;
    while (a < b) {
        const int mid = (a + b) >> 1;
        if (list[mid] < target) a = mid + 1; else b = mid;
    }
    return (a < n && list[a] == target) ? a : -1;
}

__global__ void __launch_bounds__(kThreads, 2) sidco_aggregate_kernel(const __grid_constant__ Args A) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int32_t* s_idx = reinterpret_cast<int32_t*>(smem_raw);
    float* s_val = reinterpret_cast<float*>(s_idx + kSmemEntries);
    unsigned* s_seen = reinterpret_cast<unsigned*>(s_val + kSmemEntries);
    unsigned* s_dup = s_seen + kMaxRange / 32;       // position sent by more than one worker
    __shared__ long long s_begin[kMaxWorkers];       // first entry of the range in worker w's list
    __shared__ int s_cnt[kMaxWorkers];               // entries of the range in worker w's list
    __shared__ int s_off[kMaxWorkers + 1];           // prefix sums of s_cnt
    __shared__ int s_flags, s_next, s_ndup;
    __shared__ int s_duplist[kDupList];              // entries at positions that several workers sent

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long lo = (long long)blockIdx.x * A.per_cta;
    long long hi = lo + A.per_cta;
    if (hi > A.d) hi = A.d;
    if (lo >= hi) return;
    if (threadIdx.x == 0) { s_flags = 0; s_next = 0; s_ndup = 0; }
    for (int i = threadIdx.x; i < 2 * (kMaxRange / 32); i += kThreads) s_seen[i] = 0u;
    __syncthreads();
    const int N = A.n_workers;
    const double n_workers = (double)N;

    // ---- where the range lies in every worker's list: the first warps take workers in turn, each finding both
    // ends of the range at once (the two searches' loads are in flight together)
    for (int w = warp; w < N; w += kWarps) {
        long long cnt = __ldg(A.counts + w);
        int flag = 0;
        if (cnt < 0) { cnt = 0; flag = SIDCO_AGG_ST_COUNT; }
        if (cnt > A.stride) { cnt = A.stride; flag = SIDCO_AGG_ST_COUNT; }
        long long b, e;
        warp_lower_bound2(A.idx_all + (long long)w * A.stride, cnt, lo, hi, b, e);
        if (lane == 0) {
            s_begin[w] = b;
            s_cnt[w] = (int)(e - b);
            if (flag) atomicOr(&s_flags, flag);
        }
    }

    // ---- zeros over the range: warps take 8 KB blocks in turn (the warps that searched join late and take
    // fewer); every store instruction of a warp covers 512 contiguous bytes
    {
        float* out = A.out;
        const int n_blocks = (int)((hi - lo + kFillBlock - 1) / kFillBlock);
        for (;;) {
            int blk = 0;
            if (lane == 0) blk = atomicAdd(&s_next, 1);
            blk = __shfl_sync(kFull, blk, 0);
            if (blk >= n_blocks) break;
            const long long b0 = lo + (long long)blk * kFillBlock;
            const long long b1 = b0 + kFillBlock < hi ? b0 + kFillBlock : hi;
            if (A.vec_ok && b1 - b0 == kFillBlock) {
                float4* o4 = reinterpret_cast<float4*>(out + b0);
                const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
                #pragma unroll
                for (int k = 0; k < kFillBlock / 128; ++k) o4[k * 32 + lane] = z;
            } else {
                for (long long i = b0 + lane; i < b1; i += 32) out[i] = 0.0f;
            }
        }
    }
    __syncthreads();      // the searches are done, and every zero of this range is ordered before the values below

    if (threadIdx.x == 0) {
        int o = 0;
        for (int w = 0; w < N; ++w) { s_off[w] = o; o += s_cnt[w]; }
        s_off[N] = o;
    }
    __syncthreads();
    const int E = s_off[N];
    if (E == 0) {
        if (threadIdx.x == 0 && s_flags && A.status) atomicOr(A.status, s_flags);
        return;
    }
    const bool in_smem = E <= kSmemEntries;
    auto worker_of = [&](int f) -> int {
        int w = 0;
        while (f >= s_off[w + 1]) ++w;
        return w;
    };
    auto entry = [&](int f, int& w, int& idx, float& val) {
        w = worker_of(f);
        if (in_smem) { idx = s_idx[f]; val = s_val[f]; }
        else {
            const long long at = (long long)w * A.stride + s_begin[w] + (f - s_off[w]);
            idx = __ldg(A.idx_all + at);
            val = __ldg(A.val_all + at);
        }
    };
    if (in_smem) {
        // one flat loop over all workers' entries, eight loads in flight per thread
        for (int f0 = threadIdx.x; f0 < E; f0 += 4 * kThreads) {
            int32_t ti[4];
            float tv[4];
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int f = f0 + u * kThreads;
                if (f < E) {
                    const int w = worker_of(f);
                    const long long at = (long long)w * A.stride + s_begin[w] + (f - s_off[w]);
                    ti[u] = __ldg(A.idx_all + at);
                    tv[u] = __ldg(A.val_all + at);
                }
            }
            #pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int f = f0 + u * kThreads;
                if (f < E) { s_idx[f] = ti[u]; s_val[f] = tv[u]; }
            }
        }
        __syncthreads();
    }

    // ---- which positions were sent by more than one worker
    int bad = 0;
    for (int f = threadIdx.x; f < E; f += kThreads) {
        int w, idx;
        float val;
        entry(f, w, idx, val);
        if (idx < lo || idx >= hi) { bad = 1; continue; }          // a list that is not ascending: skipped, reported
        const unsigned r = (unsigned)(idx - lo), bit = 1u << (r & 31);
        if (atomicOr(&s_seen[r >> 5], bit) & bit) atomicOr(&s_dup[r >> 5], bit);
    }
    __syncthreads();

    // ---- the sparse correction, one thread per entry.  A position only one worker sent is that value over N.
    // A position several workers sent is written once, by the entry of the first worker that has it: that
    // thread looks it up in the later workers' lists and adds their values in worker order in fp64.  Those
    // entries are few and scattered over the warps, so they are first collected in a list and then worked off
    // with all lanes busy.
    auto shared_position = [&](int w, int idx, float val) {
        for (int u = 0; u < w; ++u) {
            const int hit = in_smem ? find_index(s_idx + s_off[u], s_cnt[u], idx)
                                    : find_index(A.idx_all + (long long)u * A.stride + s_begin[u], s_cnt[u], idx);
            if (hit >= 0) return;                           // an earlier worker's entry writes this position
        }
        double sum = 0.0 + (double)val;
        for (int u = w + 1; u < N; ++u) {
            if (in_smem) {
                const int hit = find_index(s_idx + s_off[u], s_cnt[u], idx);
                if (hit >= 0) sum += (double)s_val[s_off[u] + hit];
            } else {
                const int32_t* gi = A.idx_all + (long long)u * A.stride + s_begin[u];
                const int hit = find_index(gi, s_cnt[u], idx);
                if (hit >= 0) sum += (double)__ldg(A.val_all + (long long)u * A.stride + s_begin[u] + hit);
            }
        }
        A.out[idx] = (float)(sum / n_workers);
    };
    const bool pow2 = (N & (N - 1)) == 0;
    const float inv_n = 1.0f / (float)N;                    // exact for a power of two
    for (int f = threadIdx.x; f < E; f += kThreads) {
        int w, idx;
        float val;
        entry(f, w, idx, val);
        if (idx < lo || idx >= hi) continue;
        const unsigned r = (unsigned)(idx - lo);
        if ((s_dup[r >> 5] >> (r & 31)) & 1u) {
            const int q = atomicAdd(&s_ndup, 1);
            if (q < kDupList) s_duplist[q] = f;
            else shared_position(w, idx, val);              // (list full: done in place)
        } else {
            // (a power of two divides exactly in fp32, which is what the fp64 quotient rounds to)
            A.out[idx] = pow2 ? (0.0f + val) * inv_n : (float)((0.0 + (double)val) / n_workers);
        }
    }
    __syncthreads();
    const int n_dup = s_ndup < kDupList ? s_ndup : kDupList;
    for (int q = threadIdx.x; q < n_dup; q += kThreads) {
        int w, idx;
        float val;
        entry(s_duplist[q], w, idx, val);
        shared_position(w, idx, val);
    }
    if (bad) atomicOr(&s_flags, SIDCO_AGG_ST_ORDER);
    __syncthreads();
    if (threadIdx.x == 0 && s_flags && A.status) atomicOr(A.status, s_flags);
}

}  // namespace sidco_agg

extern "C" {

int sidco_aggregate(const int32_t* idx_all, const float* val_all, const int32_t* counts, int n_workers,
                    int64_t stride, int64_t d, float* out_dense, int32_t* status, void* stream_v) {
    if (!idx_all || !val_all || !counts || !out_dense) return SIDCO_E_NULL;
    if (n_workers < 1 || n_workers > SIDCO_AGG_MAX_WORKERS) return SIDCO_E_PARAMS;
    if (stride < 0 || d < 0 || d > (int64_t)2147483647 - 65536) return SIDCO_E_SIZE;
    cudaStream_t stream = (cudaStream_t)stream_v;
    cudaError_t e;
    if (status && (e = cudaMemsetAsync(status, 0, sizeof(int32_t), stream)) != cudaSuccess) return (int)e;
    if (d == 0) return 0;
    static int sm_count[64] = {0};
    static std::mutex mu;
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64) return SIDCO_E_SIZE;
    std::lock_guard<std::mutex> lock(mu);
    const size_t smem = (sizeof(int32_t) + sizeof(float)) * sidco_agg::kSmemEntries + 2 * (sidco_agg::kMaxRange / 8);
    if (!sm_count[dev]) {
        int n = 0;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return (int)e;
        if ((e = cudaFuncSetAttribute(sidco_agg::sidco_aggregate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem)) != cudaSuccess)
            return (int)e;
        sm_count[dev] = n;
    }
    sidco_agg::Args a{};
    a.idx_all = idx_all;
    a.val_all = val_all;
    a.counts = counts;
    a.out = out_dense;
    a.status = status;
    a.stride = stride;
    a.d = d;
    a.n_workers = n_workers;
    a.vec_ok = (((uintptr_t)out_dense) & 15u) == 0;
    // two CTAs per SM when the vector is small enough for that; ranges are multiples of the fill block
    long long grid = 2ll * sm_count[dev];
    long long per = (d + grid - 1) / grid;
    per = (per + sidco_agg::kFillBlock - 1) / sidco_agg::kFillBlock * sidco_agg::kFillBlock;
    if (per > sidco_agg::kMaxRange) per = sidco_agg::kMaxRange;
    grid = (d + per - 1) / per;
    a.per_cta = per;
    sidco_agg::sidco_aggregate_kernel<<<(unsigned)grid, sidco_agg::kThreads, smem, stream>>>(a);
    if ((e = cudaGetLastError()) != cudaSuccess) return (int)e;
    sidco_internal::note_launch();
    return 0;
}

}  // extern "C"
