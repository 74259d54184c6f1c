// Host side of the SIDCo sparsifier library: argument checks, chunk tables, workspace,
// per-residual state, and the cooperative launch of the persistent kernel.
#include "sidco_kernel.cuh"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/sidco.h"
#include "sidco_internal.h"

namespace {

using sidco::Args;
using sidco::Control;
using sidco::SegDev;
using sidco::kThreads;
using sidco::kChunk;

struct Params {
    double delta1 = 0.25, eps_H = 0.2, eps_L = 0.2;
    int Q = 5;
    int gamma_exact = 0, ratio_counts = 0, adapt_rev = 0;      // sidco_set_policy
};

struct DeviceInfo {
    int sm_count = 0;
    int ctas_per_sm = 0;     // min over the kernel instantiations
    int grid = 0;            // CTAs per launch (all co-resident)
    bool ready = false;
};

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Offsets of the workspace parts for d elements, S segments, T chunks and G CTAs.
struct Layout {
    size_t chunk_start, chunk_seg, seg_chunk0, seg_n, seg_runs, seg_tile0, tile_arr, tile_part, cta_desc;
    size_t part, part_n, side_cnt, chunk_cnt, side_val, side_mask, stage_idx, stage_val, cta_total, cta_dir, cta_ns, cta_dbg, slot_spill_e, slot_spill_seg, seg, ctl;
    size_t total;
};

Layout make_layout(int64_t d, int S, int64_t T, int G) {
    Layout L{};
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
    L.chunk_start = take(sizeof(int32_t) * (size_t)(T + 1));
    L.chunk_seg = take(sizeof(int32_t) * (size_t)(T + 1));
    L.seg_chunk0 = take(sizeof(int32_t) * (size_t)(S + 1));
    L.seg_n = take(sizeof(int32_t) * (size_t)(S + 1));
    L.seg_runs = take(sizeof(int32_t) * (size_t)(S + 1));
    L.seg_tile0 = take(sizeof(int32_t) * (size_t)(S + 2));
    const size_t tiles = (size_t)(T / sidco::kTile + S + 2);          // upper bound on the tiles of giant segments
    L.tile_arr = take(sizeof(int32_t) * tiles);
    L.tile_part = take(sizeof(double) * 3 * tiles);
    L.cta_desc = take(sizeof(int4) * (size_t)(G + 1));
    L.part = take(sizeof(double) * 3 * (size_t)(T + 1));
    L.part_n = take(sizeof(int32_t) * (size_t)(T + 1));
    L.side_cnt = take(sizeof(int32_t) * (size_t)(T + 1));
    L.chunk_cnt = take(sizeof(int32_t) * (size_t)(T + 1));
    L.side_val = take(sizeof(float) * (size_t)kChunk * (size_t)(T + 1));
    L.side_mask = take(sizeof(unsigned) * 32 * (size_t)(T + 1));
    L.stage_idx = take(sizeof(int32_t) * (size_t)(d + 4));
    L.stage_val = take(sizeof(float) * (size_t)(d + 4));
    L.cta_total = take(sizeof(unsigned long long) * (size_t)(G + 1));
    L.cta_dir = take(sizeof(int32_t) * (size_t)(G + 1));
    L.cta_ns = take(sizeof(unsigned long long) * 4 * (size_t)(G + 1));
    L.cta_dbg = take(sizeof(int) * 8 * (size_t)(G + 1));
    L.slot_spill_e = take(sizeof(int32_t) * (size_t)(d / 8 + G + 8));
    L.slot_spill_seg = take((size_t)(d / 8 + G + 8));
    L.seg = take(sizeof(SegDev) * (size_t)(S + 1));
    L.ctl = take(sizeof(Control));
    L.total = o;
    return L;
}

// Upper bound on the chunk count: every window and every segment start opens at most one chunk.
int64_t max_chunks(int64_t d, int S) { return (d + kChunk - 1) / kChunk + S + 1; }

constexpr int kMaxGrid = 148 * 8 * 2;   // generous bound used only for sizing sidco_workspace_bytes

struct Context {
    int device = -1;
    int64_t d = 0;
    int S = 0, T = 0, G = 0;
    std::vector<int64_t> offsets;          // segment table the device tables were built from
    void* ws = nullptr;
    size_t ws_bytes = 0;
    bool ws_owned = false;
    bool tables_valid = false;
    Layout L{};
    // staging for sidco_compress_host
    float* h_grad = nullptr; float* h_res = nullptr;
    int32_t* h_idx = nullptr; float* h_val = nullptr; int32_t* h_k = nullptr;
    int64_t staging_d = -1; int staging_S = -1;
};

// Switches for tests (sidco_set_test_hooks); the first two start from the environment variables SIDCO_GRID
// (run with fewer CTAs) and SIDCO_SPEC (0: no candidate pre-selection), read once.
struct Hooks {
    int grid = 0;                                  // 0: every CTA the device can hold
    int spec_enable = 1;
    long long spin_limit = sidco::kSpinLimit;
    int drop_pub_seg = -1;
    bool from_env = false;
};
Hooks g_hooks;

Hooks& hooks() {
    if (!g_hooks.from_env) {
        g_hooks.from_env = true;
        if (const char* env = getenv("SIDCO_GRID")) {
            const int want = atoi(env);
            if (want >= 1) g_hooks.grid = want;
        }
        if (const char* env = getenv("SIDCO_SPEC")) g_hooks.spec_enable = env[0] == '0' ? 0 : (env[0] == '2' ? 2 : 1);
    }
    return g_hooks;
}

std::mutex g_mu;
Params g_params;
std::unordered_map<const void*, Context*> g_ctx;
std::unordered_map<int, DeviceInfo> g_dev;
std::atomic<int64_t> g_launches{0};

}  // namespace

void sidco_internal::note_launch() { g_launches.fetch_add(1); }

namespace {

template <int SID, bool EXACT = false>
cudaError_t occupancy(int* out) {
    cudaError_t e = cudaFuncSetAttribute(sidco::sidco_persistent_kernel<SID, EXACT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, sidco::kDynSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(out, sidco::sidco_persistent_kernel<SID, EXACT>, kThreads,
                                                         sidco::kDynSmemBytes);
}

cudaError_t device_info(int dev, DeviceInfo** out) {
    DeviceInfo& di = g_dev[dev];
    if (!di.ready) {
        cudaDeviceProp prop;
        cudaError_t e = cudaGetDeviceProperties(&prop, dev);
        if (e != cudaSuccess) return e;
        if (!prop.cooperativeLaunch) return cudaErrorNotSupported;
        int a = 0, b = 0, c = 0, x = 0;
        if ((e = occupancy<0>(&a)) != cudaSuccess) return e;
        if ((e = occupancy<1>(&b)) != cudaSuccess) return e;
        if ((e = occupancy<2>(&c)) != cudaSuccess) return e;
        if ((e = occupancy<1, true>(&x)) != cudaSuccess) return e;
        int occ = a < b ? a : b;
        occ = occ < c ? occ : c;
        occ = occ < x ? occ : x;
        if (occ < 1) return cudaErrorLaunchOutOfResources;
        di.sm_count = prop.multiProcessorCount;
        di.ctas_per_sm = occ;
        di.grid = di.sm_count * occ;
        di.ready = true;
    }
    *out = &di;
    return cudaSuccess;
}

void free_context(Context* c) {
    if (c->ws_owned && c->ws) cudaFree(c->ws);
    if (c->h_grad) cudaFree(c->h_grad);
    if (c->h_res) cudaFree(c->h_res);
    if (c->h_idx) cudaFree(c->h_idx);
    if (c->h_val) cudaFree(c->h_val);
    if (c->h_k) cudaFree(c->h_k);
    delete c;
}

int check_args(const void* grad, const void* residual, const int64_t* off, int n_segs, float delta, int sid,
               int max_stages, const void* out_idx, const void* out_val, const void* out_k) {
    if (!grad || !residual || !off || !out_idx || !out_val || !out_k) return SIDCO_E_NULL;
    if (n_segs < 1 || off[0] != 0) return SIDCO_E_SEGMENTS;
    for (int s = 0; s < n_segs; ++s)
        if (off[s + 1] < off[s]) return SIDCO_E_SEGMENTS;
    if (off[n_segs] > (int64_t)2147483647 - 65536) return SIDCO_E_SEGMENTS;
    if (!(delta > 0.0f && delta < 1.0f)) return SIDCO_E_DELTA;
    if (sid < 0 || sid > 2) return SIDCO_E_SID;
    if (max_stages == 0 || max_stages > SIDCO_MAX_STAGES || max_stages < -SIDCO_MAX_STAGES) return SIDCO_E_STAGES;
    return 0;
}

// CTAs a launch for this device uses: all that are co-resident, or fewer if a test asked for that.
int launch_grid(const DeviceInfo& di) {
    const int want = hooks().grid;
    return (want >= 1 && want < di.grid) ? want : di.grid;
}

// Host copies of the tables a segment table gives rise to; the arrays are the caller's (sized for
// max_chunks(d, S) + 1 chunks, S + 1 segments and G + 1 CTAs).
struct HostTables {
    int32_t* chunk_start; int32_t* chunk_seg;                  // [T + 1]
    int32_t* seg_chunk0; int32_t* seg_n; int32_t* seg_runs;    // [S + 1]
    int32_t* seg_tile0;                                         // [S + 1]
    int32_t* cta_chunk0;                                        // [G + 1]
    int4* cta_desc;                                             // [G + 1]
};

// Cut the vector into chunks (at every multiple of kChunk elements and at every segment boundary), partition
// the chunks over G CTAs as contiguous runs balanced by elements plus a per-chunk overhead, and count the runs
// that hold chunks of each segment (the arrivals expected per statistics phase).  Returns the chunk count.
int compute_tables(const int64_t* off, int S, int G, const HostTables& t) {
    int T = 0;
    for (int s = 0; s < S; ++s) {
        t.seg_chunk0[s] = T;
        t.seg_n[s] = (int32_t)(off[s + 1] - off[s]);
        t.seg_runs[s] = 0;
        int64_t at = off[s];
        while (at < off[s + 1]) {
            int64_t end = (at / kChunk + 1) * kChunk;
            if (end > off[s + 1]) end = off[s + 1];
            t.chunk_start[T] = (int32_t)at;
            t.chunk_seg[T] = s;
            ++T;
            at = end;
        }
    }
    t.seg_chunk0[S] = T;
    t.seg_n[S] = 0;
    t.seg_runs[S] = 0;
    // tiles of the giant segments (summed in two levels)
    int tiles = 0;
    for (int s = 0; s < S; ++s) {
        t.seg_tile0[s] = tiles;
        const int chunks = t.seg_chunk0[s + 1] - t.seg_chunk0[s];
        if (chunks > sidco::kGiantSeg) tiles += (chunks + sidco::kTile - 1) / sidco::kTile;
    }
    t.seg_tile0[S] = tiles;
    t.chunk_start[T] = (int32_t)off[S];
    t.chunk_seg[T] = 0;
    const double per_chunk = 128.0;
    double total = 0.0;
    for (int q = 0; q < T; ++q) total += (t.chunk_start[q + 1] - t.chunk_start[q]) + per_chunk;
    double acc = 0.0;
    int cta = 0;
    t.cta_chunk0[0] = 0;
    for (int q = 0; q < T; ++q) {
        // chunk q goes to the CTA whose share contains the chunk's midpoint
        const double w = (t.chunk_start[q + 1] - t.chunk_start[q]) + per_chunk;
        int want = (int)((acc + 0.5 * w) / total * G);
        if (want > G - 1) want = G - 1;
        while (cta < want) t.cta_chunk0[++cta] = q;
        acc += w;
    }
    while (cta < G) t.cta_chunk0[++cta] = T;
    // per-CTA descriptor {first chunk, end chunk, first segment, number of segments spanned}
    for (int g = 0; g < G; ++g) {
        int prev = -1;
        for (int q = t.cta_chunk0[g]; q < t.cta_chunk0[g + 1]; ++q)
            if (t.chunk_seg[q] != prev) { prev = t.chunk_seg[q]; ++t.seg_runs[prev]; }
        const int a = t.cta_chunk0[g], b = t.cta_chunk0[g + 1];
        t.cta_desc[g] = a < b ? make_int4(a, b, t.chunk_seg[a], t.chunk_seg[b - 1] - t.chunk_seg[a] + 1)
                              : make_int4(a, a, 0, 0);
    }
    t.cta_desc[G] = make_int4(T, T, 0, 0);
    return T;
}

// Build the chunk tables for a segment table and upload them together with fresh per-segment state.
// The adaptation state of an existing context survives a table rebuild when the segment count is unchanged.
cudaError_t build_tables(Context* c, const int64_t* off, int S, cudaStream_t stream) {
    const int64_t d = off[S];
    DeviceInfo* di = nullptr;
    cudaError_t e = device_info(c->device, &di);
    if (e != cudaSuccess) return e;
    const int G = launch_grid(*di);

    const size_t cap = (size_t)max_chunks(d, S) + 1;
    std::vector<int32_t> chunk_start(cap), chunk_seg(cap), seg_chunk0(S + 1), seg_n(S + 1), seg_runs(S + 1),
        seg_tile0(S + 1), cta_chunk0(G + 1);
    std::vector<int4> cta_desc(G + 1);
    const int T = compute_tables(off, S, G, HostTables{chunk_start.data(), chunk_seg.data(), seg_chunk0.data(),
                                                       seg_n.data(), seg_runs.data(), seg_tile0.data(),
                                                       cta_chunk0.data(), cta_desc.data()});

    const Layout L = make_layout(d, S, T, G);
    if (c->ws && c->ws_bytes < L.total) {
        if (!c->ws_owned) return cudaErrorMemoryAllocation;
        cudaFree(c->ws);
        c->ws = nullptr;
    }
    bool fresh = false;
    if (!c->ws) {
        if ((e = cudaMalloc(&c->ws, L.total)) != cudaSuccess) return e;
        c->ws_bytes = L.total;
        c->ws_owned = true;
        fresh = true;
    }
    const bool same_segments = c->tables_valid && c->S == S;
    // A reset that no call has consumed yet ("the residual is empty") outlives the rebuild.
    Control ctl_host;
    std::memset(&ctl_host, 0, sizeof(Control));
    if (c->tables_valid && !fresh) {
        Control old;
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return e;
        if ((e = cudaMemcpy(&old, (char*)c->ws + c->L.ctl, sizeof(Control), cudaMemcpyDeviceToHost)) != cudaSuccess)
            return e;
        ctl_host.residual_is_zero = old.residual_is_zero;
    }
    c->tables_valid = false;               // until the uploads below have succeeded
    // keep adaptation state across a table rebuild only when the segment count is unchanged
    std::vector<SegDev> seg_host(S + 1);
    if (same_segments && !fresh) {
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return e;
        if ((e = cudaMemcpy(seg_host.data(), (char*)c->ws + c->L.seg, sizeof(SegDev) * S, cudaMemcpyDeviceToHost)) !=
            cudaSuccess)
            return e;
        for (auto& sg : seg_host) { sg.arrived = 0; sg.k_acc = 0; sg.k_arr = 0; sg.pub = 0; }    // (the call numbering restarts below)
    } else {
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return e;
        for (auto& sg : seg_host) {
            std::memset(&sg, 0, sizeof(SegDev));
            sg.M = 1;
        }
    }
    char* base = (char*)c->ws;
    auto up = [&](size_t at, const void* src, size_t bytes) {
        return cudaMemcpy(base + at, src, bytes, cudaMemcpyHostToDevice);
    };
    if ((e = up(L.chunk_start, chunk_start.data(), sizeof(int32_t) * (T + 1))) != cudaSuccess) return e;
    if ((e = up(L.chunk_seg, chunk_seg.data(), sizeof(int32_t) * (T + 1))) != cudaSuccess) return e;
    if ((e = up(L.seg_chunk0, seg_chunk0.data(), sizeof(int32_t) * (S + 1))) != cudaSuccess) return e;
    if ((e = up(L.seg_n, seg_n.data(), sizeof(int32_t) * (S + 1))) != cudaSuccess) return e;
    if ((e = up(L.seg_runs, seg_runs.data(), sizeof(int32_t) * (S + 1))) != cudaSuccess) return e;
    if ((e = up(L.seg_tile0, seg_tile0.data(), sizeof(int32_t) * (S + 1))) != cudaSuccess) return e;
    if ((e = cudaMemset(base + L.tile_arr, 0, sizeof(int32_t) * (size_t)(T / sidco::kTile + S + 2))) != cudaSuccess) return e;
    if ((e = up(L.cta_desc, cta_desc.data(), sizeof(int4) * (G + 1))) != cudaSuccess) return e;
    if ((e = up(L.seg, seg_host.data(), sizeof(SegDev) * (S + 1))) != cudaSuccess) return e;
    if ((e = up(L.ctl, &ctl_host, sizeof(Control))) != cudaSuccess) return e;
    // (the call numbering restarts: no run's published count may carry a number of the old numbering)
    if ((e = cudaMemset(base + L.cta_total, 0, sizeof(unsigned long long) * (G + 1))) != cudaSuccess) return e;
    if ((e = cudaMemset(base + L.cta_dir, 0, sizeof(int32_t) * (G + 1))) != cudaSuccess) return e;
    if ((e = cudaMemset(base + L.chunk_cnt, 0, sizeof(int32_t) * (T + 1))) != cudaSuccess) return e;

    c->L = L;
    c->d = d;
    c->S = S;
    c->T = T;
    c->G = G;
    c->offsets.assign(off, off + S + 1);
    c->tables_valid = true;
    return cudaSuccess;
}

// Logarithms of the stage ratios (see Args::ln_ratio).
void fill_ln_tables(Args& a, double delta, double delta1) {
    for (int M = 0; M <= sidco::kMaxStages; ++M) {
        const double ratio = M == 0 ? delta1 : sidco::stage_ratio(delta, delta1, M, M - 1);
        a.ln_ratio[M] = std::log(ratio);
        a.ln_inv_ratio[M] = std::log(1.0 / ratio);
    }
}

// Cooperative launch: all CTAs of the persistent kernel are co-resident.
cudaError_t launch_persistent(const void* fn, int grid, void** kargs, cudaStream_t stream) {
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), kargs, sidco::kDynSmemBytes, stream);
}

// Fill the kernel's argument block for a workspace at `base` laid out as `L` and enqueue the persistent kernel.
// Used by every entry point, so that they cannot drift apart.
int launch_compress(char* base, const Layout& L, int64_t d, int T, int S, int G, const float* grad, float* residual, float delta,
                    int sid, int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k, cudaStream_t stream,
                    const Params& prm, bool grad_bf16 = false) {
    Args a{};
    a.grad = grad;
    a.residual = residual;
    a.out_idx = out_idx;
    a.out_val = out_val;
    a.out_k = out_k;
    a.chunk_start = (const int32_t*)(base + L.chunk_start);
    a.chunk_seg = (const int32_t*)(base + L.chunk_seg);
    a.seg_chunk0 = (const int32_t*)(base + L.seg_chunk0);
    a.seg_n = (const int32_t*)(base + L.seg_n);
    a.seg_runs = (const int32_t*)(base + L.seg_runs);
    a.seg_tile0 = (const int32_t*)(base + L.seg_tile0);
    a.tile_arr = (int32_t*)(base + L.tile_arr);
    a.tile_part = (double*)(base + L.tile_part);
    a.cta_desc = (const int4*)(base + L.cta_desc);
    a.part = (double*)(base + L.part);
    a.part_n = (int32_t*)(base + L.part_n);
    a.chunk_cnt = (int32_t*)(base + L.chunk_cnt);
    a.side_val = (float*)(base + L.side_val);
    a.side_mask = (unsigned*)(base + L.side_mask);
    a.side_cnt = (int32_t*)(base + L.side_cnt);
    a.stage_idx = (int32_t*)(base + L.stage_idx);
    a.stage_val = (float*)(base + L.stage_val);
    a.cta_pub = (unsigned long long*)(base + L.cta_total);
    a.cta_dir = (int32_t*)(base + L.cta_dir);
    a.cta_ns = (unsigned long long*)(base + L.cta_ns);
    a.cta_dbg = (int*)(base + L.cta_dbg);
    a.slot_spill_e = (int32_t*)(base + L.slot_spill_e);
    a.slot_spill_seg = (unsigned char*)(base + L.slot_spill_seg);
    a.seg = (SegDev*)(base + L.seg);
    a.ctl = (Control*)(base + L.ctl);
    a.delta = (double)delta;
    a.delta1 = prm.delta1;
    fill_ln_tables(a, (double)delta, prm.delta1);
    a.eps_H = prm.eps_H;
    a.eps_L = prm.eps_L;
    a.Q = prm.Q;
    a.sid = sid;
    a.max_stages = max_stages;
    a.C = T;
    a.S = S;
    a.G = G;
    a.d = (int)d;
    // 256-bit accesses to the residual and an fp32 gradient, 128-bit ones to a bf16 gradient
    a.vec_ok = (((uintptr_t)residual & 31u) | ((uintptr_t)grad & (grad_bf16 ? 15u : 31u))) == 0;
    a.grad_bf16 = grad_bf16 ? 1 : 0;
    a.pol_gamma_exact = prm.gamma_exact;
    a.pol_ratio_counts = prm.ratio_counts;
    a.pol_adapt_rev = prm.adapt_rev;
    const Hooks& h = hooks();
    a.spec_enable = h.spec_enable;           // (the result is the same with or without the pre-selection)
    a.spin_limit = h.spin_limit;
    a.drop_pub_seg = h.drop_pub_seg;

    void* kargs[] = {(void*)&a};
    const void* fn = sid == 0   ? (const void*)sidco::sidco_persistent_kernel<0>
                     : sid == 1 ? (prm.gamma_exact ? (const void*)sidco::sidco_persistent_kernel<1, true>
                                                   : (const void*)sidco::sidco_persistent_kernel<1>)
                                : (const void*)sidco::sidco_persistent_kernel<2>;
    const cudaError_t e = launch_persistent(fn, G, kargs, stream);
    if (e != cudaSuccess) return (int)e;
    g_launches.fetch_add(1);
    return 0;
}

int compress_impl(Context* c, const float* grad, float* residual, const int64_t* off, int S, float delta, int sid,
                  int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k, cudaStream_t stream,
                  const Params& prm, bool grad_bf16 = false) {
    cudaError_t e;
    const bool same = c->tables_valid && c->S == S &&
                      std::memcmp(c->offsets.data(), off, sizeof(int64_t) * (S + 1)) == 0;
    if (!same) {
        // allocation, uploads and a stream synchronisation: not something a capturing stream can record
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if ((e = cudaStreamIsCapturing(stream, &cap)) != cudaSuccess) return (int)e;
        if (cap != cudaStreamCaptureStatusNone) return SIDCO_E_CAPTURE;
        if ((e = build_tables(c, off, S, stream)) != cudaSuccess) return (int)e;
    }
    return launch_compress((char*)c->ws, c->L, c->d, c->T, c->S, c->G, grad, residual, delta, sid, max_stages, out_idx,
                           out_val, out_k, stream, prm, grad_bf16);
}

Context* find_or_create(const void* key, int dev) {
    auto it = g_ctx.find(key);
    if (it != g_ctx.end()) {
        if (it->second->device == dev) return it->second;
        free_context(it->second);
        g_ctx.erase(it);
    }
    Context* c = new Context();
    c->device = dev;
    g_ctx[key] = c;
    return c;
}

}  // namespace

extern "C" {

int sidco_compress(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs, float delta,
                   int sid_type, int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k, void* stream) {
    int rc = check_args(grad, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx, out_val, out_k);
    if (rc) return rc;
    const int64_t d = seg_offsets[n_segs];
    if ((grad < residual + d) && (residual < grad + d) && d > 0) return SIDCO_E_ALIAS;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = find_or_create(residual, dev);
    return compress_impl(c, grad, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx, out_val, out_k,
                         (cudaStream_t)stream, g_params);
}

int sidco_compress_bf16(const uint16_t* grad_bf16, float* residual, const int64_t* seg_offsets, int n_segs, float delta,
                        int sid_type, int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k, void* stream) {
    int rc = check_args(grad_bf16, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx, out_val, out_k);
    if (rc) return rc;
    const int64_t d = seg_offsets[n_segs];
    const char* g0 = (const char*)grad_bf16;
    const char* r0 = (const char*)residual;
    if ((g0 < r0 + 4 * d) && (r0 < g0 + 2 * d) && d > 0) return SIDCO_E_ALIAS;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = find_or_create(residual, dev);
    return compress_impl(c, (const float*)grad_bf16, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx,
                         out_val, out_k, (cudaStream_t)stream, g_params, true);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Entry point that allocates nothing: its workspace is a fixed array in device memory.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxElems = SIDCO_STATIC_MAX_ELEMS;
constexpr int kStaticMaxSegs = SIDCO_STATIC_MAX_SEGS;
constexpr int kStaticMaxChunks = kStaticMaxElems / kChunk + kStaticMaxSegs + 1;
constexpr size_t kStaticBytes = 18u << 20;

// The workspace itself.  Device code could name it directly; host code may only take its address
// through cudaGetSymbolAddress, because on the host this name is a stand-in, not a device pointer.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

struct StaticContext {
    bool ready = false;              // device address looked up
    unsigned char* base = nullptr;   // device address of g_static_scratch on this device
    bool tables_valid = false;
    const void* key = nullptr;       // residual pointer the adaptation state belongs to
    int S = 0, T = 0, G = 0;
    Layout L{};
    int64_t offsets[kStaticMaxSegs + 1];
    int32_t chunk_start[kStaticMaxChunks + 1], chunk_seg[kStaticMaxChunks + 1];
    int32_t seg_chunk0[kStaticMaxSegs + 1], seg_n[kStaticMaxSegs + 1], seg_runs[kStaticMaxSegs + 1];
    int32_t seg_tile0[kStaticMaxSegs + 1];
    int32_t cta_chunk0[kMaxGrid + 1];
    int4 cta_desc[kMaxGrid + 1];
    SegDev seg_init[kStaticMaxSegs + 1];
};

constexpr int kMaxDevices = 64;
StaticContext g_static[kMaxDevices];

}  // namespace

extern "C" {

int sidco_compress_static(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs, float delta,
                          int sid_type, int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k,
                          void* stream_v) {
    int rc = check_args(grad, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx, out_val, out_k);
    if (rc) return rc;
    const int64_t d = seg_offsets[n_segs];
    if (d > kStaticMaxElems || n_segs > kStaticMaxSegs) return SIDCO_E_SIZE;
    if ((grad < residual + d) && (residual < grad + d) && d > 0) return SIDCO_E_ALIAS;
    cudaStream_t stream = (cudaStream_t)stream_v;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= kMaxDevices) return SIDCO_E_SIZE;
    std::lock_guard<std::mutex> lock(g_mu);
    StaticContext& c = g_static[dev];
    if (!c.ready) {
        // Once per device, with that device current: ask the runtime where the array lives there.
        void* p = nullptr;
        if ((e = cudaGetSymbolAddress(&p, g_static_scratch)) != cudaSuccess) return (int)e;
        c.base = (unsigned char*)p;
        c.ready = true;
    }
    DeviceInfo* di = nullptr;
    if ((e = device_info(dev, &di)) != cudaSuccess) return (int)e;
    const bool same = c.tables_valid && c.key == residual && c.S == n_segs &&
                      std::memcmp(c.offsets, seg_offsets, sizeof(int64_t) * (n_segs + 1)) == 0;
    if (!same) {
        // New residual or segment table: rebuild the tables and start the adaptation state afresh.  The uploads
        // and the synchronisation below are not something a capturing stream can record.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if ((e = cudaStreamIsCapturing(stream, &cap)) != cudaSuccess) return (int)e;
        if (cap != cudaStreamCaptureStatusNone) return SIDCO_E_CAPTURE;
        // From here until the last upload has completed the context describes no usable tables.
        c.tables_valid = false;
        c.key = nullptr;
        const int G = launch_grid(*di);
        if (G > kMaxGrid) return SIDCO_E_SIZE;
        c.T = compute_tables(seg_offsets, n_segs, G, HostTables{c.chunk_start, c.chunk_seg, c.seg_chunk0, c.seg_n,
                                                                c.seg_runs, c.seg_tile0, c.cta_chunk0, c.cta_desc});
        c.S = n_segs;
        c.G = G;
        for (int s = 0; s <= n_segs; ++s) c.offsets[s] = seg_offsets[s];
        c.L = make_layout(d, n_segs, c.T, c.G);
        if (c.L.total > kStaticBytes) return SIDCO_E_SIZE;
        for (int s = 0; s <= n_segs; ++s) {
            std::memset(&c.seg_init[s], 0, sizeof(SegDev));
            c.seg_init[s].M = 1;
        }
        const Layout& L = c.L;
        auto up = [&](size_t at, const void* src, size_t bytes) {
            return cudaMemcpyAsync(c.base + at, src, bytes, cudaMemcpyHostToDevice, stream);
        };
        if ((e = up(L.chunk_start, c.chunk_start, sizeof(int32_t) * (c.T + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.chunk_seg, c.chunk_seg, sizeof(int32_t) * (c.T + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.seg_chunk0, c.seg_chunk0, sizeof(int32_t) * (n_segs + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.seg_n, c.seg_n, sizeof(int32_t) * (n_segs + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.seg_runs, c.seg_runs, sizeof(int32_t) * (n_segs + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.seg_tile0, c.seg_tile0, sizeof(int32_t) * (n_segs + 1))) != cudaSuccess) return (int)e;
        if ((e = cudaMemsetAsync(c.base + L.tile_arr, 0, sizeof(int32_t) * (size_t)(c.T / sidco::kTile + n_segs + 2), stream)) != cudaSuccess) return (int)e;
        if ((e = up(L.cta_desc, c.cta_desc, sizeof(int4) * (c.G + 1))) != cudaSuccess) return (int)e;
        if ((e = up(L.seg, c.seg_init, sizeof(SegDev) * (n_segs + 1))) != cudaSuccess) return (int)e;
        // The array keeps whatever the last call left.  What must start at zero (the control block: finished-CTA
        // count, call number, time-out flag; the published run counts; the per-chunk counts) is cleared here,
        // when this residual and segment table are first seen; from then on it is state that is meant to
        // persist, and everything else is rewritten before it is read.
        if ((e = cudaMemsetAsync(c.base + L.cta_dir, 0, sizeof(int32_t) * (c.G + 1), stream)) != cudaSuccess) return (int)e;
        if ((e = cudaMemsetAsync(c.base + L.ctl, 0, sizeof(Control), stream)) != cudaSuccess) return (int)e;
        if ((e = cudaMemsetAsync(c.base + L.cta_total, 0, sizeof(unsigned long long) * (c.G + 1), stream)) != cudaSuccess) return (int)e;
        if ((e = cudaMemsetAsync(c.base + L.chunk_cnt, 0, sizeof(int32_t) * (c.T + 1), stream)) != cudaSuccess) return (int)e;
        // the uploads read the fixed host arrays: let them finish before those can change again
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return (int)e;
        c.key = residual;
        c.tables_valid = true;
    }
    return launch_compress((char*)c.base, c.L, d, c.T, c.S, c.G, grad, residual, delta, sid_type, max_stages, out_idx,
                           out_val, out_k, stream, g_params);
}

int sidco_compress_host(const float* grad, float* residual, const int64_t* seg_offsets, int n_segs, float delta,
                        int sid_type, int max_stages, int32_t* out_idx, float* out_val, int32_t* out_k,
                        void* stream_v) {
    int rc = check_args(grad, residual, seg_offsets, n_segs, delta, sid_type, max_stages, out_idx, out_val, out_k);
    if (rc) return rc;
    const int64_t d = seg_offsets[n_segs];
    cudaStream_t stream = (cudaStream_t)stream_v;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = find_or_create(residual, dev);
    if (c->staging_d != d || c->staging_S != n_segs) {
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return (int)e;
        if (c->h_grad) { cudaFree(c->h_grad); cudaFree(c->h_res); cudaFree(c->h_idx); cudaFree(c->h_val); cudaFree(c->h_k); }
        c->h_grad = c->h_res = c->h_val = nullptr; c->h_idx = c->h_k = nullptr;
        const size_t n = (size_t)d + 4;
        if ((e = cudaMalloc(&c->h_grad, n * 4)) != cudaSuccess) return (int)e;
        if ((e = cudaMalloc(&c->h_res, n * 4)) != cudaSuccess) return (int)e;
        if ((e = cudaMalloc(&c->h_idx, n * 4)) != cudaSuccess) return (int)e;
        if ((e = cudaMalloc(&c->h_val, n * 4)) != cudaSuccess) return (int)e;
        if ((e = cudaMalloc(&c->h_k, sizeof(int32_t) * (size_t)(n_segs + 1))) != cudaSuccess) return (int)e;
        c->staging_d = d;
        c->staging_S = n_segs;
    }
    const size_t bytes = (size_t)d * 4;
    if ((e = cudaMemcpyAsync(c->h_grad, grad, bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return (int)e;
    if ((e = cudaMemcpyAsync(c->h_res, residual, bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return (int)e;
    rc = compress_impl(c, c->h_grad, c->h_res, seg_offsets, n_segs, delta, sid_type, max_stages, c->h_idx, c->h_val,
                       c->h_k, stream, g_params);
    if (rc) return rc;
    if ((e = cudaMemcpyAsync(out_k, c->h_k, sizeof(int32_t) * (size_t)(n_segs + 1), cudaMemcpyDeviceToHost, stream)) !=
        cudaSuccess)
        return (int)e;
    if ((e = cudaMemcpyAsync(residual, c->h_res, bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return (int)e;
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return (int)e;
    const size_t kb = (size_t)out_k[n_segs] * 4;
    if (kb) {
        if ((e = cudaMemcpyAsync(out_idx, c->h_idx, kb, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return (int)e;
        if ((e = cudaMemcpyAsync(out_val, c->h_val, kb, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return (int)e;
        if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return (int)e;
    }
    return 0;
}

size_t sidco_workspace_bytes(int64_t d, int n_segs) {
    if (d < 0 || n_segs < 1) return 0;
    return make_layout(d, n_segs, max_chunks(d, n_segs), kMaxGrid).total;
}

int sidco_set_workspace(const float* residual, void* device_ptr, size_t bytes) {
    if (!residual || !device_ptr) return SIDCO_E_NULL;
    if (((uintptr_t)device_ptr & (kAlign - 1)) != 0) return SIDCO_E_WORKSPACE;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = find_or_create(residual, dev);
    if (c->tables_valid) return SIDCO_E_WORKSPACE;      // too late: a workspace is already in use
    c->ws = device_ptr;
    c->ws_bytes = bytes;
    c->ws_owned = false;
    return 0;
}

int sidco_set_params(double delta1, double eps_H, double eps_L, int Q) {
    if (!(delta1 > 0.0 && delta1 < 1.0) || !(eps_H >= 0.0 && eps_H < 1.0) || !(eps_L >= 0.0 && eps_L < 1.0) || Q < 1)
        return SIDCO_E_PARAMS;
    std::lock_guard<std::mutex> lock(g_mu);
    g_params.delta1 = delta1;
    g_params.eps_H = eps_H;
    g_params.eps_L = eps_L;
    g_params.Q = Q;
    return 0;
}

int sidco_set_policy(int gamma_exact, int ratio_from_counts, int adapt_reversed) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_params.gamma_exact = gamma_exact ? 1 : 0;
    g_params.ratio_counts = ratio_from_counts ? 1 : 0;
    g_params.adapt_rev = adapt_reversed ? 1 : 0;
    return 0;
}

static int with_segments(const float* residual, int n_segs, Context** out) {
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    if (n_segs != it->second->S) return SIDCO_E_SEGMENTS;
    *out = it->second;
    return 0;
}

int sidco_reset_state(const float* residual) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    Context* c = it->second;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    std::vector<SegDev> seg(c->S + 1);
    for (auto& sg : seg) { std::memset(&sg, 0, sizeof(SegDev)); sg.M = 1; }
    char* base = (char*)c->ws;
    if ((e = cudaMemcpy(base + c->L.seg, seg.data(), sizeof(SegDev) * (c->S + 1), cudaMemcpyHostToDevice)) != cudaSuccess)
        return (int)e;
    // call numbering and barrier count restart with the segment records; the residual counts as empty
    Control ctl;
    std::memset(&ctl, 0, sizeof(Control));
    ctl.residual_is_zero = 1;
    if ((e = cudaMemset(base + c->L.cta_total, 0, sizeof(unsigned long long) * (c->G + 1))) != cudaSuccess) return (int)e;
    if ((e = cudaMemset(base + c->L.tile_arr, 0, sizeof(int32_t) * (size_t)(c->T / sidco::kTile + c->S + 2))) != cudaSuccess) return (int)e;
    if ((e = cudaMemcpy(base + c->L.ctl, &ctl, sizeof(Control), cudaMemcpyHostToDevice)) != cudaSuccess) return (int)e;
    return 0;
}

int sidco_reset_state_async(const float* residual, void* stream) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    Context* c = it->second;
    sidco::sidco_reset_state_kernel<<<(c->S + 255) / 256, 256, 0, (cudaStream_t)stream>>>(
        (SegDev*)((char*)c->ws + c->L.seg), c->S, (Control*)((char*)c->ws + c->L.ctl));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    g_launches.fetch_add(1);
    return 0;
}

int sidco_get_debug(const float* residual, sidco_seg_debug* out, int n_segs) {
    if (!out) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = nullptr;
    int rc = with_segments(residual, n_segs, &c);
    if (rc) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    std::vector<SegDev> seg(c->S);
    Control ctl;
    char* base = (char*)c->ws;
    if ((e = cudaMemcpy(seg.data(), base + c->L.seg, sizeof(SegDev) * c->S, cudaMemcpyDeviceToHost)) != cudaSuccess)
        return (int)e;
    if ((e = cudaMemcpy(&ctl, base + c->L.ctl, sizeof(Control), cudaMemcpyDeviceToHost)) != cudaSuccess) return (int)e;
    for (int s = 0; s < c->S; ++s) {
        out[s].M_used = seg[s].M_eff;
        out[s].M_next = seg[s].M;
        out[s].status = seg[s].status | (ctl.timeout ? SIDCO_ST_TIMEOUT : 0) | (ctl.bounds ? SIDCO_ST_BOUNDS : 0);
        out[s].calls = seg[s].calls;
        out[s].k_sum = seg[s].k_sum;
        for (int m = 0; m < SIDCO_MAX_STAGES; ++m) {
            out[s].eta[m] = seg[s].eta[m];
            out[s].k_stage[m] = seg[s].k_stage[m];
        }
    }
    return 0;
}

int sidco_get_phase_times(const float* residual, double* us_out) {
#ifndef SIDCO_PROFILE
    (void)residual; (void)us_out;
    return SIDCO_E_UNSUPPORTED;
#else
    if (!us_out) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    Context* c = it->second;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    Control ctl;
    if ((e = cudaMemcpy(&ctl, (char*)c->ws + c->L.ctl, sizeof(Control), cudaMemcpyDeviceToHost)) != cudaSuccess)
        return (int)e;
    auto us = [&](int a, int b) { return (double)(long long)(ctl.t_ns[b] - ctl.t_ns[a]) * 1e-3; };
    for (int i = 0; i < 5; ++i) us_out[i] = us(i, i + 1);
    us_out[5] = us(0, 5);
    us_out[6] = us(0, 6);      // first sweep of CTA 0 alone
    us_out[7] = us(6, 7);      // its arrivals and fits
    us_out[8] = us(1, 8);      // stage-2 sweep of CTA 0 alone (meaningless if no segment used M >= 2)
    us_out[9] = us(8, 9);
    us_out[10] = us(10, 11);   // arrivals and fits of the last refit stage
    us_out[11] = us(3, 12);    // survivor staging sweep of CTA 0 alone
    return 0;
#endif
}

int sidco_get_cta_sweep_times(const float* residual, double* us_out, int max_ctas) {
#ifndef SIDCO_PROFILE
    (void)residual; (void)us_out; (void)max_ctas;
    return SIDCO_E_UNSUPPORTED;
#else
    if (!us_out) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    Context* c = it->second;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    Control ctl;
    std::vector<unsigned long long> ns(4 * (size_t)c->G);
    if ((e = cudaMemcpy(&ctl, (char*)c->ws + c->L.ctl, sizeof(Control), cudaMemcpyDeviceToHost)) != cudaSuccess)
        return (int)e;
    if ((e = cudaMemcpy(ns.data(), (char*)c->ws + c->L.cta_ns, ns.size() * 8, cudaMemcpyDeviceToHost)) != cudaSuccess)
        return (int)e;
    const int n = c->G < max_ctas ? c->G : max_ctas;
    for (int i = 0; i < 4 * n; ++i) us_out[i] = (double)(long long)(ns[i] - ctl.t_ns[0]) * 1e-3;
    return n;
#endif
}

int sidco_get_cta_selection_info(const float* residual, int32_t* out, int max_ctas) {
#ifndef SIDCO_PROFILE
    (void)residual; (void)out; (void)max_ctas;
    return SIDCO_E_UNSUPPORTED;
#else
    if (!out) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end() || !it->second->tables_valid) return SIDCO_E_UNKNOWN_KEY;
    Context* c = it->second;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    const int n = c->G < max_ctas ? c->G : max_ctas;
    if ((e = cudaMemcpy(out, (char*)c->ws + c->L.cta_dbg, sizeof(int32_t) * 8 * n, cudaMemcpyDeviceToHost)) != cudaSuccess)
        return (int)e;
    return n;
#endif
}

int sidco_set_test_hooks(int grid, int spec_enable, long long spin_limit, int drop_publication_seg) {
    if (grid < 0 || spin_limit < 0) return SIDCO_E_PARAMS;
    std::lock_guard<std::mutex> lock(g_mu);
    Hooks& h = hooks();
    h.grid = grid;
    h.spec_enable = spec_enable == 2 ? 2 : (spec_enable ? 1 : 0);
    h.spin_limit = spin_limit ? spin_limit : sidco::kSpinLimit;
    h.drop_pub_seg = drop_publication_seg;
    return 0;
}

int sidco_build_flags(void) {
    int f = 0;
#ifdef SIDCO_PROFILE
    f |= SIDCO_BUILD_PROFILE;
#endif
#ifdef SIDCO_BOUNDS_CHECK
    f |= SIDCO_BUILD_BOUNDS_CHECK;
#endif
    return f;
}

int sidco_state_save(const float* residual, int64_t* blob, int n_segs) {
    if (!blob) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = nullptr;
    int rc = with_segments(residual, n_segs, &c);
    if (rc) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    std::vector<SegDev> seg(c->S);
    if ((e = cudaMemcpy(seg.data(), (char*)c->ws + c->L.seg, sizeof(SegDev) * c->S, cudaMemcpyDeviceToHost)) !=
        cudaSuccess)
        return (int)e;
    for (int s = 0; s < c->S; ++s) {
        blob[3 * s + 0] = seg[s].M;
        blob[3 * s + 1] = seg[s].calls;
        blob[3 * s + 2] = seg[s].k_sum;
    }
    return 0;
}

int sidco_state_load(const float* residual, const int64_t* blob, int n_segs) {
    if (!blob) return SIDCO_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    Context* c = nullptr;
    int rc = with_segments(residual, n_segs, &c);
    if (rc) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return (int)e;
    std::vector<SegDev> seg(c->S);
    char* at = (char*)c->ws + c->L.seg;
    if ((e = cudaMemcpy(seg.data(), at, sizeof(SegDev) * c->S, cudaMemcpyDeviceToHost)) != cudaSuccess) return (int)e;
    for (int s = 0; s < c->S; ++s) {
        if (blob[3 * s] < 1 || blob[3 * s] > SIDCO_MAX_STAGES || blob[3 * s + 1] < 0 || blob[3 * s + 2] < 0)
            return SIDCO_E_PARAMS;
        seg[s].M = (int32_t)blob[3 * s + 0];
        seg[s].calls = (int32_t)blob[3 * s + 1];
        seg[s].k_sum = blob[3 * s + 2];
    }
    if ((e = cudaMemcpy(at, seg.data(), sizeof(SegDev) * c->S, cudaMemcpyHostToDevice)) != cudaSuccess) return (int)e;
    return 0;
}

int sidco_release(const float* residual) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ctx.find(residual);
    if (it == g_ctx.end()) return SIDCO_E_UNKNOWN_KEY;
    cudaDeviceSynchronize();
    free_context(it->second);
    g_ctx.erase(it);
    return 0;
}

int sidco_release_all(void) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ctx.empty()) cudaDeviceSynchronize();
    for (auto& kv : g_ctx) free_context(kv.second);
    g_ctx.clear();
    return 0;
}

int64_t sidco_launch_count(void) { return g_launches.load(); }

const char* sidco_error_string(int code) {
    switch (code) {
        case 0: return "success";
        case SIDCO_E_NULL: return "a required pointer is NULL";
        case SIDCO_E_SEGMENTS: return "bad segment table (n_segs < 1, offsets[0] != 0, decreasing, or d too large)";
        case SIDCO_E_DELTA: return "delta must lie in (0, 1)";
        case SIDCO_E_SID: return "unknown sid_type";
        case SIDCO_E_STAGES: return "max_stages must be non-zero and at most SIDCO_MAX_STAGES in magnitude";
        case SIDCO_E_PARAMS: return "parameter out of range";
        case SIDCO_E_UNKNOWN_KEY: return "no state for this residual pointer";
        case SIDCO_E_WORKSPACE: return "workspace too small, misaligned, or set too late";
        case SIDCO_E_ALIAS: return "grad and residual overlap";
        case SIDCO_E_SIZE: return "size beyond the limit of this entry point";
        case SIDCO_E_CAPTURE:
            return "first call for this residual and segment table must be made before stream capture begins";
        case SIDCO_E_UNSUPPORTED: return "not available in this build of the library";
        default: break;
    }
    if (code > 0) return cudaGetErrorString((cudaError_t)code);
    return "unknown error";
}

int sidco_version(void) { return 200; }

}  // extern "C"
