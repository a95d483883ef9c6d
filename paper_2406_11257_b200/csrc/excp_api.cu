// The C ABI of include/excp.h: handle, argument checks, grouping of the tensor
// list, and the order of the kernel launches.  No arithmetic of the method
// lives here.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/excp.h"
#include "excp_common.cuh"

using namespace excp;

namespace excp {
// Launch counter and optional CUDA-event timing of the stages of one call.
struct Profiler {
    bool enabled = false;
    std::vector<cudaEvent_t> ev;
    std::vector<int> stage;
    size_t used = 0;
    double ms[ST_COUNT] = {};
    unsigned long long launches = 0;
    void begin(cudaStream_t s) {
        used = 0;
        launches = 0;
        for (double& m : ms) m = 0.0;
        if (enabled && !ev.empty()) cudaEventRecord(ev[0], s);
    }
    void finish() {   // after the stream has been synchronised
        if (!enabled) return;
        for (size_t i = 1; i <= used; ++i) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, ev[i - 1], ev[i]) == cudaSuccess) ms[stage[i]] += t;
        }
    }
};
void prof_mark(const LaunchCfg& cfg, int stage, int launches) {
    Profiler* p = cfg.prof;
    if (!p) return;
    p->launches += (unsigned long long)launches;
    if (p->enabled && p->used + 1 < p->ev.size()) {
        ++p->used;
        p->stage[p->used] = stage;
        cudaEventRecord(p->ev[p->used], cfg.stream);
    }
}
}  // namespace excp

struct excp_handle_s {
    int device = 0;
    int sms = 0;
    size_t cap_tiles = 0;
    Workspace ws{};
    KmArrays km{};
    TensorState* d_state = nullptr;      // MAX_GROUP_TENSORS
    DecState* d_dstate = nullptr;        // MAX_GROUP_TENSORS
    CallState* d_call = nullptr;
    void* d_desc = nullptr;              // TensorDesc[] or DecDesc[] of the whole call
    TensorResult* d_results = nullptr;
    void* h_desc = nullptr;              // pinned
    TensorResult* h_results = nullptr;   // pinned
    CallState* h_call = nullptr;         // pinned
    size_t tensor_cap = 0;               // entries the per-call arrays hold
    int last_cuda_error = 0;
    int km_margin = 1;                   // see excp_set_kmeans_margin
    unsigned long long wait_limit_ns = 2000000000ull;   // see excp_set_wait_limit
    bool report_sse = false;             // see excp_set_report_sse
    Profiler prof;
    // host-buffer path: two staging slots (inputs + records), its own copy streams
    float* stage[2][4] = {};
    unsigned char* stage_blob[2] = {};
    size_t stage_blob_bytes = 0;
    int stage_bits = 0;                  // code width the record staging is sized for
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
    cudaEvent_t ev_h2d[2] = {}, ev_compute[2] = {}, ev_d2h[2] = {};
};

namespace {

constexpr size_t DESC_BYTES = sizeof(TensorDesc) > sizeof(DecDesc) ? sizeof(TensorDesc) : sizeof(DecDesc);
constexpr unsigned long long MAX_NUMEL = 1ull << 31;

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int now = -1;
        if (prev >= 0 && cudaGetDevice(&now) == cudaSuccess && now != prev) cudaSetDevice(prev);
    }
};

bool check(excp_handle h, cudaError_t e) {
    if (e == cudaSuccess) return true;
    h->last_cuda_error = (int)e;
    return false;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void free_call_arrays(excp_handle h) {
    if (h->d_desc) cudaFree(h->d_desc);
    if (h->d_results) cudaFree(h->d_results);
    if (h->h_desc) cudaFreeHost(h->h_desc);
    if (h->h_results) cudaFreeHost(h->h_results);
    h->d_desc = nullptr; h->d_results = nullptr; h->h_desc = nullptr; h->h_results = nullptr;
    h->tensor_cap = 0;
}

bool ensure_call_arrays(excp_handle h, size_t n) {
    if (n <= h->tensor_cap) return true;
    free_call_arrays(h);
    size_t cap = 4096;
    while (cap < n) cap *= 2;
    if (!check(h, cudaMalloc(&h->d_desc, cap * DESC_BYTES))) return false;
    if (!check(h, cudaMalloc(reinterpret_cast<void**>(&h->d_results), cap * sizeof(TensorResult)))) return false;
    if (!check(h, cudaMallocHost(&h->h_desc, cap * DESC_BYTES))) return false;
    if (!check(h, cudaMallocHost(reinterpret_cast<void**>(&h->h_results), cap * sizeof(TensorResult)))) return false;
    h->tensor_cap = cap;
    return true;
}

struct Group { size_t first, count; u32 tiles; };

// Consecutive tensors whose tiles fit the workspace (and the per-group state).
bool make_groups(excp_handle h, const size_t* numel, size_t n, std::vector<Group>& out) {
    Group g{0, 0, 0};
    for (size_t i = 0; i < n; ++i) {
        if (numel[i] > MAX_NUMEL) return false;
        const size_t t = (numel[i] + TILE - 1) / TILE;
        if (t > h->cap_tiles) return false;
        if (g.count && (g.tiles + t > h->cap_tiles || g.count >= (size_t)MAX_GROUP_TENSORS)) {
            out.push_back(g);
            g = Group{i, 0, 0};
        }
        g.tiles += (u32)t;
        ++g.count;
    }
    if (g.count) out.push_back(g);
    return true;
}

excp_status validate_params(const excp_params* params) {
    if (!params) return EXCP_ERR_INVALID_ARG;
    if ((params->bits != 2 && params->bits != 4 && params->bits != 8) || params->kmeans_iters < 0 || (params->flags & ~OPT_ALL) ||
        (params->median_source != 0 && params->median_source != 1) ||
        !(params->alpha >= 0.f) || !(params->beta >= 0.f) || std::isinf(params->alpha) ||
        std::isinf(params->beta))
        return EXCP_ERR_INVALID_ARG;
    return EXCP_OK;
}

Params to_params(excp_handle h, const excp_params* params) {
    Params p;
    p.km_margin = h->km_margin;
    p.wait_ns = h->wait_limit_ns;
    p.alpha = params->alpha; p.beta = params->beta; p.bits = params->bits;
    p.kmeans_iters = params->kmeans_iters; p.seed = params->seed; p.median_source = params->median_source;
    p.flags = params->flags;
    p.wfmt = WF_F32;
    return p;
}

// All kernels of one group, in order.
bool run_group(excp_handle h, const LaunchCfg& cfg, const TensorDesc* descs, int nt, u32 tiles,
               const Params& p, unsigned char* blob, u64 blob_capacity, TensorResult* results, bool want_sse) {
    if (!check(h, cudaMemsetAsync(h->d_state, 0, nt * sizeof(TensorState), cfg.stream))) return false;
    if (!check(h, cudaMemsetAsync(h->ws.cst, 0, nt * sizeof(CellState), cfg.stream))) return false;
    // the per-tile survivor counts start at zero, so that no kernel can meet a stale count where a sweep gave up
    if (tiles && (!check(h, cudaMemsetAsync(h->ws.tile_cnt_w, 0, (size_t)tiles * sizeof(u32), cfg.stream)) ||
                  !check(h, cudaMemsetAsync(h->ws.tile_cnt_o, 0, (size_t)tiles * sizeof(u32), cfg.stream))))
        return false;
    launch_stats(cfg, descs, h->d_state, nt, tiles, h->ws, p, h->d_call);
    launch_mask_compact(cfg, descs, h->d_state, nt, tiles, h->ws, p, h->d_call, blob_capacity);
    if (!(p.flags & OPT_NO_QUANT)) launch_kmeans(cfg, descs, h->d_state, nt, tiles, h->ws, h->km, p, h->d_call);
    launch_pack(cfg, descs, h->d_state, nt, tiles, h->ws, p, blob, h->d_call, results, want_sse);
    return check(h, cudaGetLastError());
}

void fill_outputs(excp_handle h, size_t first, size_t count, const size_t* numel, size_t base,
                  size_t* tensor_offsets_out, excp_tensor_stats* stats_out) {
    for (size_t i = first; i < first + count; ++i) {
        const TensorResult& r = h->h_results[i];
        tensor_offsets_out[i] = base + (size_t)r.blob_off;
        tensor_offsets_out[i + 1] = base + (size_t)(r.blob_off + r.blob_bytes);
        if (stats_out) {
            excp_tensor_stats& s = stats_out[i];
            s.numel = numel[i]; s.nnz_w = r.nnz_w; s.nnz_o = r.nnz_o; s.blob_bytes = r.blob_bytes;
            s.median = r.median; s.mean_abs_ea = r.mean_abs_ea; s.thr_w = r.thr_w; s.thr_o = r.thr_o;
            s.sse_w = r.sse[0]; s.sse_ea = r.sse[1]; s.sse_eas = r.sse[2];
        }
    }
}

// Staging of the host-buffer path.  The record staging holds the largest records a group can
// produce at `bits` (every element a survivor); a call with wider codes than any before it on this
// handle gets a larger one.
bool ensure_host_path(excp_handle h, int bits) {
    const size_t elems = h->cap_tiles * (size_t)TILE;
    if (bits > h->stage_bits) {
        if (h->s_d2h && !check(h, cudaStreamSynchronize(h->s_d2h))) return false;
        h->stage_blob_bytes = (size_t)record_bytes(elems, elems, elems, bits) + (size_t)MAX_GROUP_TENSORS * 512;
        for (int k = 0; k < 2; ++k) {
            if (h->stage_blob[k]) cudaFree(h->stage_blob[k]);
            h->stage_blob[k] = nullptr;
            if (!check(h, cudaMalloc(reinterpret_cast<void**>(&h->stage_blob[k]), h->stage_blob_bytes))) {
                h->stage_bits = 0;
                return false;
            }
        }
        h->stage_bits = bits;
    }
    if (h->s_h2d) return true;
    bool ok = true;
    for (int k = 0; k < 2 && ok; ++k) {
        for (int j = 0; j < 4 && ok; ++j)
            if (!h->stage[k][j]) ok = check(h, cudaMalloc(reinterpret_cast<void**>(&h->stage[k][j]), elems * sizeof(float)));
        if (!h->ev_h2d[k]) ok = ok && check(h, cudaEventCreateWithFlags(&h->ev_h2d[k], cudaEventDisableTiming));
        if (!h->ev_compute[k]) ok = ok && check(h, cudaEventCreateWithFlags(&h->ev_compute[k], cudaEventDisableTiming));
        if (!h->ev_d2h[k]) ok = ok && check(h, cudaEventCreateWithFlags(&h->ev_d2h[k], cudaEventDisableTiming));
    }
    if (!h->s_d2h) ok = ok && check(h, cudaStreamCreateWithFlags(&h->s_d2h, cudaStreamNonBlocking));
    ok = ok && check(h, cudaStreamCreateWithFlags(&h->s_h2d, cudaStreamNonBlocking));   // last: marks the path as ready
    return ok;
}

excp_status status_from_flags(u32 flags) {
    if (flags & FLAG_TIMEOUT) return EXCP_ERR_TIMEOUT;
    if (flags & FLAG_INTERNAL) return EXCP_ERR_CUDA;
    if (flags & FLAG_NONFINITE) return EXCP_ERR_NONFINITE_INPUT;
    if (flags & FLAG_CORRUPT) return EXCP_ERR_CORRUPT_BLOB;
    if (flags & FLAG_UNSUPPORTED) return EXCP_ERR_UNSUPPORTED;
    if (flags & FLAG_BLOB_FULL) return EXCP_ERR_BUFFER_TOO_SMALL;
    return EXCP_OK;
}

}  // namespace

extern "C" {

excp_status excp_create(excp_handle* out, int device, size_t workspace_numel) {
    if (!out) return EXCP_ERR_INVALID_ARG;
    *out = nullptr;
    if (workspace_numel == 0 || workspace_numel > (1ull << 40)) return EXCP_ERR_INVALID_ARG;
    excp_handle h = new (std::nothrow) excp_handle_s();
    if (!h) return EXCP_ERR_CUDA;
    h->device = device;
    DeviceGuard guard(device);
    cudaDeviceProp prop;
    bool ok = guard.ok && check(h, cudaGetDeviceProperties(&prop, device));
    if (ok) {
        h->sms = prop.multiProcessorCount;
        h->cap_tiles = (workspace_numel + TILE - 1) / TILE;
        const size_t elems = h->cap_tiles * (size_t)TILE;
        for (int k = 0; k < 3 && ok; ++k) {
            ok = check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.surv[k]), elems * sizeof(float)));
            ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.bkt[k]), elems * sizeof(float)));
        }
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.cst), MAX_GROUP_TENSORS * sizeof(CellState)));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->km.pending), sizeof(u32)));
        const size_t rows = (size_t)std::min(h->sms * 2, (int)KM_MAX_GRID) + MAX_GROUP_TENSORS;
        for (int k = 0; k < 3 && ok; ++k) {
            ok = check(h, cudaMalloc(reinterpret_cast<void**>(&h->km.rows[k]), rows * NCELL * sizeof(u32)));
            ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->km.pos[k]), rows * NCELL * sizeof(u32)));
        }
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.bm_w), elems / 8));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.bm_o), elems / 8));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.tile_cnt_w), h->cap_tiles * 4));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.tile_cnt_o), h->cap_tiles * 4));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.tile_off_w), h->cap_tiles * 4));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->ws.tile_off_o), h->cap_tiles * 4));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->d_state), MAX_GROUP_TENSORS * sizeof(TensorState)));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->d_dstate), MAX_GROUP_TENSORS * sizeof(DecState)));
        ok = ok && check(h, cudaMalloc(reinterpret_cast<void**>(&h->d_call), sizeof(CallState)));
        ok = ok && check(h, cudaMallocHost(reinterpret_cast<void**>(&h->h_call), sizeof(CallState)));
        ok = ok && ensure_call_arrays(h, 1);
    }
    if (!ok) {
        excp_destroy(h);
        return EXCP_ERR_CUDA;
    }
    *out = h;
    return EXCP_OK;
}

excp_status excp_destroy(excp_handle h) {
    if (!h) return EXCP_OK;
    DeviceGuard guard(h->device);
    for (int k = 0; k < 3; ++k) {
        if (h->ws.surv[k]) cudaFree(h->ws.surv[k]);
        if (h->ws.bkt[k]) cudaFree(h->ws.bkt[k]);
    }
    if (h->ws.cst) cudaFree(h->ws.cst);
    if (h->km.pending) cudaFree(h->km.pending);
    for (int k = 0; k < 3; ++k) {
        if (h->km.rows[k]) cudaFree(h->km.rows[k]);
        if (h->km.pos[k]) cudaFree(h->km.pos[k]);
    }
    if (h->ws.bm_w) cudaFree(h->ws.bm_w);
    if (h->ws.bm_o) cudaFree(h->ws.bm_o);
    if (h->ws.tile_cnt_w) cudaFree(h->ws.tile_cnt_w);
    if (h->ws.tile_cnt_o) cudaFree(h->ws.tile_cnt_o);
    if (h->ws.tile_off_w) cudaFree(h->ws.tile_off_w);
    if (h->ws.tile_off_o) cudaFree(h->ws.tile_off_o);
    if (h->d_state) cudaFree(h->d_state);
    if (h->d_dstate) cudaFree(h->d_dstate);
    if (h->d_call) cudaFree(h->d_call);
    if (h->h_call) cudaFreeHost(h->h_call);
    free_call_arrays(h);
    for (int k = 0; k < 2; ++k) {
        for (int j = 0; j < 4; ++j) if (h->stage[k][j]) cudaFree(h->stage[k][j]);
        if (h->stage_blob[k]) cudaFree(h->stage_blob[k]);
        if (h->ev_h2d[k]) cudaEventDestroy(h->ev_h2d[k]);
        if (h->ev_compute[k]) cudaEventDestroy(h->ev_compute[k]);
        if (h->ev_d2h[k]) cudaEventDestroy(h->ev_d2h[k]);
    }
    if (h->s_h2d) cudaStreamDestroy(h->s_h2d);
    if (h->s_d2h) cudaStreamDestroy(h->s_d2h);
    for (cudaEvent_t e : h->prof.ev) cudaEventDestroy(e);
    delete h;
    return EXCP_OK;
}

size_t excp_record_bytes(size_t numel, size_t nnz_w, size_t nnz_o, int bits) {
    if (bits != 2 && bits != 4 && bits != 8 && bits != 32) return 0;
    return (size_t)record_bytes(numel, nnz_w, nnz_o, bits);
}

size_t excp_compress_bound(size_t numel, int bits) { return excp_record_bytes(numel, numel, numel, bits); }

const char* excp_status_string(excp_status s) {
    switch (s) {
        case EXCP_OK: return "ok";
        case EXCP_ERR_INVALID_ARG: return "invalid argument";
        case EXCP_ERR_UNSUPPORTED: return "unsupported code width";
        case EXCP_ERR_BUFFER_TOO_SMALL: return "output buffer too small";
        case EXCP_ERR_CUDA: return "CUDA error";
        case EXCP_ERR_CORRUPT_BLOB: return "corrupt record";
        case EXCP_ERR_NONFINITE_INPUT: return "non-finite input or negative second moment";
        case EXCP_ERR_TIMEOUT: return "timeout";
    }
    return "unknown status";
}

excp_status excp_last_cuda_error(excp_handle h, int* cuda_err) {
    if (!h || !cuda_err) return EXCP_ERR_INVALID_ARG;
    *cuda_err = h->last_cuda_error;
    return EXCP_OK;
}

static excp_status compress_impl(excp_handle h, const excp_params* params, size_t num_tensors,
                                 const void* const* w_t, const void* const* w_prev,
                                 const float* const* ea, const float* const* eas,
                                 const size_t* numel, int wfmt, void* blob_out, size_t blob_capacity,
                                 size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                 void* cuda_stream, const size_t* tensor_index = nullptr) {
    if (!h || !params || !tensor_offsets_out) return EXCP_ERR_INVALID_ARG;
    if (wfmt != WF_F32 && wfmt != WF_F16 && wfmt != WF_BF16) return EXCP_ERR_INVALID_ARG;
    if (num_tensors && (!w_t || !w_prev || !ea || !eas || !numel)) return EXCP_ERR_INVALID_ARG;
    if (!blob_out || !aligned16(blob_out)) return EXCP_ERR_INVALID_ARG;
    const excp_status ps = validate_params(params);
    if (ps != EXCP_OK) return ps;
    for (size_t i = 0; i < num_tensors; ++i) {
        if (numel[i] == 0) continue;
        const bool need_prev = !(params->flags & OPT_NO_RESIDUAL);     // without the residual W^_(t-1) is not read
        if (!w_t[i] || (need_prev && !w_prev[i]) || !ea[i] || !eas[i]) return EXCP_ERR_INVALID_ARG;
        if (!aligned16(w_t[i]) || !aligned16(w_prev[i]) || !aligned16(ea[i]) || !aligned16(eas[i]))
            return EXCP_ERR_INVALID_ARG;
    }
    tensor_offsets_out[0] = 0;
    if (num_tensors == 0) return EXCP_OK;

    std::vector<Group> groups;
    if (!make_groups(h, numel, num_tensors, groups)) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    if (!ensure_call_arrays(h, num_tensors)) return EXCP_ERR_CUDA;

    TensorDesc* hd = static_cast<TensorDesc*>(h->h_desc);
    for (const Group& g : groups) {
        u32 tile = 0;
        for (size_t i = g.first; i < g.first + g.count; ++i) {
            TensorDesc& d = hd[i];
            d.w_t = w_t[i]; d.w_prev = w_prev[i]; d.ea = ea[i]; d.eas = eas[i];
            d.numel = numel[i];
            d.tensor_index = tensor_index ? tensor_index[i] : i;
            d.tile_begin = tile;
            d.num_tiles = (u32)((numel[i] + TILE - 1) / TILE);
            tile += d.num_tiles;
        }
    }
    Params p = to_params(h, params);
    p.wfmt = wfmt;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, &h->prof};
    h->prof.begin(stream);
    TensorDesc* dd = static_cast<TensorDesc*>(h->d_desc);
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    ok = ok && check(h, cudaMemcpyAsync(dd, hd, num_tensors * sizeof(TensorDesc), cudaMemcpyHostToDevice, stream));
    for (size_t gi = 0; ok && gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        ok = run_group(h, cfg, dd + g.first, (int)g.count, g.tiles, p, static_cast<unsigned char*>(blob_out),
                       blob_capacity, h->d_results + g.first, stats_out != nullptr && h->report_sse);
    }
    ok = ok && check(h, cudaMemcpyAsync(h->h_results, h->d_results, num_tensors * sizeof(TensorResult),
                                        cudaMemcpyDeviceToHost, stream));
    ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
    if (!check(h, cudaStreamSynchronize(stream)) || !ok) return EXCP_ERR_CUDA;
    h->prof.finish();
    fill_outputs(h, 0, num_tensors, numel, 0, tensor_offsets_out, stats_out);
    return status_from_flags(h->h_call->flags);
}

excp_status excp_compress_checkpoint(excp_handle h, const excp_params* params, size_t num_tensors,
                                     const float* const* w_t, const float* const* w_prev,
                                     const float* const* ea, const float* const* eas,
                                     const size_t* numel, void* blob_out, size_t blob_capacity,
                                     size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                     void* cuda_stream) {
    return compress_impl(h, params, num_tensors, reinterpret_cast<const void* const*>(w_t),
                         reinterpret_cast<const void* const*>(w_prev), ea, eas, numel, WF_F32, blob_out, blob_capacity,
                         tensor_offsets_out, stats_out, cuda_stream);
}

excp_status excp_compress_checkpoint_indexed(excp_handle h, const excp_params* params, size_t num_tensors,
                                             const float* const* w_t, const float* const* w_prev,
                                             const float* const* ea, const float* const* eas,
                                             const size_t* numel, const size_t* tensor_index,
                                             void* blob_out, size_t blob_capacity,
                                             size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                             void* cuda_stream) {
    if (num_tensors && !tensor_index) return EXCP_ERR_INVALID_ARG;
    return compress_impl(h, params, num_tensors, reinterpret_cast<const void* const*>(w_t),
                         reinterpret_cast<const void* const*>(w_prev), ea, eas, numel, WF_F32, blob_out, blob_capacity,
                         tensor_offsets_out, stats_out, cuda_stream, tensor_index);
}

excp_status excp_compress_checkpoint_w16(excp_handle h, const excp_params* params, size_t num_tensors,
                                         const void* const* w_t, const void* const* w_prev,
                                         const float* const* ea, const float* const* eas,
                                         const size_t* numel, int weight_format, void* blob_out, size_t blob_capacity,
                                         size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                         void* cuda_stream) {
    if (weight_format != WF_F16 && weight_format != WF_BF16) return EXCP_ERR_INVALID_ARG;
    return compress_impl(h, params, num_tensors, w_t, w_prev, ea, eas, numel, weight_format, blob_out, blob_capacity,
                         tensor_offsets_out, stats_out, cuda_stream);
}

excp_status excp_compress_checkpoint_host(excp_handle h, const excp_params* params, size_t num_tensors,
                                          const float* const* w_t, const float* const* w_prev,
                                          const float* const* ea, const float* const* eas,
                                          const size_t* numel, void* blob_out, size_t blob_capacity,
                                          size_t* tensor_offsets_out, excp_tensor_stats* stats_out,
                                          void* cuda_stream) {
    if (!h || !params || !tensor_offsets_out || !blob_out) return EXCP_ERR_INVALID_ARG;
    if (num_tensors && (!w_t || !w_prev || !ea || !eas || !numel)) return EXCP_ERR_INVALID_ARG;
    const excp_status ps = validate_params(params);
    if (ps != EXCP_OK) return ps;
    if (params->flags & OPT_NO_QUANT) return EXCP_ERR_UNSUPPORTED;   // the record staging is sized for coded records
    for (size_t i = 0; i < num_tensors; ++i)
        if (numel[i] && (!w_t[i] || !w_prev[i] || !ea[i] || !eas[i])) return EXCP_ERR_INVALID_ARG;
    tensor_offsets_out[0] = 0;
    if (num_tensors == 0) return EXCP_OK;

    std::vector<Group> groups;
    if (!make_groups(h, numel, num_tensors, groups)) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    if (!ensure_call_arrays(h, num_tensors) || !ensure_host_path(h, params->bits)) return EXCP_ERR_CUDA;

    TensorDesc* hd = static_cast<TensorDesc*>(h->h_desc);
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        const int slot = (int)(gi & 1);
        u32 tile = 0;
        for (size_t i = g.first; i < g.first + g.count; ++i) {
            TensorDesc& d = hd[i];
            const size_t off = (size_t)tile * TILE;
            d.w_t = h->stage[slot][0] + off; d.w_prev = h->stage[slot][1] + off;
            d.ea = h->stage[slot][2] + off; d.eas = h->stage[slot][3] + off;
            d.numel = numel[i];
            d.tensor_index = i;
            d.tile_begin = tile;
            d.num_tiles = (u32)((numel[i] + TILE - 1) / TILE);
            tile += d.num_tiles;
        }
    }
    const Params p = to_params(h, params);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, &h->prof};
    h->prof.begin(stream);
    TensorDesc* dd = static_cast<TensorDesc*>(h->d_desc);
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    ok = ok && check(h, cudaMemcpyAsync(dd, hd, num_tensors * sizeof(TensorDesc), cudaMemcpyHostToDevice, stream));

    // copies of group g into its slot; the slot is free once group g-2 has been computed
    auto issue_h2d = [&](size_t gi) {
        const Group& g = groups[gi];
        const int slot = (int)(gi & 1);
        bool k = true;
        if (gi >= 2) k = check(h, cudaStreamWaitEvent(h->s_h2d, h->ev_compute[slot], 0));
        const float* const* src[4] = {w_t, w_prev, ea, eas};
        for (size_t i = g.first; k && i < g.first + g.count; ++i) {
            if (!numel[i]) continue;
            const size_t off = (size_t)hd[i].tile_begin * TILE;
            for (int j = 0; k && j < 4; ++j)
                k = check(h, cudaMemcpyAsync(h->stage[slot][j] + off, src[j][i], numel[i] * sizeof(float),
                                             cudaMemcpyHostToDevice, h->s_h2d));
        }
        return k && check(h, cudaEventRecord(h->ev_h2d[slot], h->s_h2d));
    };

    size_t host_off = 0;
    u32 flags = 0;
    ok = ok && issue_h2d(0);
    for (size_t gi = 0; ok && gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        const int slot = (int)(gi & 1);
        if (gi + 1 < groups.size()) ok = issue_h2d(gi + 1);
        ok = ok && check(h, cudaStreamWaitEvent(stream, h->ev_h2d[slot], 0));
        if (gi >= 2) ok = ok && check(h, cudaStreamWaitEvent(stream, h->ev_d2h[slot], 0));
        ok = ok && check(h, cudaMemsetAsync(&h->d_call->blob_cursor, 0, sizeof(u64), stream));
        ok = ok && run_group(h, cfg, dd + g.first, (int)g.count, g.tiles, p, h->stage_blob[slot],
                             h->stage_blob_bytes, h->d_results + g.first, stats_out != nullptr && h->report_sse);
        ok = ok && check(h, cudaMemcpyAsync(h->h_results + g.first, h->d_results + g.first,
                                            g.count * sizeof(TensorResult), cudaMemcpyDeviceToHost, stream));
        ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
        ok = ok && check(h, cudaEventRecord(h->ev_compute[slot], stream));
        ok = ok && check(h, cudaEventSynchronize(h->ev_compute[slot]));
        if (!ok) break;
        const size_t bytes = (size_t)h->h_call->blob_cursor;
        flags |= h->h_call->flags;
        // a group whose records outgrew the staging wrote none of them: nothing to copy
        if ((flags & FLAG_BLOB_FULL) || bytes > h->stage_blob_bytes) { flags |= FLAG_BLOB_FULL; break; }
        if (host_off + bytes > blob_capacity) { flags |= FLAG_BLOB_FULL; break; }
        ok = check(h, cudaStreamWaitEvent(h->s_d2h, h->ev_compute[slot], 0));
        ok = ok && check(h, cudaMemcpyAsync(static_cast<unsigned char*>(blob_out) + host_off, h->stage_blob[slot],
                                            bytes, cudaMemcpyDeviceToHost, h->s_d2h));
        ok = ok && check(h, cudaEventRecord(h->ev_d2h[slot], h->s_d2h));
        fill_outputs(h, g.first, g.count, numel, host_off, tensor_offsets_out, stats_out);
        host_off += bytes;
    }
    const bool s1 = check(h, cudaStreamSynchronize(h->s_h2d));
    const bool s2 = check(h, cudaStreamSynchronize(h->s_d2h));
    const bool s3 = check(h, cudaStreamSynchronize(stream));
    if (!ok || !s1 || !s2 || !s3) return EXCP_ERR_CUDA;
    h->prof.finish();
    return status_from_flags(flags);
}

excp_status excp_compress_tensor(excp_handle h, const excp_params* params,
                                 const float* w_t, const float* w_prev, const float* ea, const float* eas,
                                 size_t numel, void* blob_out, size_t blob_capacity,
                                 size_t* blob_bytes_out, excp_tensor_stats* stats_out, void* cuda_stream) {
    if (!blob_bytes_out) return EXCP_ERR_INVALID_ARG;
    size_t offs[2] = {0, 0};
    const excp_status s = excp_compress_checkpoint(h, params, 1, &w_t, &w_prev, &ea, &eas, &numel, blob_out,
                                                   blob_capacity, offs, stats_out, cuda_stream);
    *blob_bytes_out = offs[1] - offs[0];
    return s;
}

static excp_status decompress_impl(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                   size_t num_tensors, const void* const* w_prev, const size_t* numel, int wfmt,
                                   void* const* w_out, float* const* ea_out, float* const* eas_out,
                                   void* cuda_stream) {
    if (!h || !blob || !tensor_offsets || !aligned16(blob)) return EXCP_ERR_INVALID_ARG;
    if (num_tensors == 0) return EXCP_OK;
    if (!w_prev || !numel || !w_out || !ea_out || !eas_out) return EXCP_ERR_INVALID_ARG;
    for (size_t i = 0; i < num_tensors; ++i) {
        if (tensor_offsets[i + 1] < tensor_offsets[i] || (tensor_offsets[i] & 15u)) return EXCP_ERR_INVALID_ARG;
        if (numel[i] == 0) continue;
        if (!w_prev[i] || !w_out[i] || !ea_out[i] || !eas_out[i]) return EXCP_ERR_INVALID_ARG;
        if (!aligned16(w_prev[i]) || !aligned16(w_out[i]) || !aligned16(ea_out[i]) || !aligned16(eas_out[i]))
            return EXCP_ERR_INVALID_ARG;
    }
    std::vector<Group> groups;
    if (!make_groups(h, numel, num_tensors, groups)) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    if (!ensure_call_arrays(h, num_tensors)) return EXCP_ERR_CUDA;

    DecDesc* hd = static_cast<DecDesc*>(h->h_desc);
    const unsigned char* base = static_cast<const unsigned char*>(blob);
    for (const Group& g : groups) {
        u32 tile = 0;
        for (size_t i = g.first; i < g.first + g.count; ++i) {
            DecDesc& d = hd[i];
            d.rec = base + tensor_offsets[i];
            d.rec_avail = tensor_offsets[i + 1] - tensor_offsets[i];
            d.w_prev = w_prev[i]; d.w_out = w_out[i]; d.ea_out = ea_out[i]; d.eas_out = eas_out[i];
            d.numel = numel[i];
            d.tile_begin = tile;
            d.num_tiles = (u32)((numel[i] + TILE - 1) / TILE);
            tile += d.num_tiles;
        }
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, &h->prof};
    h->prof.begin(stream);
    DecDesc* dd = static_cast<DecDesc*>(h->d_desc);
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    ok = ok && check(h, cudaMemcpyAsync(dd, hd, num_tensors * sizeof(DecDesc), cudaMemcpyHostToDevice, stream));
    for (size_t gi = 0; ok && gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        launch_decode(cfg, dd + g.first, h->d_dstate, (int)g.count, g.tiles, h->ws, h->d_call, wfmt);
        ok = check(h, cudaGetLastError());
    }
    ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
    if (!check(h, cudaStreamSynchronize(stream)) || !ok) return EXCP_ERR_CUDA;
    h->prof.finish();
    return status_from_flags(h->h_call->flags);
}

excp_status excp_decompress_checkpoint(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                       size_t num_tensors, const float* const* w_prev, const size_t* numel,
                                       float* const* w_out, float* const* ea_out, float* const* eas_out,
                                       void* cuda_stream) {
    return decompress_impl(h, blob, tensor_offsets, num_tensors, reinterpret_cast<const void* const*>(w_prev), numel,
                           WF_F32, reinterpret_cast<void* const*>(w_out), ea_out, eas_out, cuda_stream);
}

excp_status excp_decompress_checkpoint_w16(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                           size_t num_tensors, const void* const* w_prev, const size_t* numel,
                                           int weight_format, void* const* w_out, float* const* ea_out,
                                           float* const* eas_out, void* cuda_stream) {
    if (weight_format != WF_F16 && weight_format != WF_BF16) return EXCP_ERR_INVALID_ARG;
    return decompress_impl(h, blob, tensor_offsets, num_tensors, w_prev, numel, weight_format, w_out, ea_out, eas_out,
                           cuda_stream);
}

excp_status excp_set_kmeans_margin(excp_handle h, int margin) {
    if (!h || margin < -1) return EXCP_ERR_INVALID_ARG;
    h->km_margin = margin;
    return EXCP_OK;
}

excp_status excp_set_report_sse(excp_handle h, int enable) {
    if (!h) return EXCP_ERR_INVALID_ARG;
    h->report_sse = enable != 0;
    return EXCP_OK;
}

excp_status excp_set_wait_limit(excp_handle h, unsigned long long nanoseconds) {
    if (!h) return EXCP_ERR_INVALID_ARG;
    h->wait_limit_ns = nanoseconds;
    return EXCP_OK;
}

excp_status excp_selftest_wait_timeout(excp_handle h, unsigned long long nanoseconds, void* cuda_stream) {
    if (!h || nanoseconds > 1000000000ull) return EXCP_ERR_INVALID_ARG;      // at most a second: this wait always runs out
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, nullptr};
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    if (ok) launch_wait_selftest(cfg, h->d_call, nanoseconds);
    ok = ok && check(h, cudaGetLastError());
    ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
    if (!check(h, cudaStreamSynchronize(stream)) || !ok) return EXCP_ERR_CUDA;
    return status_from_flags(h->h_call->flags);
}

excp_status excp_profile_enable(excp_handle h, int enable) {
    if (!h) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (enable && h->prof.ev.empty()) {
        h->prof.ev.resize(8192);
        h->prof.stage.assign(8192, 0);
        for (cudaEvent_t& e : h->prof.ev)
            if (!check(h, cudaEventCreate(&e))) return EXCP_ERR_CUDA;
    }
    h->prof.enabled = enable != 0;
    return EXCP_OK;
}

int excp_profile_stage_count(void) { return ST_COUNT; }

const char* excp_profile_stage_name(int stage) {
    static const char* names[ST_COUNT] = {
        "stats1", "stats2", "mask_compact", "scan_layout", "kmeans_start", "cell_count", "cell_gather",
        "kmeans_iterate", "cell_plan", "header_edges", "pack_codes", "copy_bitmaps", "dec_prep", "decode", "kmeans_retry", "dense"};
    return stage >= 0 && stage < ST_COUNT ? names[stage] : "";
}

excp_status excp_profile_read(excp_handle h, double* stage_ms_out, unsigned long long* launches_out) {
    if (!h) return EXCP_ERR_INVALID_ARG;
    if (stage_ms_out) for (int i = 0; i < ST_COUNT; ++i) stage_ms_out[i] = h->prof.ms[i];
    if (launches_out) *launches_out = h->prof.launches;
    return EXCP_OK;
}

excp_status excp_decompress_tensor(excp_handle h, const void* blob, size_t blob_bytes,
                                   const float* w_prev, size_t numel,
                                   float* w_out, float* ea_out, float* eas_out, void* cuda_stream) {
    const size_t offs[2] = {0, blob_bytes};
    return excp_decompress_checkpoint(h, blob, offs, 1, &w_prev, &numel, &w_out, &ea_out, &eas_out, cuda_stream);
}

size_t excp_dense_bytes(size_t numel, int bits) {
    if (bits != 2 && bits != 4 && bits != 8) return 0;
    return (size_t)dense_bytes(numel, bits);
}

excp_status excp_checkpoint_to_dense(excp_handle h, const void* blob, const size_t* tensor_offsets,
                                     size_t num_tensors, const size_t* numel, void* dense_out,
                                     size_t dense_capacity, size_t* dense_offsets_out, void* cuda_stream) {
    if (!h || !blob || !tensor_offsets || !aligned16(blob) || !dense_offsets_out) return EXCP_ERR_INVALID_ARG;
    dense_offsets_out[0] = 0;
    if (num_tensors == 0) return EXCP_OK;
    if (!numel || !dense_out || !aligned16(dense_out)) return EXCP_ERR_INVALID_ARG;
    for (size_t i = 0; i < num_tensors; ++i) {
        if (tensor_offsets[i + 1] < tensor_offsets[i] || (tensor_offsets[i] & 15u)) return EXCP_ERR_INVALID_ARG;
        dense_offsets_out[i + 1] = dense_offsets_out[i] + (size_t)dense_bytes(numel[i], 4);
    }
    if (dense_offsets_out[num_tensors] > dense_capacity) return EXCP_ERR_BUFFER_TOO_SMALL;
    std::vector<Group> groups;
    if (!make_groups(h, numel, num_tensors, groups)) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    if (!ensure_call_arrays(h, num_tensors)) return EXCP_ERR_CUDA;

    DecDesc* hd = static_cast<DecDesc*>(h->h_desc);
    const unsigned char* base = static_cast<const unsigned char*>(blob);
    for (const Group& g : groups) {
        u32 tile = 0;
        for (size_t i = g.first; i < g.first + g.count; ++i) {
            DecDesc& d = hd[i];
            d = DecDesc{};
            d.rec = base + tensor_offsets[i];
            d.rec_avail = tensor_offsets[i + 1] - tensor_offsets[i];
            d.dense = static_cast<unsigned char*>(dense_out) + dense_offsets_out[i];
            d.dense_avail = dense_offsets_out[i + 1] - dense_offsets_out[i];
            d.numel = numel[i];
            d.tile_begin = tile;
            d.num_tiles = (u32)((numel[i] + TILE - 1) / TILE);
            tile += d.num_tiles;
        }
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, &h->prof};
    h->prof.begin(stream);
    DecDesc* dd = static_cast<DecDesc*>(h->d_desc);
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    ok = ok && check(h, cudaMemcpyAsync(dd, hd, num_tensors * sizeof(DecDesc), cudaMemcpyHostToDevice, stream));
    for (size_t gi = 0; ok && gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        launch_record_to_dense(cfg, dd + g.first, h->d_dstate, (int)g.count, g.tiles, h->ws, h->d_call);
        ok = check(h, cudaGetLastError());
    }
    ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
    if (!check(h, cudaStreamSynchronize(stream)) || !ok) return EXCP_ERR_CUDA;
    h->prof.finish();
    return status_from_flags(h->h_call->flags);
}

excp_status excp_record_to_dense(excp_handle h, const void* record, size_t record_bytes, size_t numel,
                                 void* dense_out, size_t dense_capacity, size_t* dense_bytes_out,
                                 void* cuda_stream) {
    const size_t offs[2] = {0, record_bytes};
    size_t douts[2] = {0, 0};
    const excp_status s = excp_checkpoint_to_dense(h, record, offs, 1, &numel, dense_out, dense_capacity, douts,
                                                   cuda_stream);
    if (dense_bytes_out) *dense_bytes_out = douts[1];
    return s;
}

excp_status excp_decompress_dense_checkpoint(excp_handle h, const void* dense, const size_t* dense_offsets,
                                             size_t num_tensors, const float* const* w_prev, const size_t* numel,
                                             float* const* w_out, float* const* ea_out, float* const* eas_out,
                                             void* cuda_stream) {
    if (!h || !dense || !dense_offsets || !aligned16(dense)) return EXCP_ERR_INVALID_ARG;
    if (num_tensors == 0) return EXCP_OK;
    if (!w_prev || !numel || !w_out || !ea_out || !eas_out) return EXCP_ERR_INVALID_ARG;
    for (size_t i = 0; i < num_tensors; ++i) {
        if (dense_offsets[i + 1] < dense_offsets[i] || (dense_offsets[i] & 15u)) return EXCP_ERR_INVALID_ARG;
        if (numel[i] == 0) continue;
        if (!w_prev[i] || !w_out[i] || !ea_out[i] || !eas_out[i]) return EXCP_ERR_INVALID_ARG;
        if (!aligned16(w_prev[i]) || !aligned16(w_out[i]) || !aligned16(ea_out[i]) || !aligned16(eas_out[i]))
            return EXCP_ERR_INVALID_ARG;
    }
    std::vector<Group> groups;
    if (!make_groups(h, numel, num_tensors, groups)) return EXCP_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EXCP_ERR_CUDA;
    if (!ensure_call_arrays(h, num_tensors)) return EXCP_ERR_CUDA;

    DecDesc* hd = static_cast<DecDesc*>(h->h_desc);
    const unsigned char* base = static_cast<const unsigned char*>(dense);
    for (const Group& g : groups) {
        u32 tile = 0;
        for (size_t i = g.first; i < g.first + g.count; ++i) {
            DecDesc& d = hd[i];
            d = DecDesc{};
            d.rec = base + dense_offsets[i];
            d.rec_avail = dense_offsets[i + 1] - dense_offsets[i];
            d.w_prev = w_prev[i]; d.w_out = w_out[i]; d.ea_out = ea_out[i]; d.eas_out = eas_out[i];
            d.numel = numel[i];
            d.tile_begin = tile;
            d.num_tiles = (u32)((numel[i] + TILE - 1) / TILE);
            tile += d.num_tiles;
        }
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    LaunchCfg cfg{h->sms, stream, &h->prof};
    h->prof.begin(stream);
    DecDesc* dd = static_cast<DecDesc*>(h->d_desc);
    bool ok = check(h, cudaMemsetAsync(h->d_call, 0, sizeof(CallState), stream));
    ok = ok && check(h, cudaMemcpyAsync(dd, hd, num_tensors * sizeof(DecDesc), cudaMemcpyHostToDevice, stream));
    for (size_t gi = 0; ok && gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        launch_dense_decode(cfg, dd + g.first, h->d_dstate, (int)g.count, g.tiles, h->d_call);
        ok = check(h, cudaGetLastError());
    }
    ok = ok && check(h, cudaMemcpyAsync(h->h_call, h->d_call, sizeof(CallState), cudaMemcpyDeviceToHost, stream));
    if (!check(h, cudaStreamSynchronize(stream)) || !ok) return EXCP_ERR_CUDA;
    h->prof.finish();
    return status_from_flags(h->h_call->flags);
}

excp_status excp_decompress_dense_tensor(excp_handle h, const void* dense, size_t dense_bytes_in,
                                         const float* w_prev, size_t numel,
                                         float* w_out, float* ea_out, float* eas_out, void* cuda_stream) {
    const size_t offs[2] = {0, dense_bytes_in};
    return excp_decompress_dense_checkpoint(h, dense, offs, 1, &w_prev, &numel, &w_out, &ea_out, &eas_out,
                                            cuda_stream);
}

}  // extern "C"
