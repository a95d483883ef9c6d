// excp_decompress_tensor_noalloc: Algorithm 2 for one tensor without a handle and without
// allocating anything.  The decode kernels need a little scratch memory (per-tile survivor
// counts and offsets, the parsed header, an error flag); here it lives in a file-scope device
// array of fixed size, which every GPU that loads the library holds until the process ends.
//
// Why: restoring a checkpoint often happens in places where memory cannot be asked for --
// a training job whose framework allocator has already reserved the whole device (cudaMalloc
// fails there), or a recovery path that must not run into the device-wide synchronisation of
// cudaMalloc / cudaFree while other streams are busy.  Such a caller owns its input and output
// buffers already; this entry point needs nothing more.
//
// The array is shared by every call on the device and keeps what the last call left in it:
// the parts that must start at zero are cleared by the call itself, and two calls that overlap
// on the GPU (different streams, or different host threads) would race on it.
#include <mutex>

#include "../../include/excp.h"
#include "excp_common.cuh"

using namespace excp;

namespace {

constexpr u32 NA_MAX_TILES = EXCP_NOALLOC_MAX_NUMEL / TILE;
constexpr size_t NA_OFF_CALL = 0;                       // CallState
constexpr size_t NA_OFF_DESC = 256;                     // DecDesc
constexpr size_t NA_OFF_STATE = 512;                    // DecState
constexpr size_t NA_OFF_TILES = 4096;                   // 4 arrays of NA_MAX_TILES u32
constexpr size_t NA_BYTES = NA_OFF_TILES + 4ull * sizeof(u32) * NA_MAX_TILES;
static_assert(sizeof(CallState) <= 256 && sizeof(DecDesc) <= 256 && sizeof(DecState) <= 3584, "scratch layout");

// In host code this name is only a handle for cudaGetSymbolAddress, never an address to pass on.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_BYTES];

// Writes the call's descriptor and clears the error flag (both live in the scratch array).
__global__ void noalloc_setup_kernel(DecDesc d) {
    *reinterpret_cast<DecDesc*>(g_noalloc_scratch + NA_OFF_DESC) = d;
    CallState* c = reinterpret_cast<CallState*>(g_noalloc_scratch + NA_OFF_CALL);
    c->blob_cursor = 0;
    c->flags = 0;
}

constexpr int NA_MAX_DEVICES = 64;
struct PerDevice {
    unsigned char* base = nullptr;   // device address of g_noalloc_scratch on this device
    int sms = 0;
};
PerDevice g_dev[NA_MAX_DEVICES];
std::mutex g_dev_mutex;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" excp_status excp_decompress_tensor_noalloc(const void* blob, size_t blob_bytes, const float* w_prev,
                                                      size_t numel, float* w_out, float* ea_out, float* eas_out,
                                                      void* cuda_stream) {
    if (!blob || !aligned16(blob)) return EXCP_ERR_INVALID_ARG;
    if (numel > EXCP_NOALLOC_MAX_NUMEL) return EXCP_ERR_INVALID_ARG;        // beyond the fixed scratch
    if (numel && (!w_prev || !w_out || !ea_out || !eas_out)) return EXCP_ERR_INVALID_ARG;
    if (numel && (!aligned16(w_prev) || !aligned16(w_out) || !aligned16(ea_out) || !aligned16(eas_out)))
        return EXCP_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return EXCP_ERR_CUDA;

    // once per device, with that device current: the array's device address and the SM count
    PerDevice pd;
    {
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (!g_dev[dev].base) {
            unsigned char* p = nullptr;
            if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch) != cudaSuccess || !p)
                return EXCP_ERR_CUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
                return EXCP_ERR_CUDA;
            g_dev[dev].base = p;
            g_dev[dev].sms = sms;
        }
        pd = g_dev[dev];
    }

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    DecDesc d{};
    d.rec = static_cast<const unsigned char*>(blob);
    d.rec_avail = blob_bytes;
    d.w_prev = w_prev; d.w_out = w_out; d.ea_out = ea_out; d.eas_out = eas_out;
    d.numel = numel;
    d.tile_begin = 0;
    d.num_tiles = (u32)((numel + TILE - 1) / TILE);

    Workspace ws{};                                        // only the per-tile arrays are used by decode
    u32* tiles = reinterpret_cast<u32*>(pd.base + NA_OFF_TILES);
    ws.tile_cnt_w = tiles;
    ws.tile_cnt_o = tiles + NA_MAX_TILES;
    ws.tile_off_w = tiles + 2 * NA_MAX_TILES;
    ws.tile_off_o = tiles + 3 * NA_MAX_TILES;
    CallState* call = reinterpret_cast<CallState*>(pd.base + NA_OFF_CALL);

    noalloc_setup_kernel<<<1, 1, 0, stream>>>(d);
    LaunchCfg cfg{pd.sms, stream, nullptr};
    launch_decode(cfg, reinterpret_cast<const DecDesc*>(pd.base + NA_OFF_DESC),
                  reinterpret_cast<DecState*>(pd.base + NA_OFF_STATE), 1, d.num_tiles, ws, call);
    if (cudaGetLastError() != cudaSuccess) return EXCP_ERR_CUDA;
    CallState host_call;                                   // read the flag back (no allocation: plain copy)
    if (cudaMemcpyAsync(&host_call, call, sizeof(CallState), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return EXCP_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return EXCP_ERR_CUDA;
    if (host_call.flags & FLAG_TIMEOUT) return EXCP_ERR_TIMEOUT;
    if (host_call.flags & FLAG_CORRUPT) return EXCP_ERR_CORRUPT_BLOB;
    return EXCP_OK;
}
