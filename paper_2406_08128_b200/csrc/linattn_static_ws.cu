// chela_linattn_fwd_static_ws: chela_linattn_fwd for callers that cannot hand the library a workspace.
//
// Some hosts of this library own no device allocator of their own: an inference-server plug-in whose
// process gave every byte of device memory to another framework's pool at start-up, a latency-critical
// loop where cudaMalloc (which may synchronise the whole device) is forbidden after initialisation, a
// component that is only ever handed finished input and output buffers.  For them the scratch the
// tensor-core path needs (the asynchronous status word and the per-group state sums of sequences that
// are split along L) lives in a fixed array that is part of the library image, below.
#include <mutex>

#include "common.cuh"

namespace {

// Built-in scratch: 8 MiB per GPU that loads the library, held until the process exits.
constexpr size_t kStaticWsBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_ws_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device.  In host code `g_static_ws` is only a
// handle for the runtime, not an address a kernel could use, so the address is looked up once per device
// (with that device current) and cached.
chela_status_t static_ws_pointer(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CHELA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_ws_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return CHELA_ERR_CUDA;
        g_ws_ptr[dev] = p;
    }
    *out = g_ws_ptr[dev];
    return CHELA_OK;
}

}  // namespace

extern "C" chela_status_t chela_linattn_fwd_static_ws(const void *q, const void *k, const void *v, void *o, int B,
                                                      int H, int L, int d_k, int d_v, int chunk,
                                                      chela_dtype_t in_dtype, chela_dtype_t out_dtype,
                                                      chela_norm_t norm, float norm_eps, float scale,
                                                      cudaStream_t stream)
{
    const size_t need = chela_linattn_workspace_bytes(B, H, L, d_k, d_v, chunk);
    if (need > kStaticWsBytes) return CHELA_ERR_WORKSPACE;   // beyond the built-in scratch: use chela_linattn_fwd
    void *ws = nullptr;
    const chela_status_t st = static_ws_pointer(&ws);
    if (st != CHELA_OK) return st;
    // The status word is cleared on the stream by the launch itself; the state sums are written by the
    // state kernel before the main kernel reads them, so nothing else has to start at zero.
    return chela_linattn_fwd(q, k, v, o, B, H, L, d_k, d_v, chunk, in_dtype, out_dtype, norm, norm_eps, scale, ws,
                             kStaticWsBytes, stream);
}

// The asynchronous status word of the last chela_linattn_fwd_static_ws call on the current device (no allocation: one
// word copied into a stack variable).
extern "C" chela_status_t chela_linattn_static_ws_status(cudaStream_t stream)
{
    void *ws = nullptr;
    const chela_status_t st = static_ws_pointer(&ws);
    if (st != CHELA_OK) return st;
    return chela_async_status(ws, stream);
}
