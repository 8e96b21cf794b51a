// gta_decode_static: the decode step for callers that cannot hand the library a workspace.
//
// Some hosts of this library have no way to allocate device memory when a decode step is due: a
// serving process whose memory pool claimed the whole device at start-up (a later cudaMalloc
// simply fails), a plug-in that is not allowed to touch the host application's allocator, or a
// latency-critical loop in which the implicit device-wide synchronisation of cudaMalloc / cudaFree
// is not acceptable.  For them the split-KV partial results of the decode kernels live in one
// fixed array that is part of the library image instead of a caller-provided workspace.
#include <mutex>

#include "gta_common.cuh"

namespace {

// The scratch array.  Every GPU that loads the library holds these bytes until the process
// exits, so the size is kept modest: it covers the bf16 decode workloads up to batch 128 with
// 8 maps of 1024 latent columns, not arbitrarily large problems.
static __device__ __align__(256) unsigned char g_decode_scratch[GTA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_decode_scratch, per device ordinal

// In host code `g_decode_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use is asked for once per device, with that device current.
gta_status_t scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GTA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) {
            cudaGetLastError();   // leave no sticky error behind for the caller's next call
            return GTA_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return GTA_OK;
}

}  // namespace

extern "C" gta_status_t gta_decode_static(const gta_shape_t* shape, const void* q, const void* k_cache,
                                          const void* c_cache, const int32_t* seq_lens, int32_t S_cap,
                                          const void* x_t, const void* w_p, const void* w_g, void* out,
                                          int32_t* status_word, void* cuda_stream) {
    // The same host-side checks as gta_decode, in the same order, so that both calls answer a bad
    // argument alike; nothing of CUDA has been touched yet.
    gta::Dims d;
    bool empty = false;
    gta_status_t st = gta::decode_check_args(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                             status_word, &d, &empty);
    if (st != GTA_OK) return st;
    if (empty) return GTA_OK;
    // Size check, still on the host: a problem that does not fit the built-in array is refused,
    // never truncated.
    if (gta_decode_workspace_bytes(shape, S_cap) > (size_t)GTA_STATIC_SCRATCH_BYTES) return GTA_ERR_STATIC_SCRATCH;
    if ((st = gta::check_current_device()) != GTA_OK) return st;
    // Only a call that will launch looks the array up (the first one on a device loads it).
    void* scratch = nullptr;
    if ((st = scratch_address(&scratch)) != GTA_OK) return st;
    // Same kernels as gta_decode; they write every scratch word before reading it, so nothing in
    // the array has to be cleared between calls.
    return gta_decode(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, scratch,
                      (size_t)GTA_STATIC_SCRATCH_BYTES, status_word, cuda_stream);
}
