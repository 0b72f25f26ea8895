// gdn_bwd for callers that cannot allocate device memory: the workspace is a fixed array inside the library.
#include "gdn_internal.cuh"

namespace {

// Scratch shared by every call of gdn_bwd_noalloc on a device.  It exists once per GPU that loads this library
// and is held until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_ws[GDN_NOALLOC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_ws_addr[kMaxDevices] = {};   // device address of g_noalloc_ws, per device ordinal (0 = not looked up yet)

}  // namespace

// Device address of the array on the current device (looked up once per device), or NULL if CUDA refuses.
static void* scratch_address() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (!g_ws_addr[dev]) {
        // In host code the array's name is only a handle; the kernels need its address on the current device.
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_ws) != cudaSuccess || !ptr) return nullptr;
        g_ws_addr[dev] = ptr;
    }
    return g_ws_addr[dev];
}

extern "C" gdn_status gdn_bwd_noalloc(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g,
                                      const float* beta, const float* h0, const void* dO, const float* dhT,
                                      const int32_t* cu_seqlens_dev, void* dq, void* dk, void* dv, float* dg, float* dbeta,
                                      float* dh0, void* cuda_stream) {
    size_t need = 0;
    gdn_status s = gdn_workspace_bytes(desc, nullptr, &need);
    if (s != GDN_OK) return s;
    if (need > (size_t)GDN_NOALLOC_WORKSPACE_BYTES) return GDN_ERR_WORKSPACE_TOO_SMALL;   // beyond the built-in scratch
    void* ws = scratch_address();
    if (!ws) return GDN_ERR_CUDA;
    // every argument error is refused here, before anything is enqueued
    s = gdn::check_bwd_args(desc, q, k, v, g, beta, h0, dO, dhT, cu_seqlens_dev, dq, dk, dv, dg, dbeta, dh0, ws,
                            (size_t)GDN_NOALLOC_WORKSPACE_BYTES);
    if (s != GDN_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left.  Only the header (status word, chunk count) has to start from
    // zero; every other region is written before it is read.
    if (cudaMemsetAsync(ws, 0, 256, st) != cudaSuccess) return GDN_ERR_CUDA;
    return gdn_bwd(desc, q, k, v, g, beta, h0, dO, dhT, cu_seqlens_dev, dq, dk, dv, dg, dbeta, dh0, ws,
                   (size_t)GDN_NOALLOC_WORKSPACE_BYTES, /*workspace_is_fresh_from_fwd=*/0, cuda_stream);
}

extern "C" gdn_status gdn_noalloc_last_device_status(void* cuda_stream) {
    void* ws = scratch_address();
    if (!ws) return GDN_ERR_CUDA;
    return gdn_last_device_status(ws, cuda_stream);   // a 4-byte copy into a host variable: nothing is allocated
}
