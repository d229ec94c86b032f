// rkv_compress_static: the whole compression step with its scratch in a static device array, for callers
// that have no way of handing over a workspace.  See include/rkv.h for the contract.
//
// The array below is part of the library's device image: every GPU that loads the library holds
// RKV_STATIC_SCRATCH_BYTES of it until the process exits, whether or not this entry point is ever called.
#include <mutex>

#include "rkv_common.cuh"

namespace rkv {

namespace {

// Scratch of every rkv_compress_static call on this device.  In host code this name is only a handle for
// the runtime's symbol lookup -- it is NOT a device address and must never be given to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[RKV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_lock;
void *g_scratch_ptr[kMaxDevices];      // device address of g_static_scratch on device d, once looked up
bool g_scratch_ready[kMaxDevices];

// Device address of the scratch array on the current device.  The first call on a device asks the runtime
// for it (which also makes the runtime load this library's device image there); later calls read the cache.
int scratch_address(void **out, cudaStream_t stream)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RKV_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_scratch_ready[dev]) {
        // the lookup may load the device image: not something to do in the middle of a stream capture
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(stream, &capturing);
        if (e != cudaSuccess) return RKV_ERR_CUDA;
        if (capturing != cudaStreamCaptureStatusNone) return RKV_ERR_INVALID_ARG;
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) return RKV_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_ptr[dev];
    return RKV_OK;
}

}  // namespace
}  // namespace rkv

using namespace rkv;

extern "C" {

int rkv_compress_static(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                        int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                        int32_t *out_idx, void *stream)
{
    if (!desc) return RKV_ERR_INVALID_ARG;
    // size check first: a shape that does not fit is refused without touching the device
    const size_t need = rkv_workspace_bytes(desc, budget, buffer, alpha);
    if (need == 0) {
        // bad shape: the ordinary argument checks name the problem (invalid or unsupported) before any launch
        rkv_desc_t probe = *desc;
        probe.workspace = nullptr;
        probe.workspace_bytes = 0;
        return rkv_compress_ex(&probe, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lambda, out_idx,
                               stream);
    }
    if (need > (size_t)RKV_STATIC_SCRATCH_BYTES) return RKV_ERR_WORKSPACE;
    void *scratch = nullptr;
    const int rc = scratch_address(&scratch, static_cast<cudaStream_t>(stream));
    if (rc != RKV_OK) return rc;
    rkv_desc_t inner = *desc;       // the caller's workspace fields, if any, are ignored
    inner.workspace = scratch;
    inner.workspace_bytes = RKV_STATIC_SCRATCH_BYTES;
    return rkv_compress_ex(&inner, k_cache, v_cache, q_window, seq_lens, budget, buffer, alpha, lambda, out_idx,
                           stream);
}

}  // extern "C"
