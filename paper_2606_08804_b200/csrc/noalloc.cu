// Forward entry point that needs no workspace from its caller and allocates nothing.
//
// Who needs it: callers that cannot allocate device memory at the point of the call -- an inference
// server that has handed all free HBM to its own cache pool at start-up (a workspace request would
// fail or force the pool to shrink), or code running where an allocation's implicit device-wide
// synchronisation is not acceptable (between latency-critical launches of other streams).  For those,
// the scratch the chunkwise forward needs (decay prefix, diag(gamma)Q, P, W~^T, U~^T, status word) lives
// in a fixed array that is part of this library's device image, sized for short prompts.
//
// Rules of the shared array:
//  * one array per device; every call on that device uses it, so two calls that overlap in time (on
//    different streams, or from different threads) race on it -- callers serialise them, e.g. by
//    issuing them on one stream;
//  * nothing in it needs a particular value between calls except the status word (first 256 bytes),
//    which must start at zero: each call clears it on the caller's stream before its first kernel;
//  * the first call on a device performs the set-up below (it looks up the array's address; the
//    driver may load this module at that moment), so the first call on each device should be made
//    before any stream capture begins;
//  * no call here uses cudaMalloc/cudaFree or any allocating library routine.  (The per-kernel timing
//    aid of the library creates events when it is switched on; leave it off with this entry point.)
#include <cuda_runtime.h>

#include <mutex>

#include "internal.h"

namespace {

constexpr size_t kStaticScratchBytes = QDELTA_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices];          // address of the array on each device, once looked up

// Address of the array on the current device; looked up once per device with that device current.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return QD_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return QD_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
        if (e != cudaSuccess || !p) return QD_ERR_CUDA;
        if ((uintptr_t)p & 255) return QD_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return QD_OK;
}

}  // namespace

extern "C" int qdelta_chunk_fwd_static(const qd_shape* shape, const void* q, const void* k, const void* v,
                                       const void* beta, const void* alpha, const void* lambda, const float* h0,
                                       void* o, float* hT, unsigned* status_out, qd_stream stream) {
    const int src = qd::check_shape(shape);                         // the same code qdelta_chunk_fwd reports for a bad shape
    if (src != QD_OK) return src;
    if (status_out && ((uintptr_t)status_out & 3)) return QD_ERR_INVALID_ARG;
    const size_t need = qdelta_chunk_workspace_bytes(shape, 0);
    if (need == 0) return QD_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return QD_ERR_STATIC_SCRATCH;    // larger than the built-in array
    void* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != QD_OK) return rc;
    // the forward proper: clears the status word, then runs its kernels with the array as workspace
    const int frc = qdelta_chunk_fwd(shape, q, k, v, beta, alpha, lambda, h0, o, hT, scratch, kStaticScratchBytes, 0u, stream);
    if (frc != QD_OK) return frc;
    if (status_out &&
        cudaMemcpyAsync(status_out, scratch, sizeof(unsigned), cudaMemcpyDeviceToDevice, (cudaStream_t)stream) != cudaSuccess)
        return QD_ERR_CUDA;
    return QD_OK;
}
