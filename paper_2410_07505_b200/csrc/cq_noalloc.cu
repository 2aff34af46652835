// cq_quantize_act_noalloc: the activation quantizer for callers that cannot allocate device memory.
//
// cq_quantize_act needs a few megabytes of device scratch (scale vectors, their reciprocals, the
// partial maxima of the first pass) and asks the caller for it.  Some callers have nowhere to get it:
// a serving process that handed the whole GPU to one pool at start-up, a plug-in running on a hot path
// where the host framework forbids cudaMalloc (it synchronises the device and can fail when memory is
// fragmented), a component whose memory budget was fixed before it was loaded.  For them this file
// keeps the scratch inside the library image: one fixed array per GPU, held from the moment the CUDA
// runtime has loaded this file's device code on that GPU (at the latest during the first call there,
// which should therefore come early) until the process exits.
#include <cuda_runtime.h>

#include <mutex>

#include "cq.h"
#include "cq_host.h"

namespace {

// The array itself.  Its name is only meaningful to device code; host code must ask the runtime for
// the address it has on the current device (cudaGetSymbolAddress) and hand that to the kernels.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CQ_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_address[kMaxDevices];   // per device: where g_noalloc_scratch lives, nullptr until looked up
std::mutex g_scratch_mutex;

// Looks the array's device address up once per device, with that device current.
int scratch_of_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_address[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) return CQ_ERR_CUDA;
        g_scratch_address[dev] = p;
    }
    *out = g_scratch_address[dev];
    return CQ_OK;
}

}  // namespace

extern "C" int cq_quantize_act_noalloc(const void* X, int dtype, int64_t T, int64_t I, int64_t ld,
                                       double alpha, int bits,
                                       float* t, float* c, float* row_scale, float* col_scale,
                                       void* codes, void* deq, int deq_dtype,
                                       unsigned long long* zero_count, void* stream) {
    if (T < 0 || I < 0) return CQ_ERR_SHAPE;
    // Shapes whose scratch does not fit in the fixed array are refused here, before anything is enqueued.
    const size_t need = cq_workspace_bytes(T, I);
    if (need == 0 || need > static_cast<size_t>(CQ_NOALLOC_SCRATCH_BYTES)) return CQ_ERR_TOO_LARGE;
    void* scratch = nullptr;
    const int rc = scratch_of_current_device(&scratch);
    if (rc != CQ_OK) return rc;
    // Nothing in the scratch has to start at zero: every word the kernels read from it in this call
    // is written earlier in the same call (partial maxima by the first pass, vectors by the second
    // kernel), so the previous call's contents are simply overwritten.
    return cq::quantize_act_impl(X, dtype, T, I, ld, alpha, bits, nullptr, nullptr, t, c, row_scale, col_scale,
                                 codes, deq, deq_dtype, zero_count, scratch, CQ_NOALLOC_SCRATCH_BYTES,
                                 static_cast<cudaStream_t>(stream));
}
