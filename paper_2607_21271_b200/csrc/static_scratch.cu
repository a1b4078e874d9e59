// eqlinear_bwd_weight_static: the weight gradient for callers that cannot hand the library a scratch
// buffer because they cannot allocate device memory at the point of the call.
//
// The split partial spectra that eqlinear_bwd_weight keeps in caller-provided scratch live here in a
// fixed array that is part of the library image.  Every GPU on which this library is loaded holds the
// array (EQL_STATIC_SCRATCH_BYTES) from the moment the module is loaded until the process exits.
#include <mutex>

#include "eql_internal.h"

namespace {

// File-scope device array.  In host code this name is only a host-side handle for the symbol, NOT a
// device address: the address is looked up per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[EQL_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the CURRENT device; looked up once per device, with that device
// current, and cached.  Returns nullptr and sets *err on failure.
void* static_scratch_address(int device, cudaError_t* err) {
    *err = cudaSuccess;
    if (device < 0 || device >= kMaxDevices) { *err = cudaErrorInvalidDevice; return nullptr; }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[device] == nullptr) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) { *err = (e != cudaSuccess) ? e : cudaErrorInvalidSymbol; return nullptr; }
        g_scratch_addr[device] = ptr;
    }
    return g_scratch_addr[device];
}

}  // namespace

extern "C" eql_status_t eqlinear_bwd_weight_static(eqlinear_plan_t plan, const void* x, const void* dy, void* dw,
                                                   void* db, int64_t N, void* stream) {
    if (!plan) return EQL_ERR_INVALID_ARG;
    if (N < 0) return EQL_ERR_INVALID_ARG;
    size_t need = 0;
    eql_status_t st = eqlinear_bwd_weight_scratch_bytes(plan, N, &need);
    if (st != EQL_OK) return st;
    if (N > 0 && need > (size_t)EQL_STATIC_SCRATCH_BYTES) return EQL_ERR_WORKSPACE;   // beyond the built-in array

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return EQL_ERR_CUDA;
    if (dev != plan->device) return EQL_ERR_INVALID_ARG;          // the plan's workspace lives on another GPU
    cudaError_t e;
    void* scratch = static_scratch_address(dev, &e);
    if (scratch == nullptr) return EQL_ERR_CUDA;
    return eqlinear_bwd_weight(plan, x, dy, dw, db, N, scratch, (size_t)EQL_STATIC_SCRATCH_BYTES, stream);
}
