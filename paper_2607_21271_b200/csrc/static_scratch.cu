// eqlinear_bwd_weight_static: the weight gradient for callers that cannot hand the library a scratch
// buffer because they cannot allocate device memory at the point of the call.
//
// The split partial spectra that eqlinear_bwd_weight keeps in caller-provided scratch live here in a
// fixed array that is part of the library image.  A GPU holds the array (EQL_STATIC_SCRATCH_BYTES)
// from the moment this translation unit's module is loaded on it until the process exits.  CUDA
// loads modules lazily, and this module has no kernel of its own, so that moment is the first
// look-up of the array's address on the device: eqlinear_plan does that look-up, which keeps the
// load -- and the reservation of the array's memory that comes with it -- out of every later call.
#include <mutex>

#include "eql_internal.h"

namespace {

// File-scope device array.  In host code this name is only a host-side handle for the symbol, NOT a
// device address: the address is looked up per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[EQL_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

}  // namespace

namespace eql {

void* static_scratch_address(int device, cudaError_t* err) {
    cudaError_t dummy;
    if (err == nullptr) err = &dummy;
    *err = cudaSuccess;
    if (device < 0 || device >= kMaxDevices) { *err = cudaErrorInvalidDevice; return nullptr; }
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[device] == nullptr) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            *err = (e != cudaSuccess) ? e : cudaErrorInvalidSymbol;
            cudaGetLastError();                    // the failure is reported through *err, not left as a sticky-looking error
            return nullptr;
        }
        g_scratch_addr[device] = ptr;
    }
    return g_scratch_addr[device];
}

}  // namespace eql

extern "C" eql_status_t eqlinear_bwd_weight_static(eqlinear_plan_t plan, const void* x, const void* dy, void* dw,
                                                   void* db, int64_t N, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;   // also: the plan's GPU must be current
    if (N < 0) return EQL_ERR_INVALID_ARG;
    size_t need = 0;
    eql_status_t st = eqlinear_bwd_weight_scratch_bytes(plan, N, &need);
    if (st != EQL_OK) return st;
    if (N > 0 && need > (size_t)EQL_STATIC_SCRATCH_BYTES) return EQL_ERR_WORKSPACE;   // beyond the built-in array

    cudaError_t e;
    void* scratch = eql::static_scratch_address(plan->device, &e);   // cached by eqlinear_plan on this device
    if (scratch == nullptr) return EQL_ERR_CUDA;
    return eqlinear_bwd_weight(plan, x, dy, dw, db, N, scratch, (size_t)EQL_STATIC_SCRATCH_BYTES, stream);
}
