// Internal declarations shared by the translation units of libeqlinear (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "../../include/eqlinear.h"

namespace eql {

constexpr int kNumSMs = 148;            // B200
constexpr size_t kWsAlign = 256;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Device workspace layout of a plan (offsets in bytes from the workspace base).
struct WorkspaceLayout {
    size_t status;        // int32 status word (+ padding)
    size_t bias;          // float [Co]
    size_t planes_fwd;    // float [T][Ci][Co]   pre-scaled spectral weight, forward operand order
    size_t planes_bwd;    // float [T][Co][Ci]   conjugated, data-gradient operand order
    size_t umma_fwd;      // half  tensor-core operand image for fwd       (FP16 plans only)
    size_t umma_bwd;      // half  tensor-core operand image for bwd_data  (FP16 plans only)
    size_t umma_fwd_bytes, umma_bwd_bytes;
    size_t total;
};
// T: length of a group tuple (the cyclic order, or 2 x rotations for a dihedral plan, which has no tensor-core images)
WorkspaceLayout workspace_layout(int T, int Ci, int Co, eql_dtype_t dtype, bool tensor_cores = true);

// Raises a kernel's dynamic shared-memory limit once per device.  One object per kernel instantiation (a function-local
// static of the launcher); safe to use from several host threads: a bit is published only after the attribute call
// has returned, and setting the attribute twice is harmless.
struct SmemLimitOnce {
    std::atomic<unsigned long long> done{0};
    template <class Kernel>
    cudaError_t ensure(Kernel kernel, int bytes) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        if ((done.load(std::memory_order_acquire) >> dev) & 1ull) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
        done.fetch_or(1ull << dev, std::memory_order_release);
        return cudaSuccess;
    }
};

// Group orders the library is built for: every order up to 8, and 12, 16, 32.  The powers of two use butterflies and (4
// to 32, 2 not) the tensor-core kernels; the others run the CUDA-core kernels with a table-driven transform.
// Launches `kernel` so that it may start while the kernel before it in the stream is finishing (programmatic dependent
// launch); the kernel must call ptx::grid_dependency_wait() before its first access to global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline bool supported_T(int T) { return (T >= 1 && T <= 8) || T == 12 || T == 16 || T == 32; }

// ---- CUDA-core (FFMA) kernels, direct_kernels.cu -------------------------------------------------
// Spectral weight: w[Co][Ci][T] -> planes_fwd[T][Ci][Co], planes_bwd[T][Co][Ci] (float), bias -> float.
cudaError_t launch_plan_weights(int T, eql_dtype_t dtype, bool correlation, const void* w, const void* bias,
                                int Ci, int Co, float* planes_fwd, float* planes_bwd, float* bias_f32,
                                cudaStream_t stream);

// out[N, Cout*T] = inverse_dft( dft(in[N, Cin*T]) (x) planes[T][Cin][Cout] ) + bias   (bias may be NULL)
cudaError_t launch_direct_linear(int T, eql_dtype_t dtype, const void* in, void* out, int64_t N,
                                 int Cin, int Cout, const float* planes, const float* bias_f32,
                                 cudaStream_t stream, int act = 0);

// Split-K layout of the weight-gradient reduction.
struct BwdWeightSplit {
    int splits;               // number of token ranges
    int64_t tokens_per_split; // multiple of the kernel's token chunk
    size_t scratch_bytes;     // splits * (T*Co*Ci + Co) floats, rounded up
};
BwdWeightSplit direct_bwd_weight_split(int T, int Ci, int Co, int64_t N);

// Partial spectra part[split][T][Co][Ci], db partials [split][Co] -> dw[Co][Ci][T], db[Co].
cudaError_t launch_direct_bwd_weight(int T, eql_dtype_t dtype, bool correlation, const void* x, const void* dy,
                                     float* dw, float* db, int64_t N, int Ci, int Co,
                                     const BwdWeightSplit& split, float* scratch, cudaStream_t stream);

// ---- tcgen05 tensor-core kernels (FP16 I/O), umma_linear.cu ----------------------------------------
struct UmmaLinearShape {
    int T, Cin, Cout;
    int elem_bytes;     // 2: half or bfloat16 I/O (kind::f16), 4: float I/O (kind::tf32, 3xTF32 split)
    bool bf16;          // elem_bytes == 2: the elements are bfloat16 instead of IEEE half
    int CoT;            // output channels per tile: multiple of 16, T*CoT <= 512 TMEM columns
    int nTiles;         // output-channel tiles
    int nK;             // chunks of the reduction dimension (16 channels for half, 8 for float)
    int rowsB;          // (2T-2)*CoT rows of the weight image per (tile, chunk)
    size_t image_bytes;
    // A shape may describe one SEGMENT of a layer's reduction: input channels [cin0, cin0 + Cin) of CinTotal.
    int cin0, CinTotal;
    // CTA-pair form (tcgen05 cta_group::2): two CTAs on two SMs share every weight tile, half each; the operand image is
    // laid out for it, so a shape is either one or the other.
    bool pair;
    int act;            // 1: GELU on the result before it is stored (forward only)
};
bool umma_linear_supported(int T, eql_dtype_t dtype);
bool umma_linear_pair_supported(int T, eql_dtype_t dtype);
UmmaLinearShape umma_linear_shape(int T, int Cin, int Cout, eql_dtype_t dtype);
// FP32 plans reduce at most kFp32SegmentChannels channels in one TMEM accumulator (the tensor core adds with
// truncation, so the error is linear in the accumulation depth); longer reductions run as several launches whose
// results are added in global memory with round-to-nearest (TMA reduce-add).  Returns the number of segments and
// their length (a multiple of 16); segment k covers channels [k * len, min(Cin, (k + 1) * len)).
constexpr int kFp32SegmentChannels = 256;
int umma_reduction_segments(int Cin, eql_dtype_t dtype, int* seg_len);
UmmaLinearShape umma_linear_segment(int T, int Cin, int Cout, eql_dtype_t dtype, int k, int seg_len);
size_t umma_linear_image_bytes(int T, int Cin, int Cout, eql_dtype_t dtype);       // all segments
// planes[T][Cin][Cout] (float) -> operand image for umma_linear_kernel.
cudaError_t launch_build_umma_image(const UmmaLinearShape& s, const float* planes, void* image, cudaStream_t stream);
// out[N, Cout*T] = IDFT( DFT(in[N, Cin*T]) (x) image ) + bias, fp16 I/O, tcgen05 MMA with FP32 accumulation in TMEM.
cudaError_t launch_umma_linear(const UmmaLinearShape& s, const void* in, void* out, int64_t N, const void* image,
                               const float* bias_f32, int* status, int num_sms, cudaStream_t stream, bool accumulate = false);

// ---- tcgen05 kernel with resident transformed activations (FP16, T = 4 or 8), umma_linear_res.cu -----
struct UmmaResShape {
    int T, Cin, Cout;
    int nTok;           // tokens per tile = 512 / T
    int nK;             // 16-channel chunks of the reduction dimension
    int x_slots;        // x^ chunk buffers in shared memory: nK (token tile resident) or a ring of 3 (one channel tile)
    int nCT;            // tiles of 128 output channels
    int w_slots, n_tw;  // weight-ring slots, transform warps
    bool fits;          // the spectrum of one token tile plus the rings fit in shared memory
    bool paired;        // x^ also keeps -Re of the complex frequencies: two MMAs per complex frequency instead of three
    size_t image_bytes;
    int act;            // 1: GELU on the result before it is stored (forward only)
    bool bf16;          // bfloat16 I/O instead of IEEE half
};
bool umma_res_supported(int T, eql_dtype_t dtype);
UmmaResShape umma_res_shape(int T, int Cin, int Cout, eql_dtype_t dtype = EQL_FP16);
cudaError_t launch_build_umma_res_image(const UmmaResShape& s, const float* planes, void* image, cudaStream_t stream);
struct UmmaBwdWeightShape;
// stash (optional): also write the spectrum of `in` as the operand image of the saved-spectrum weight-gradient kernel
cudaError_t launch_umma_linear_res(const UmmaResShape& s, const void* in, void* out, int64_t N, const void* image,
                                   const float* bias_f32, int* status, int num_sms, cudaStream_t stream,
                                   const UmmaBwdWeightShape* stash_shape = nullptr, void* stash = nullptr);

// ---- tcgen05 weight-gradient kernel (FP16 inputs; FP32 inputs with the 3xTF32 split), umma_bwd_weight.cu --------------------------------
struct UmmaBwdWeightShape {
    int T, Ci, Co;
    int elem_bytes;             // 2: half or bfloat16 inputs (kind::f16), 4: float inputs (kind::tf32, 3xTF32 split)
    bool bf16;                  // elem_bytes == 2: bfloat16 instead of IEEE half
    int CiT, nCiTiles;          // input-channel tile (UMMA M side, <= 128 lanes, CiT*T <= 1024)
    int CoT, nCoTiles;          // output-channel tile (UMMA N side, T*CoT <= 512 TMEM columns)
    int nXs, nYs;               // 64-element raw slabs of x / dy per 16-token chunk
    int splits;                 // token ranges
    int64_t chunks_per_split;   // 16-token chunks per range
    size_t scratch_bytes;       // splits * (T*Co*Ci + Co) floats
    int64_t total_chunks;       // 16-token chunks in all
    size_t stash_bytes;         // FP16: saved spectrum of x as operand image, nCiTiles * total_chunks * T*CiT*32 bytes (else 0)
    // FP32: tokens one launch covers (a multiple of 16, or N itself).  The fields above then describe a launch over
    // min(N, block_tokens) tokens; the caller runs the blocks one after the other and the finalize kernel adds each
    // block's result to dw / db.
    int64_t block_tokens;
    int raw_slots;              // 48 KB raw slots in shared memory (2, or 1 beside a large FP32 stage)
    int y_slab0;                // first slab of dy inside a raw slot: 16 (fixed layout) or nXs (packed layout)
};
bool umma_bwd_weight_supported(int T, eql_dtype_t dtype);
UmmaBwdWeightShape umma_bwd_weight_shape(int T, int Ci, int Co, eql_dtype_t dtype, int64_t N, int num_sms);
// Phase 1 only: partial spectra + db partials into scratch (same layout as the CUDA-core kernel's).
cudaError_t launch_umma_bwd_weight(const UmmaBwdWeightShape& s, const void* x, const void* dy, int64_t N,
                                   float* scratch, int* status, cudaStream_t stream);
// The same from a saved spectrum of x (umma_bwd_weight_saved.cu, FP16): the image written by the forward pass, or by
// launch_xhat_image, replaces x.
cudaError_t launch_xhat_image(const UmmaBwdWeightShape& s, const void* x, int64_t N, void* stash, cudaStream_t stream);
cudaError_t launch_umma_bwd_weight_saved(const UmmaBwdWeightShape& s, const void* stash, const void* dy, int64_t N,
                                         float* scratch, int* status, cudaStream_t stream);
// Phase 2 (direct_kernels.cu): fixed-order sum over splits, 1/T, inverse DFT -> dw, db.
cudaError_t launch_bwd_weight_finalize(int T, bool correlation, const float* scratch, int splits, int Ci, int Co,
                                       float* dw, float* db, cudaStream_t stream, bool accumulate = false);

// ---- dihedral group D_T on the CUDA cores (dihedral_kernels.cu); T = number of rotations, tuples have 2T elements ----
bool dihedral_supported_T(int T);
int64_t dihedral_macs_per_pair(int T);
cudaError_t launch_dihedral_plan_weights(int T, eql_dtype_t dtype, const void* w, const void* bias, int Ci, int Co,
                                         float* planes_fwd, float* planes_bwd, float* bias_f32, cudaStream_t stream);
cudaError_t launch_dihedral_linear(int T, eql_dtype_t dtype, const void* in, void* out, int64_t N, int Cin, int Cout,
                                   const float* planes, const float* bias_f32, cudaStream_t stream, int act);
BwdWeightSplit dihedral_bwd_weight_split(int T, int Ci, int Co, int64_t N);
cudaError_t launch_dihedral_bwd_weight(int T, eql_dtype_t dtype, const void* x, const void* dy, float* dw, float* db,
                                       int64_t N, int Ci, int Co, const BwdWeightSplit& split, float* scratch,
                                       cudaStream_t stream);

// Device address, on `device`, of the scratch array built into the library for eqlinear_bwd_weight_static
// (static_scratch.cu).  `device` must be the current device.  Looked up once per device and cached; the first look-up
// on a device loads the module that holds the array.  Returns nullptr on failure (*err, if given, says why).
void* static_scratch_address(int device, cudaError_t* err);

}  // namespace eql

// Copy pipeline of the host-buffer entry points: token chunks travel host -> device on one stream, are computed on
// the caller's stream and travel back on a third, so that the two copy directions and the kernels overlap.
// Created on first use, destroyed with the plan (streams and events only: no device memory).
constexpr int kHostChunks = 16;
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, out_done = nullptr;
    cudaEvent_t in_done[kHostChunks] = {}, out_ready[kHostChunks] = {};
};

// The host object behind eqlinear_plan_t.
struct eqlinear_plan_s {
    int T, Ci, Co;                  // T: elements per group tuple (cyclic order; 2 x rot for a dihedral plan)
    bool dihedral = false;          // EQL_FLAG_DIHEDRAL
    int rot = 0;                    // dihedral plans: number of rotations (the T the caller passed)
    eql_dtype_t dtype;
    unsigned flags;
    bool has_bias;
    int device;
    char* ws;                       // caller-owned device workspace
    eql::WorkspaceLayout lay;
    int fwd_kernel, bwd_data_kernel, bwd_weight_kernel;
    int num_sms;
    eql::UmmaLinearShape umma_fwd, umma_bwd;
    eql::UmmaResShape res_fwd, res_bwd;   // used when the kernel id is 2
    HostPipe* pipe = nullptr;
};

// Every call that takes a plan launches on the current device with pointers (workspace, tensor maps) that belong to the
// plan's device: refuse, before any launch, when the two differ.
inline eql_status_t eql_check_plan(eqlinear_plan_t plan) {
    if (!plan) return EQL_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return EQL_ERR_CUDA;
    return dev == plan->device ? EQL_OK : EQL_ERR_INVALID_ARG;
}
