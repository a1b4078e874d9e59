// C ABI of libeqlinear: argument validation, the plan object, kernel selection, host-buffer variants.
// Every step of the path itself runs in the kernels of the other translation units.
#include <cuda_fp16.h>

#include <new>

#include "eql_internal.h"

namespace eql {

WorkspaceLayout workspace_layout(int T, int Ci, int Co, eql_dtype_t dtype, bool tensor_cores) {
    WorkspaceLayout l{};
    size_t off = 0;
    l.status = off;      off += kWsAlign;
    l.bias = off;        off += align_up((size_t)Co * sizeof(float), kWsAlign);
    l.planes_fwd = off;  off += align_up((size_t)T * Ci * Co * sizeof(float), kWsAlign);
    l.planes_bwd = off;  off += align_up((size_t)T * Ci * Co * sizeof(float), kWsAlign);
    l.umma_fwd = off;    l.umma_fwd_bytes = 0;
    l.umma_bwd = off;    l.umma_bwd_bytes = 0;
    if (tensor_cores && umma_linear_supported(T, dtype)) {
        l.umma_fwd_bytes = umma_linear_image_bytes(T, Ci, Co, dtype);
        l.umma_bwd_bytes = umma_linear_image_bytes(T, Co, Ci, dtype);
        if (umma_res_supported(T, dtype)) {          // one region serves whichever tensor-core kernel the plan selects
            const size_t rf = umma_res_shape(T, Ci, Co, dtype).image_bytes, rb = umma_res_shape(T, Co, Ci, dtype).image_bytes;
            if (rf > l.umma_fwd_bytes) l.umma_fwd_bytes = rf;
            if (rb > l.umma_bwd_bytes) l.umma_bwd_bytes = rb;
        }
        l.umma_fwd = off;  off += l.umma_fwd_bytes;
        l.umma_bwd = off;  off += l.umma_bwd_bytes;
    }
    l.total = off;
    return l;
}

}  // namespace eql

namespace {

using namespace eql;

inline size_t elem_size(eql_dtype_t d) { return d == EQL_FP32 ? 4 : 2; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// T: the group parameter the caller passed (cyclic order, or rotations of a dihedral plan); *tuple = elements per tuple
eql_status_t check_shape(int T, int Ci, int Co, int dtype, unsigned flags = 0, int* tuple = nullptr) {
    if (dtype != EQL_FP32 && dtype != EQL_FP16 && dtype != EQL_BF16) return EQL_ERR_INVALID_ARG;
    if (T < 1 || Ci < 1 || Co < 1) return EQL_ERR_INVALID_ARG;
    if (flags & EQL_FLAG_DIHEDRAL) {
        if (!dihedral_supported_T(T)) return EQL_ERR_UNSUPPORTED;
        T = 2 * T;
    } else if (!supported_T(T)) {
        return EQL_ERR_UNSUPPORTED;
    }
    if (tuple) *tuple = T;
    if ((int64_t)Ci * T > (1 << 20) || (int64_t)Co * T > (1 << 20)) return EQL_ERR_UNSUPPORTED;
    const size_t e = elem_size((eql_dtype_t)dtype);
    if (((size_t)Ci * T * e) % 16 != 0 || ((size_t)Co * T * e) % 16 != 0) return EQL_ERR_ALIGNMENT;
    return EQL_OK;
}

eql_status_t check_tokens(int64_t N) {
    if (N < 0) return EQL_ERR_INVALID_ARG;
    if (N > ((int64_t)1 << 31) - 1024) return EQL_ERR_UNSUPPORTED;
    return EQL_OK;
}

eql_status_t build_weights(eqlinear_plan_t p, const void* w, const void* bias, cudaStream_t s) {
    if (p->dihedral) {
        cudaError_t de = launch_dihedral_plan_weights(p->rot, p->dtype, w, bias, p->Ci, p->Co,
                                                      (float*)(p->ws + p->lay.planes_fwd), (float*)(p->ws + p->lay.planes_bwd),
                                                      (float*)(p->ws + p->lay.bias), s);
        return de == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    cudaError_t e = launch_plan_weights(p->T, p->dtype, (p->flags & EQL_FLAG_CORRELATION) != 0, w, bias, p->Ci, p->Co,
                                        (float*)(p->ws + p->lay.planes_fwd), (float*)(p->ws + p->lay.planes_bwd),
                                        (float*)(p->ws + p->lay.bias), s);
    if (e != cudaSuccess) return EQL_ERR_CUDA;
    // streaming kernel: one operand image per segment of the reduction (one segment except for wide FP32 layers)
    auto build_segments = [&](int Cin, int Cout, size_t planes_off, size_t image_off, bool pair) -> cudaError_t {
        int len = 0;
        const int nseg = umma_reduction_segments(Cin, p->dtype, &len);
        size_t off = 0;
        for (int k = 0; k < nseg; ++k) {
            UmmaLinearShape sh = umma_linear_segment(p->T, Cin, Cout, p->dtype, k, len);
            sh.pair = pair;
            cudaError_t err = launch_build_umma_image(sh, (const float*)(p->ws + planes_off), p->ws + image_off + off, s);
            if (err != cudaSuccess) return err;
            off += sh.image_bytes;
        }
        return cudaSuccess;
    };
    if (p->fwd_kernel == 1 || p->fwd_kernel == 3) {
        e = build_segments(p->Ci, p->Co, p->lay.planes_fwd, p->lay.umma_fwd, p->fwd_kernel == 3);
        if (e != cudaSuccess) return EQL_ERR_CUDA;
    }
    if (p->bwd_data_kernel == 1 || p->bwd_data_kernel == 3) {
        e = build_segments(p->Co, p->Ci, p->lay.planes_bwd, p->lay.umma_bwd, p->bwd_data_kernel == 3);
        if (e != cudaSuccess) return EQL_ERR_CUDA;
    }
    if (p->fwd_kernel == 2) {
        e = launch_build_umma_res_image(p->res_fwd, (const float*)(p->ws + p->lay.planes_fwd), p->ws + p->lay.umma_fwd, s);
        if (e != cudaSuccess) return EQL_ERR_CUDA;
    }
    if (p->bwd_data_kernel == 2) {
        e = launch_build_umma_res_image(p->res_bwd, (const float*)(p->ws + p->lay.planes_bwd), p->ws + p->lay.umma_bwd, s);
        if (e != cudaSuccess) return EQL_ERR_CUDA;
    }
    return EQL_OK;
}

// Streaming tensor-core kernel over every segment of the reduction: the first launch writes out = bias + its share,
// the others add theirs (one launch in all except for FP32 layers with more than 256 reduced channels).
cudaError_t run_streaming(eqlinear_plan_t p, int Cin, int Cout, const void* in, void* out, int64_t N, size_t image_off,
                          const float* bias, cudaStream_t s, bool pair, int act = 0) {
    int len = 0;
    const int nseg = umma_reduction_segments(Cin, p->dtype, &len);
    size_t off = 0;
    for (int k = 0; k < nseg; ++k) {
        UmmaLinearShape sh = umma_linear_segment(p->T, Cin, Cout, p->dtype, k, len);
        sh.pair = pair;
        sh.act = act;                                            // (plans with an activation have one segment)
        cudaError_t e = launch_umma_linear(sh, in, out, N, p->ws + image_off + off, k == 0 ? bias : nullptr,
                                           (int*)(p->ws + p->lay.status), p->num_sms, s, k > 0);
        if (e != cudaSuccess) return e;
        off += sh.image_bytes;
    }
    return cudaSuccess;
}

void destroy_pipe(HostPipe* hp) {
    if (!hp) return;
    if (hp->in) cudaStreamDestroy(hp->in);
    if (hp->out) cudaStreamDestroy(hp->out);
    if (hp->start) cudaEventDestroy(hp->start);
    if (hp->out_done) cudaEventDestroy(hp->out_done);
    for (int i = 0; i < kHostChunks; ++i) {
        if (hp->in_done[i]) cudaEventDestroy(hp->in_done[i]);
        if (hp->out_ready[i]) cudaEventDestroy(hp->out_ready[i]);
    }
    delete hp;
}

HostPipe* get_pipe(eqlinear_plan_t p) {
    if (p->pipe) return p->pipe;
    HostPipe* hp = new (std::nothrow) HostPipe();
    if (!hp) return nullptr;
    bool ok = cudaStreamCreateWithFlags(&hp->in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp->out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp->start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp->out_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < kHostChunks && ok; ++i)
        ok = cudaEventCreateWithFlags(&hp->in_done[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp->out_ready[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { destroy_pipe(hp); return nullptr; }
    p->pipe = hp;
    return hp;
}

// Tokens per chunk of the copy pipeline: whole 128-token tiles, at most kHostChunks chunks; small batches travel whole.
int64_t host_chunk_tokens(int64_t N) {
    if (N < 8192) return N;
    const int64_t per = (N + kHostChunks - 1) / kHostChunks;
    return (per + 127) / 128 * 128;
}

// fwd (and, with dy/dx, the data gradient) of N tokens from host buffers through the three-stream pipeline.
// On return every copy and kernel has been enqueued; with join, `s` also waits for the last device -> host copy.
eql_status_t pipelined_host(eqlinear_plan_t plan, const void* x_host, const void* dy_host, void* y_host, void* dx_host,
                            int64_t N, void* x_staging, void* dy_staging, void* y_staging, void* dx_staging,
                            cudaStream_t s, bool join) {
    HostPipe* hp = get_pipe(plan);
    if (!hp) return EQL_ERR_CUDA;
    const size_t e = elem_size(plan->dtype);
    const size_t xrow = (size_t)plan->Ci * plan->T * e, yrow = (size_t)plan->Co * plan->T * e;
    const int64_t chunk = host_chunk_tokens(N);
    // the copy streams start after whatever the caller's stream did before (earlier users of the staging buffers)
    if (cudaEventRecord(hp->start, s) != cudaSuccess) return EQL_ERR_CUDA;
    if (cudaStreamWaitEvent(hp->in, hp->start, 0) != cudaSuccess) return EQL_ERR_CUDA;
    if (cudaStreamWaitEvent(hp->out, hp->start, 0) != cudaSuccess) return EQL_ERR_CUDA;
    int c = 0;
    for (int64_t n0 = 0; n0 < N; n0 += chunk, ++c) {
        const int64_t n = N - n0 < chunk ? N - n0 : chunk;
        const char* xh = (const char*)x_host + n0 * xrow;
        char* xs = (char*)x_staging + n0 * xrow;
        char* ys = (char*)y_staging + n0 * yrow;
        if (cudaMemcpyAsync(xs, xh, n * xrow, cudaMemcpyHostToDevice, hp->in) != cudaSuccess) return EQL_ERR_CUDA;
        if (dy_host &&
            cudaMemcpyAsync((char*)dy_staging + n0 * yrow, (const char*)dy_host + n0 * yrow, n * yrow,
                            cudaMemcpyHostToDevice, hp->in) != cudaSuccess) return EQL_ERR_CUDA;
        if (cudaEventRecord(hp->in_done[c], hp->in) != cudaSuccess) return EQL_ERR_CUDA;
        if (cudaStreamWaitEvent(s, hp->in_done[c], 0) != cudaSuccess) return EQL_ERR_CUDA;
        eql_status_t st = eqlinear_fwd(plan, xs, ys, n, s);
        if (st != EQL_OK) return st;
        if (dy_host) {
            st = eqlinear_bwd_data(plan, (char*)dy_staging + n0 * yrow, (char*)dx_staging + n0 * xrow, n, s);
            if (st != EQL_OK) return st;
        }
        if (cudaEventRecord(hp->out_ready[c], s) != cudaSuccess) return EQL_ERR_CUDA;
        if (cudaStreamWaitEvent(hp->out, hp->out_ready[c], 0) != cudaSuccess) return EQL_ERR_CUDA;
        if (cudaMemcpyAsync((char*)y_host + n0 * yrow, ys, n * yrow, cudaMemcpyDeviceToHost, hp->out) != cudaSuccess)
            return EQL_ERR_CUDA;
        if (dy_host &&
            cudaMemcpyAsync((char*)dx_host + n0 * xrow, (char*)dx_staging + n0 * xrow, n * xrow, cudaMemcpyDeviceToHost,
                            hp->out) != cudaSuccess) return EQL_ERR_CUDA;
    }
    if (cudaEventRecord(hp->out_done, hp->out) != cudaSuccess) return EQL_ERR_CUDA;
    if (join && cudaStreamWaitEvent(s, hp->out_done, 0) != cudaSuccess) return EQL_ERR_CUDA;
    return EQL_OK;
}

// Makes `s` wait for the last device -> host copy of the preceding pipelined_host(..., join = false).
eql_status_t join_pipe(eqlinear_plan_t plan, cudaStream_t s) {
    if (!plan->pipe) return EQL_OK;
    return cudaStreamWaitEvent(s, plan->pipe->out_done, 0) == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

}  // namespace

extern "C" {

const char* eqlinear_status_string(eql_status_t status) {
    switch (status) {
        case EQL_OK: return "ok";
        case EQL_ERR_INVALID_ARG: return "invalid argument";
        case EQL_ERR_UNSUPPORTED: return "unsupported shape (group order must be 1..8, 12, 16 or 32)";
        case EQL_ERR_ALIGNMENT: return "pointer or row size not 16-byte aligned";
        case EQL_ERR_WORKSPACE: return "workspace, scratch or staging buffer too small";
        case EQL_ERR_ARCH: return "device is not compute capability 10.x (B200)";
        case EQL_ERR_CUDA: return "CUDA call failed";
        case EQL_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    }
    return "unknown status";
}

eql_status_t eqlinear_count_macs(int T, int C_in, int C_out, int64_t N, int64_t* spectral_macs, int64_t* dense_macs) {
    if (T < 1 || C_in < 1 || C_out < 1 || N < 0) return EQL_ERR_INVALID_ARG;
    const int64_t n_real = (T % 2 == 0) ? 2 : 1;            // k = 0 and, for even T, k = T/2
    const int64_t n_cplx = (T - n_real) / 2;                // 0 < k < T/2
    if (spectral_macs) *spectral_macs = (n_real + 4 * n_cplx) * N * C_in * C_out;
    if (dense_macs) *dense_macs = N * ((int64_t)C_out * T) * ((int64_t)C_in * T);
    return EQL_OK;
}

eql_status_t eqlinear_workspace_bytes(int T, int C_in, int C_out, eql_dtype_t dtype, size_t* bytes) {
    return eqlinear_workspace_bytes_flags(T, C_in, C_out, dtype, 0u, bytes);
}

eql_status_t eqlinear_workspace_bytes_flags(int T, int C_in, int C_out, eql_dtype_t dtype, unsigned flags, size_t* bytes) {
    if (!bytes) return EQL_ERR_INVALID_ARG;
    int tuple = 0;
    eql_status_t st = check_shape(T, C_in, C_out, dtype, flags, &tuple);
    if (st != EQL_OK) return st;
    *bytes = workspace_layout(tuple, C_in, C_out, dtype, !(flags & EQL_FLAG_DIHEDRAL)).total;
    return EQL_OK;
}

eql_status_t eqlinear_plan(eqlinear_plan_t* plan, int T, int C_in, int C_out, eql_dtype_t dtype, const void* w,
                           const void* bias, void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!plan) return EQL_ERR_INVALID_ARG;
    *plan = nullptr;
    int tuple = 0;
    eql_status_t st = check_shape(T, C_in, C_out, dtype, flags, &tuple);
    if (st != EQL_OK) return st;
    if (!w || !workspace) return EQL_ERR_INVALID_ARG;
    const bool dihedral = (flags & EQL_FLAG_DIHEDRAL) != 0;
    // the dihedral group runs on the CUDA-core kernels of its own; flags that pick cyclic kernels or readings do not apply
    if (dihedral && (flags & (EQL_FLAG_CORRELATION | EQL_FLAG_FORCE_STREAMING | EQL_FLAG_CTA_PAIR))) return EQL_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(EQL_FLAG_CORRELATION | EQL_FLAG_FORCE_SIMT | EQL_FLAG_FORCE_STREAMING | EQL_FLAG_CTA_PAIR |
                            EQL_FLAG_NO_CTA_PAIR | EQL_FLAG_GELU | EQL_FLAG_DIHEDRAL))
        return EQL_ERR_INVALID_ARG;
    if ((flags & EQL_FLAG_CTA_PAIR) && (flags & EQL_FLAG_NO_CTA_PAIR)) return EQL_ERR_INVALID_ARG;
    {   // The fused activation is applied to the finished sum: FP32 plans whose forward reduction runs as several
        // segments added in global memory (more than 256 input channels on the tensor cores) cannot take it.
        int len = 0;
        if ((flags & EQL_FLAG_GELU) && !(flags & (EQL_FLAG_FORCE_SIMT | EQL_FLAG_DIHEDRAL)) && umma_linear_supported(T, dtype) &&
            umma_reduction_segments(C_in, dtype, &len) > 1)
            return EQL_ERR_UNSUPPORTED;
    }
    if (!aligned16(w) || (bias && !aligned16(bias))) return EQL_ERR_ALIGNMENT;
    if (reinterpret_cast<uintptr_t>(workspace) % kWsAlign != 0) return EQL_ERR_ALIGNMENT;
    WorkspaceLayout lay = workspace_layout(tuple, C_in, C_out, dtype, !dihedral);
    if (workspace_bytes < lay.total) return EQL_ERR_WORKSPACE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EQL_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return EQL_ERR_CUDA;
    if (major != 10) return EQL_ERR_ARCH;

    eqlinear_plan_s* p = new (std::nothrow) eqlinear_plan_s();
    if (!p) return EQL_ERR_INVALID_ARG;
    p->T = tuple; p->Ci = C_in; p->Co = C_out; p->dtype = dtype; p->flags = flags;
    p->dihedral = dihedral; p->rot = dihedral ? T : 0;
    p->has_bias = bias != nullptr; p->device = dev; p->ws = (char*)workspace; p->lay = lay;
    p->fwd_kernel = p->bwd_data_kernel = p->bwd_weight_kernel = 0;
    p->num_sms = kNumSMs;
    if (cudaDeviceGetAttribute(&p->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { delete p; return EQL_ERR_CUDA; }
    if (!dihedral && umma_linear_supported(T, dtype) && !(flags & EQL_FLAG_FORCE_SIMT)) {
        // 3xTF32 accumulates 1.4e-8 ... 1.6e-8 of relative error per reduced channel (measured: the tensor core adds
        // into its FP32 accumulator with truncation); FP32 plans therefore reduce at most 256 channels (4e-6) per
        // accumulator and run longer reductions as segments that are added in global memory (run_streaming below).
        p->fwd_kernel = 1;
        p->bwd_data_kernel = 1;
        p->umma_fwd = umma_linear_shape(T, C_in, C_out, dtype);
        p->umma_bwd = umma_linear_shape(T, C_out, C_in, dtype);
        if (umma_bwd_weight_supported(T, dtype)) p->bwd_weight_kernel = 1;
        // Layers with few input channels: keep the transformed activations of a token tile resident and reuse them
        // for every output-channel tile (needs a deep weight ring and reasonably full 128-channel tiles).
        if (umma_res_supported(T, dtype) && !(flags & EQL_FLAG_FORCE_STREAMING)) {
            auto prefer = [](const UmmaResShape& r) {
                return r.fits && r.w_slots >= 3 && 2 * r.Cout >= 128 * r.nCT;
            };
            p->res_fwd = umma_res_shape(T, C_in, C_out, dtype);
            p->res_bwd = umma_res_shape(T, C_out, C_in, dtype);
            if (prefer(p->res_fwd)) p->fwd_kernel = 2;
            if (prefer(p->res_bwd)) p->bwd_data_kernel = 2;
        }
        // The streaming kernel's CTA-pair form, in which two SMs share every weight tile: for wide layers (measured on
        // the T = 4 operator shapes: 2-10 % faster from 512 channels per side, 2-4 % slower below), or on request.
        if (umma_linear_pair_supported(T, dtype) && !(flags & EQL_FLAG_NO_CTA_PAIR)) {
            const bool wide = C_in >= 512 && C_out >= 512, force = (flags & EQL_FLAG_CTA_PAIR) != 0;
            if (p->fwd_kernel == 1 && (wide || force)) p->fwd_kernel = 3;
            if (p->bwd_data_kernel == 1 && (wide || force)) p->bwd_data_kernel = 3;
        }
    }

    // The built-in scratch array of eqlinear_bwd_weight_static: look its address up now, with the plan's device current,
    // so that the module holding it is loaded (and its memory reserved) here and never by a call on the hot path.
    // A failure is not an error of this call; eqlinear_bwd_weight_static reports it.
    static_scratch_address(dev, nullptr);

    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(p->ws + lay.status, 0, kWsAlign, s) != cudaSuccess) { delete p; return EQL_ERR_CUDA; }
    st = build_weights(p, w, bias, s);
    if (st != EQL_OK) { delete p; return st; }
    *plan = p;
    return EQL_OK;
}

eql_status_t eqlinear_plan_set_weight(eqlinear_plan_t plan, const void* w, const void* bias, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    if (!w) return EQL_ERR_INVALID_ARG;
    if ((bias != nullptr) != plan->has_bias) return EQL_ERR_INVALID_ARG;
    if (!aligned16(w) || (bias && !aligned16(bias))) return EQL_ERR_ALIGNMENT;
    return build_weights(plan, w, bias, (cudaStream_t)stream);
}

eql_status_t eqlinear_plan_info(eqlinear_plan_t plan, eql_info_t* info) {
    if (!plan || !info) return EQL_ERR_INVALID_ARG;
    const int64_t e = (int64_t)elem_size(plan->dtype);
    info->T = plan->dihedral ? plan->rot : plan->T; info->C_in = plan->Ci; info->C_out = plan->Co; info->dtype = plan->dtype;
    info->flags = plan->flags;
    info->fwd_kernel = plan->fwd_kernel;
    info->bwd_data_kernel = plan->bwd_data_kernel;
    info->bwd_weight_kernel = plan->bwd_weight_kernel;
    eqlinear_count_macs(plan->T, plan->Ci, plan->Co, 1, &info->macs_per_token, &info->dense_macs_per_token);
    if (plan->dihedral)            // one product per one-dimensional irrep, eight per two-dimensional one
        info->macs_per_token = dihedral_macs_per_pair(plan->rot) * plan->Ci * plan->Co;
    info->bytes_per_token_fwd = (int64_t)(plan->Ci + plan->Co) * plan->T * e;
    info->bytes_per_token_bwd_data = info->bytes_per_token_fwd;
    info->bytes_per_token_bwd_weight = info->bytes_per_token_fwd;
    info->workspace_bytes = plan->lay.total;
    return EQL_OK;
}

eql_status_t eqlinear_plan_launch_counts(eqlinear_plan_t plan, int64_t N, int32_t counts[4]) {
    if (!plan || !counts) return EQL_ERR_INVALID_ARG;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    counts[0] = counts[1] = counts[2] = counts[3] = 0;
    if (N == 0) return EQL_OK;
    int len = 0;
    counts[0] = (plan->fwd_kernel == 1 || plan->fwd_kernel == 3) ? umma_reduction_segments(plan->Ci, plan->dtype, &len) : 1;
    counts[1] = (plan->bwd_data_kernel == 1 || plan->bwd_data_kernel == 3) ? umma_reduction_segments(plan->Co, plan->dtype, &len) : 1;
    if (plan->bwd_weight_kernel == 1) {
        const UmmaBwdWeightShape bs = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N, plan->num_sms);
        const int64_t blocks = (N + bs.block_tokens - 1) / bs.block_tokens;
        counts[2] = (int32_t)(2 * blocks);                     // partial-spectra kernel + finalize kernel per block of tokens
    } else {
        counts[2] = 2;
    }
    // eqlinear_fwd_save_spectrum: the resident-activation kernel writes the spectrum itself, others add a pre-pass
    counts[3] = (plan->dtype != EQL_FP32 && plan->bwd_weight_kernel == 1 && plan->fwd_kernel != 2) ? 1 : 0;
    return EQL_OK;
}

eql_status_t eqlinear_plan_device_status(eqlinear_plan_t plan, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    int word = 0;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&word, plan->ws + plan->lay.status, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return EQL_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return EQL_ERR_CUDA;
    return word == 0 ? EQL_OK : EQL_ERR_DEVICE_TIMEOUT;
}

eql_status_t eqlinear_plan_destroy(eqlinear_plan_t plan) {
    if (plan) destroy_pipe(plan->pipe);
    delete plan;
    return EQL_OK;
}

eql_status_t eqlinear_fwd(eqlinear_plan_t plan, const void* x, void* y, int64_t N, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_OK;
    if (!x || !y || x == y) return EQL_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return EQL_ERR_ALIGNMENT;
    const float* bias = plan->has_bias ? (const float*)(plan->ws + plan->lay.bias) : nullptr;
    const int act = (plan->flags & EQL_FLAG_GELU) ? 1 : 0;
    if (plan->fwd_kernel == 2) {
        UmmaResShape rs = plan->res_fwd;
        rs.act = act;
        cudaError_t e = launch_umma_linear_res(rs, x, y, N, plan->ws + plan->lay.umma_fwd, bias,
                                               (int*)(plan->ws + plan->lay.status), plan->num_sms, (cudaStream_t)stream);
        return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    if (plan->fwd_kernel == 1 || plan->fwd_kernel == 3) {
        cudaError_t e = run_streaming(plan, plan->Ci, plan->Co, x, y, N, plan->lay.umma_fwd, bias, (cudaStream_t)stream,
                                      plan->fwd_kernel == 3, act);
        return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    if (plan->dihedral) {
        cudaError_t de = launch_dihedral_linear(plan->rot, plan->dtype, x, y, N, plan->Ci, plan->Co,
                                                (const float*)(plan->ws + plan->lay.planes_fwd), bias, (cudaStream_t)stream, act);
        return de == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    cudaError_t e = launch_direct_linear(plan->T, plan->dtype, x, y, N, plan->Ci, plan->Co,
                                         (const float*)(plan->ws + plan->lay.planes_fwd), bias, (cudaStream_t)stream, act);
    return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

eql_status_t eqlinear_bwd_data(eqlinear_plan_t plan, const void* dy, void* dx, int64_t N, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_OK;
    if (!dy || !dx || dy == dx) return EQL_ERR_INVALID_ARG;
    if (!aligned16(dy) || !aligned16(dx)) return EQL_ERR_ALIGNMENT;
    if (plan->bwd_data_kernel == 2) {
        cudaError_t e = launch_umma_linear_res(plan->res_bwd, dy, dx, N, plan->ws + plan->lay.umma_bwd, nullptr,
                                               (int*)(plan->ws + plan->lay.status), plan->num_sms, (cudaStream_t)stream);
        return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    if (plan->bwd_data_kernel == 1 || plan->bwd_data_kernel == 3) {
        cudaError_t e = run_streaming(plan, plan->Co, plan->Ci, dy, dx, N, plan->lay.umma_bwd, nullptr, (cudaStream_t)stream,
                                      plan->bwd_data_kernel == 3);
        return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    if (plan->dihedral) {
        cudaError_t de = launch_dihedral_linear(plan->rot, plan->dtype, dy, dx, N, plan->Co, plan->Ci,
                                                (const float*)(plan->ws + plan->lay.planes_bwd), nullptr, (cudaStream_t)stream, 0);
        return de == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    cudaError_t e = launch_direct_linear(plan->T, plan->dtype, dy, dx, N, plan->Co, plan->Ci,
                                         (const float*)(plan->ws + plan->lay.planes_bwd), nullptr, (cudaStream_t)stream);
    return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

eql_status_t eqlinear_bwd_weight_scratch_bytes(eqlinear_plan_t plan, int64_t N, size_t* bytes) {
    if (!plan || !bytes) return EQL_ERR_INVALID_ARG;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (plan->bwd_weight_kernel == 1)
        *bytes = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N > 0 ? N : 1, plan->num_sms).scratch_bytes;
    else if (plan->dihedral)
        *bytes = dihedral_bwd_weight_split(plan->rot, plan->Ci, plan->Co, N > 0 ? N : 1).scratch_bytes;
    else
        *bytes = direct_bwd_weight_split(plan->T, plan->Ci, plan->Co, N > 0 ? N : 1).scratch_bytes;
    return EQL_OK;
}

eql_status_t eqlinear_bwd_weight(eqlinear_plan_t plan, const void* x, const void* dy, void* dw, void* db, int64_t N,
                                 void* scratch, size_t scratch_bytes, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (!dw) return EQL_ERR_INVALID_ARG;
    if (!aligned16(dw) || (db && !aligned16(db))) return EQL_ERR_ALIGNMENT;
    cudaStream_t s = (cudaStream_t)stream;
    if (N == 0) {
        if (cudaMemsetAsync(dw, 0, (size_t)plan->Co * plan->Ci * plan->T * sizeof(float), s) != cudaSuccess) return EQL_ERR_CUDA;
        if (db && cudaMemsetAsync(db, 0, (size_t)plan->Co * sizeof(float), s) != cudaSuccess) return EQL_ERR_CUDA;
        return EQL_OK;
    }
    if (!x || !dy || !scratch) return EQL_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(dy)) return EQL_ERR_ALIGNMENT;
    if (reinterpret_cast<uintptr_t>(scratch) % kWsAlign != 0) return EQL_ERR_ALIGNMENT;
    if (plan->bwd_weight_kernel == 1) {
        UmmaBwdWeightShape bs = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N, plan->num_sms);
        if (scratch_bytes < bs.scratch_bytes) return EQL_ERR_WORKSPACE;
        // One launch, except for FP32 plans with long token ranges per accumulator: those run in blocks of tokens,
        // one after the other through the same scratch, and the finalize kernel adds each block's result to dw / db.
        const size_t xrow = (size_t)plan->Ci * plan->T * elem_size(plan->dtype);
        const size_t yrow = (size_t)plan->Co * plan->T * elem_size(plan->dtype);
        const int64_t block = bs.block_tokens;
        for (int64_t n0 = 0; n0 < N; n0 += block) {
            const int64_t nb = N - n0 < block ? N - n0 : block;
            if (nb != block || n0 > 0)
                bs = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, nb, plan->num_sms);
            if (scratch_bytes < bs.scratch_bytes) return EQL_ERR_WORKSPACE;
            cudaError_t e = launch_umma_bwd_weight(bs, (const char*)x + n0 * xrow, (const char*)dy + n0 * yrow, nb,
                                                   (float*)scratch, (int*)(plan->ws + plan->lay.status), s);
            if (e != cudaSuccess) return EQL_ERR_CUDA;
            e = launch_bwd_weight_finalize(plan->T, (plan->flags & EQL_FLAG_CORRELATION) != 0, (const float*)scratch,
                                           bs.splits, plan->Ci, plan->Co, (float*)dw, (float*)db, s, n0 > 0);
            if (e != cudaSuccess) return EQL_ERR_CUDA;
        }
        return EQL_OK;
    }
    if (plan->dihedral) {
        BwdWeightSplit ds = dihedral_bwd_weight_split(plan->rot, plan->Ci, plan->Co, N);
        if (scratch_bytes < ds.scratch_bytes) return EQL_ERR_WORKSPACE;
        cudaError_t de = launch_dihedral_bwd_weight(plan->rot, plan->dtype, x, dy, (float*)dw, (float*)db, N, plan->Ci, plan->Co,
                                                    ds, (float*)scratch, s);
        return de == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    BwdWeightSplit split = direct_bwd_weight_split(plan->T, plan->Ci, plan->Co, N);
    if (scratch_bytes < split.scratch_bytes) return EQL_ERR_WORKSPACE;
    cudaError_t e = launch_direct_bwd_weight(plan->T, plan->dtype, (plan->flags & EQL_FLAG_CORRELATION) != 0, x, dy,
                                             (float*)dw, (float*)db, N, plan->Ci, plan->Co, split, (float*)scratch, s);
    return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

// ---- training with a saved spectrum ---------------------------------------------------------------
eql_status_t eqlinear_spectrum_bytes(eqlinear_plan_t plan, int64_t N, size_t* bytes) {
    if (!plan || !bytes) return EQL_ERR_INVALID_ARG;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (plan->dtype == EQL_FP32 || plan->bwd_weight_kernel != 1) return EQL_ERR_UNSUPPORTED;
    *bytes = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N > 0 ? N : 1, plan->num_sms).stash_bytes;
    return EQL_OK;
}

eql_status_t eqlinear_fwd_save_spectrum(eqlinear_plan_t plan, const void* x, void* y, int64_t N, void* spectrum,
                                        size_t spectrum_bytes, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    size_t need = 0;
    eql_status_t st = eqlinear_spectrum_bytes(plan, N, &need);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_OK;
    if (!spectrum) return EQL_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(spectrum) % kWsAlign != 0) return EQL_ERR_ALIGNMENT;
    if (spectrum_bytes < need) return EQL_ERR_WORKSPACE;
    const UmmaBwdWeightShape bs = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N, plan->num_sms);
    if (plan->fwd_kernel == 2) {
        // the resident-activation kernel writes the spectrum while it transforms x for its own use
        if (!x || !y || x == y) return EQL_ERR_INVALID_ARG;
        if (!aligned16(x) || !aligned16(y)) return EQL_ERR_ALIGNMENT;
        const float* bias = plan->has_bias ? (const float*)(plan->ws + plan->lay.bias) : nullptr;
        UmmaResShape rs = plan->res_fwd;
        rs.act = (plan->flags & EQL_FLAG_GELU) ? 1 : 0;
        cudaError_t e = launch_umma_linear_res(rs, x, y, N, plan->ws + plan->lay.umma_fwd, bias,
                                               (int*)(plan->ws + plan->lay.status), plan->num_sms, (cudaStream_t)stream,
                                               &bs, spectrum);
        return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
    }
    // other forward kernels: a pre-pass kernel transforms x once more
    st = eqlinear_fwd(plan, x, y, N, stream);
    if (st != EQL_OK) return st;
    cudaError_t e = launch_xhat_image(bs, x, N, spectrum, (cudaStream_t)stream);
    return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

eql_status_t eqlinear_bwd_weight_from_spectrum(eqlinear_plan_t plan, const void* spectrum, size_t spectrum_bytes,
                                               const void* dy, void* dw, void* db, int64_t N, void* scratch,
                                               size_t scratch_bytes, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    size_t need = 0;
    eql_status_t st = eqlinear_spectrum_bytes(plan, N, &need);
    if (st != EQL_OK) return st;
    if (!dw) return EQL_ERR_INVALID_ARG;
    if (!aligned16(dw) || (db && !aligned16(db))) return EQL_ERR_ALIGNMENT;
    cudaStream_t s = (cudaStream_t)stream;
    if (N == 0) {
        if (cudaMemsetAsync(dw, 0, (size_t)plan->Co * plan->Ci * plan->T * sizeof(float), s) != cudaSuccess) return EQL_ERR_CUDA;
        if (db && cudaMemsetAsync(db, 0, (size_t)plan->Co * sizeof(float), s) != cudaSuccess) return EQL_ERR_CUDA;
        return EQL_OK;
    }
    if (!spectrum || !dy || !scratch) return EQL_ERR_INVALID_ARG;
    if (!aligned16(dy) || reinterpret_cast<uintptr_t>(spectrum) % kWsAlign != 0 ||
        reinterpret_cast<uintptr_t>(scratch) % kWsAlign != 0) return EQL_ERR_ALIGNMENT;
    if (spectrum_bytes < need) return EQL_ERR_WORKSPACE;
    const UmmaBwdWeightShape bs = umma_bwd_weight_shape(plan->T, plan->Ci, plan->Co, plan->dtype, N, plan->num_sms);
    if (scratch_bytes < bs.scratch_bytes) return EQL_ERR_WORKSPACE;
    cudaError_t e = launch_umma_bwd_weight_saved(bs, spectrum, dy, N, (float*)scratch, (int*)(plan->ws + plan->lay.status), s);
    if (e != cudaSuccess) return EQL_ERR_CUDA;
    e = launch_bwd_weight_finalize(plan->T, (plan->flags & EQL_FLAG_CORRELATION) != 0, (const float*)scratch, bs.splits,
                                   plan->Ci, plan->Co, (float*)dw, (float*)db, s);
    return e == cudaSuccess ? EQL_OK : EQL_ERR_CUDA;
}

// ---- host-buffer variants ---------------------------------------------------------------------
eql_status_t eqlinear_fwd_host(eqlinear_plan_t plan, const void* x_host, void* y_host, int64_t N, void* x_staging,
                               void* y_staging, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_OK;
    if (!x_host || !y_host || !x_staging || !y_staging) return EQL_ERR_INVALID_ARG;
    return pipelined_host(plan, x_host, nullptr, y_host, nullptr, N, x_staging, nullptr, y_staging, nullptr,
                          (cudaStream_t)stream, true);
}

eql_status_t eqlinear_bwd_data_host(eqlinear_plan_t plan, const void* dy_host, void* dx_host, int64_t N,
                                    void* dy_staging, void* dx_staging, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_OK;
    if (!dy_host || !dx_host || !dy_staging || !dx_staging) return EQL_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t e = elem_size(plan->dtype);
    const size_t xb = (size_t)N * plan->Ci * plan->T * e, yb = (size_t)N * plan->Co * plan->T * e;
    if (cudaMemcpyAsync(dy_staging, dy_host, yb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EQL_ERR_CUDA;
    st = eqlinear_bwd_data(plan, dy_staging, dx_staging, N, stream);
    if (st != EQL_OK) return st;
    if (cudaMemcpyAsync(dx_host, dx_staging, xb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return EQL_ERR_CUDA;
    return EQL_OK;
}

eql_status_t eqlinear_bwd_weight_host(eqlinear_plan_t plan, const void* x_host, const void* dy_host, void* dw_host,
                                      void* db_host, int64_t N, void* x_staging, void* dy_staging, void* dw_staging,
                                      void* db_staging, void* scratch, size_t scratch_bytes, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (!dw_host || !dw_staging || (db_host && !db_staging)) return EQL_ERR_INVALID_ARG;
    if (N > 0 && (!x_host || !dy_host || !x_staging || !dy_staging)) return EQL_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t e = elem_size(plan->dtype);
    const size_t xb = (size_t)N * plan->Ci * plan->T * e, yb = (size_t)N * plan->Co * plan->T * e;
    if (N > 0) {
        if (cudaMemcpyAsync(x_staging, x_host, xb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EQL_ERR_CUDA;
        if (cudaMemcpyAsync(dy_staging, dy_host, yb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EQL_ERR_CUDA;
    }
    st = eqlinear_bwd_weight(plan, x_staging, dy_staging, dw_staging, db_host ? db_staging : nullptr, N, scratch,
                             scratch_bytes, stream);
    if (st != EQL_OK) return st;
    if (cudaMemcpyAsync(dw_host, dw_staging, (size_t)plan->Co * plan->Ci * plan->T * sizeof(float),
                        cudaMemcpyDeviceToHost, s) != cudaSuccess) return EQL_ERR_CUDA;
    if (db_host && cudaMemcpyAsync(db_host, db_staging, (size_t)plan->Co * sizeof(float), cudaMemcpyDeviceToHost, s) !=
                       cudaSuccess) return EQL_ERR_CUDA;
    return EQL_OK;
}

eql_status_t eqlinear_step_host(eqlinear_plan_t plan, const void* x_host, const void* dy_host, void* y_host,
                                void* dx_host, void* dw_host, void* db_host, int64_t N, void* x_staging,
                                void* dy_staging, void* y_staging, void* dx_staging, void* dw_staging,
                                void* db_staging, void* scratch, size_t scratch_bytes, void* stream) {
    if (eql_status_t ps = eql_check_plan(plan); ps != EQL_OK) return ps;
    eql_status_t st = check_tokens(N);
    if (st != EQL_OK) return st;
    if (N == 0) return EQL_ERR_INVALID_ARG;
    if (!x_host || !dy_host || !y_host || !dx_host || !dw_host) return EQL_ERR_INVALID_ARG;
    if (!x_staging || !dy_staging || !y_staging || !dx_staging || !dw_staging) return EQL_ERR_INVALID_ARG;
    if ((db_host != nullptr) != (db_staging != nullptr)) return EQL_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // forward and data gradient chunk by chunk while the copies of the neighbouring chunks are in flight; the weight
    // gradient reduces over all tokens and runs once every chunk has arrived
    st = pipelined_host(plan, x_host, dy_host, y_host, dx_host, N, x_staging, dy_staging, y_staging, dx_staging, s, false);
    if (st != EQL_OK) return st;
    if ((st = eqlinear_bwd_weight(plan, x_staging, dy_staging, dw_staging, db_staging, N, scratch, scratch_bytes,
                                  stream)) != EQL_OK) return st;
    if (cudaMemcpyAsync(dw_host, dw_staging, (size_t)plan->Co * plan->Ci * plan->T * sizeof(float),
                        cudaMemcpyDeviceToHost, s) != cudaSuccess) return EQL_ERR_CUDA;
    if (db_host && cudaMemcpyAsync(db_host, db_staging, (size_t)plan->Co * sizeof(float), cudaMemcpyDeviceToHost, s) !=
                       cudaSuccess) return EQL_ERR_CUDA;
    return join_pipe(plan, s);                                   // the y / dx copies of the last chunks may still be in flight
}

}  // extern "C"
