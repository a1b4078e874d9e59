// CUDA-core (FFMA) kernels of the EQ-Linear path: the FP32 production path, and the bring-up /
// fallback path for FP16 I/O (half in, float math, half out).
//
// All three fuse Algorithm 1 into one GEMM-like dataflow: the group DFT (Eq. 4) is applied to each
// group tuple as it is loaded, the per-frequency complex products (Eq. 5) accumulate in registers,
// and the inverse DFT (Eq. 7) plus bias runs in the epilogue; no frequency-domain tensor touches
// global memory except the weight-gradient's split partials.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "eql_internal.h"
#include "rdft.cuh"

namespace eql {
namespace {

// element <-> float for the three I/O types
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename IO> __device__ __forceinline__ IO from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- group-tuple loads and stores (T contiguous elements, T*sizeof(IO) in {4, 8, 16, 32, ...} bytes)
template <int BYTES>
struct VecBytes { using type = uint4; static constexpr int n = BYTES / 16; };
template <> struct VecBytes<8> { using type = uint2; static constexpr int n = 1; };
template <> struct VecBytes<4> { using type = uint32_t; static constexpr int n = 1; };
// group tuples of other sizes (odd or non-power-of-two group orders) are not aligned to a vector: element by element
constexpr bool vector_tuple(int bytes) { return bytes == 4 || bytes == 8 || (bytes >= 16 && bytes % 16 == 0); }

template <int T, typename IO>
__device__ __forceinline__ void load_group(const IO* __restrict__ p, float* v) {
    if constexpr (!vector_tuple(T * sizeof(IO))) {
#pragma unroll
        for (int i = 0; i < T; ++i) {
            v[i] = to_f32(__ldg(p + i));
        }
        return;
    }
    using V = VecBytes<vector_tuple(T * sizeof(IO)) ? T * sizeof(IO) : 16>;
    union { typename V::type vec[V::n]; IO e[T]; } u;
#pragma unroll
    for (int i = 0; i < V::n; ++i) u.vec[i] = __ldg(reinterpret_cast<const typename V::type*>(p) + i);
#pragma unroll
    for (int i = 0; i < T; ++i) v[i] = to_f32(u.e[i]);
}

template <int T, typename IO>
__device__ __forceinline__ void store_group(IO* __restrict__ p, const float* v) {
    if constexpr (!vector_tuple(T * sizeof(IO))) {
#pragma unroll
        for (int i = 0; i < T; ++i) {
            p[i] = from_f32<IO>(v[i]);
        }
        return;
    }
    using V = VecBytes<vector_tuple(T * sizeof(IO)) ? T * sizeof(IO) : 16>;
    union { typename V::type vec[V::n]; IO e[T]; } u;
#pragma unroll
    for (int i = 0; i < T; ++i) u.e[i] = from_f32<IO>(v[i]);
#pragma unroll
    for (int i = 0; i < V::n; ++i) reinterpret_cast<typename V::type*>(p)[i] = u.vec[i];
}

// ---- tile shapes: 256 threads as 16 x 16, each owning TM x TN (row, column) pairs for all T planes
template <int T> struct DirectCfg {        // by register budget: T * TM * TN accumulators per thread
    static constexpr int TM = T <= 4 ? 8 : T <= 8 ? 4 : T <= 16 ? 4 : 2;
    static constexpr int TN = T <= 8 ? 4 : 2;
    static constexpr int BK = T <= 8 ? 8 : 4;
};

// Transforms of one group tuple: butterflies for the power-of-two orders, the twiddle table `tw` (T entries of
// (cos, sin)(2 pi j / T), filled by fill_twiddles at the start of the kernel) for the others.
template <int T>
__device__ __forceinline__ void dft_fwd(float* v, const float2* tw) {
    if constexpr (rdft_has_butterflies(T)) rdft_forward<T>(v); else rdft_forward_table<T>(v, tw);
}
template <int T>
__device__ __forceinline__ void dft_inv(float* v, const float2* tw) {
    if constexpr (rdft_has_butterflies(T)) rdft_inverse<T>(v); else rdft_inverse_table<T>(v, tw);
}
template <int T>
__device__ __forceinline__ void fill_twiddles(float2* tw) {
    if constexpr (!rdft_has_butterflies(T)) {
        if (threadIdx.x < T) {
            float s, c;
            sincospif(2.0f * (float)threadIdx.x / (float)T, &s, &c);
            tw[threadIdx.x] = make_float2(c, s);
        }
        __syncthreads();
    }
}

constexpr int kThreads = 256;
constexpr int kPad = 4;

// acc[p][i][j] += a[p][i] (x) b[p][j] over the real-packed planes: one product for the real
// frequencies, the four-product complex multiply for the others (Eq. 5 written in real arithmetic,
// as in Eq. 20).  CONJ_B multiplies by the conjugate of b instead.
template <int T, int TM, int TN, bool CONJ_B>
__device__ __forceinline__ void plane_mac(float (&acc)[T][TM][TN], const float (&a)[T][TM], const float (&b)[T][TN]) {
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            acc[0][i][j] = fmaf(a[0][i], b[0][j], acc[0][i][j]);
            if constexpr (T % 2 == 0) acc[T - 1][i][j] = fmaf(a[T - 1][i], b[T - 1][j], acc[T - 1][i][j]);   // k = T/2
        }
#pragma unroll
    for (int k = 1; k <= (T - 1) / 2; ++k) {
        const int pr = 2 * k - 1, pi = 2 * k;
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                if constexpr (!CONJ_B) {
                    acc[pr][i][j] = fmaf(a[pr][i], b[pr][j], acc[pr][i][j]);
                    acc[pr][i][j] = fmaf(-a[pi][i], b[pi][j], acc[pr][i][j]);
                    acc[pi][i][j] = fmaf(a[pr][i], b[pi][j], acc[pi][i][j]);
                    acc[pi][i][j] = fmaf(a[pi][i], b[pr][j], acc[pi][i][j]);
                } else {
                    acc[pr][i][j] = fmaf(a[pr][i], b[pr][j], acc[pr][i][j]);
                    acc[pr][i][j] = fmaf(a[pi][i], b[pi][j], acc[pr][i][j]);
                    acc[pi][i][j] = fmaf(a[pi][i], b[pr][j], acc[pi][i][j]);
                    acc[pi][i][j] = fmaf(-a[pr][i], b[pi][j], acc[pi][i][j]);
                }
            }
    }
}

template <int N>
__device__ __forceinline__ void lds_vec(const float* p, float* out) {
    if constexpr (N % 4 == 0) {
#pragma unroll
        for (int i = 0; i < N / 4; ++i) {
            float4 t = reinterpret_cast<const float4*>(p)[i];
            out[4 * i] = t.x; out[4 * i + 1] = t.y; out[4 * i + 2] = t.z; out[4 * i + 3] = t.w;
        }
    } else {
        static_assert(N % 2 == 0, "micro tile");
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            float2 t = reinterpret_cast<const float2*>(p)[i];
            out[2 * i] = t.x; out[2 * i + 1] = t.y;
        }
    }
}

// ================================================================================================
// Spectral weight (Algorithm 1, step 1 for the parameters): one thread per (o, i).
// planes_fwd[p][i][o] = scale_p * W^_p[o][i];  planes_bwd[p][o][i] = scale_p * conj(W^)_p[o][i].
// With the correlation flag the spectrum is conjugated (weight reversed along the group axis).
template <int T, typename IO>
__global__ void plan_weights_kernel(const IO* __restrict__ w, const IO* __restrict__ bias, int Ci, int Co,
                                    bool correlation, float* __restrict__ pf, float* __restrict__ pb,
                                    float* __restrict__ bias_f32) {
    __shared__ float2 tw[T];
    fill_twiddles<T>(tw);
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < Co && bias_f32 != nullptr) {
        bias_f32[idx] = to_f32(bias[idx]);
    }
    if (idx >= Ci * Co) return;
    const int o = idx / Ci, i = idx - o * Ci;
    float v[T];
#pragma unroll
    for (int r = 0; r < T; ++r) {
        v[r] = to_f32(w[(size_t)idx * T + r]);
    }
    dft_fwd<T>(v, tw);
#pragma unroll
    for (int p = 0; p < T; ++p) {
        const bool imag = plane_is_imag<T>(p);
        float f = v[p] * plane_inverse_scale<T>(p);
        if (imag && correlation) f = -f;
        pf[((size_t)p * Ci + i) * Co + o] = f;
        pb[((size_t)p * Co + o) * Ci + i] = imag ? -f : f;
    }
}

// ================================================================================================
// Fused forward / data-gradient kernel: out = IDFT( DFT(in) (x) planes ) + bias.
// Block tile: BM rows (tokens) x BN output channels, all T planes; input channels streamed in chunks.
template <int T, typename IO>
__global__ void __launch_bounds__(kThreads)
direct_linear_kernel(const IO* __restrict__ in, IO* __restrict__ out, int64_t N, int Cin, int Cout,
                     const float* __restrict__ planes, const float* __restrict__ bias, int act) {
    using C = DirectCfg<T>;
    constexpr int TM = C::TM, TN = C::TN, BK = C::BK, BM = 16 * TM, BN = 16 * TN;
    __shared__ __align__(16) float xs[T][BK][BM + kPad];
    __shared__ __align__(16) float ws[T][BK][BN + kPad];
    __shared__ float2 tw[T];
    fill_twiddles<T>(tw);

    const int tid = threadIdx.x, tm = tid & 15, tn = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;

    float acc[T][TM][TN];
#pragma unroll
    for (int p = 0; p < T; ++p)
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) acc[p][i][j] = 0.f;

    for (int k0 = 0; k0 < Cin; k0 += BK) {
        // group tuples of the input chunk -> DFT -> planes in shared memory
        for (int item = tid; item < BM * BK; item += kThreads) {
            const int kk = item % BK, m = item / BK;
            float v[T];
            const int64_t row = m0 + m;
            if (row < N && k0 + kk < Cin) {
                load_group<T, IO>(in + row * (int64_t)Cin * T + (int64_t)(k0 + kk) * T, v);
                dft_fwd<T>(v, tw);
            } else {
#pragma unroll
                for (int p = 0; p < T; ++p) v[p] = 0.f;
            }
#pragma unroll
            for (int p = 0; p < T; ++p) xs[p][kk][m] = v[p];
        }
        for (int idx = tid; idx < T * BK * BN; idx += kThreads) {
            const int n = idx % BN, kk = (idx / BN) % BK, p = idx / (BN * BK);
            float f = 0.f;
            if (k0 + kk < Cin && n0 + n < Cout) f = __ldg(planes + ((size_t)p * Cin + k0 + kk) * Cout + n0 + n);
            ws[p][kk][n] = f;
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = 0; kk < BK; ++kk) {
            float a[T][TM], b[T][TN];
#pragma unroll
            for (int p = 0; p < T; ++p) {
                lds_vec<TM>(&xs[p][kk][tm * TM], a[p]);
                lds_vec<TN>(&ws[p][kk][tn * TN], b[p]);
            }
            plane_mac<T, TM, TN, false>(acc, a, b);
        }
        __syncthreads();
    }

    // epilogue: inverse DFT over the planes, bias, one contiguous group tuple per (row, channel)
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t row = m0 + tm * TM + i;
        if (row >= N) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int n = n0 + tn * TN + j;
            if (n >= Cout) continue;
            float v[T];
#pragma unroll
            for (int p = 0; p < T; ++p) v[p] = acc[p][i][j];
            if (bias != nullptr) v[0] += __ldg(bias + n);     // a constant over t lives in plane k = 0
            dft_inv<T>(v, tw);
            if (act) {
#pragma unroll
                for (int q = 0; q < T; ++q) v[q] = 0.5f * v[q] * (1.0f + erff(v[q] * 0.70710678118654752440f));   // GELU
            }
            store_group<T, IO>(out + row * (int64_t)Cout * T + (int64_t)n * T, v);
        }
    }
}

// ================================================================================================
// Weight gradient, phase 1: per token range, dW^_p[o][i] += dY^_p[n][o] * conj(X^_p[n][i]).
// Block tile: BO output channels x BI input channels, all planes; tokens streamed in chunks of BK.
template <int T, typename IO>
__global__ void __launch_bounds__(kThreads)
direct_bwd_weight_kernel(const IO* __restrict__ x, const IO* __restrict__ dy, int64_t N, int Ci, int Co,
                         int64_t tokens_per_split, float* __restrict__ part, float* __restrict__ db_part) {
    using C = DirectCfg<T>;
    constexpr int TO = C::TM, TI = C::TN, BK = C::BK, BO = 16 * TO, BI = 16 * TI;
    __shared__ __align__(16) float gs[T][BK][BO + kPad];
    __shared__ __align__(16) float xs[T][BK][BI + kPad];
    __shared__ float2 tw[T];
    fill_twiddles<T>(tw);

    const int tid = threadIdx.x, to = tid & 15, ti = tid >> 4;
    const int o0 = blockIdx.x * BO, i0 = blockIdx.y * BI, split = blockIdx.z;
    const int64_t nbeg = (int64_t)split * tokens_per_split;
    const int64_t nend = (nbeg + tokens_per_split < N) ? nbeg + tokens_per_split : N;

    float acc[T][TO][TI];
    float dbacc[TO];
#pragma unroll
    for (int p = 0; p < T; ++p)
#pragma unroll
        for (int a = 0; a < TO; ++a)
#pragma unroll
            for (int b = 0; b < TI; ++b) acc[p][a][b] = 0.f;
#pragma unroll
    for (int a = 0; a < TO; ++a) dbacc[a] = 0.f;

    for (int64_t n0 = nbeg; n0 < nend; n0 += BK) {
        for (int item = tid; item < BO * BK; item += kThreads) {
            const int o = item % BO, kk = item / BO;
            float v[T];
            if (n0 + kk < nend && o0 + o < Co) {
                load_group<T, IO>(dy + (n0 + kk) * (int64_t)Co * T + (int64_t)(o0 + o) * T, v);
                dft_fwd<T>(v, tw);
            } else {
#pragma unroll
                for (int p = 0; p < T; ++p) v[p] = 0.f;
            }
#pragma unroll
            for (int p = 0; p < T; ++p) gs[p][kk][o] = v[p];
        }
        for (int item = tid; item < BI * BK; item += kThreads) {
            const int i = item % BI, kk = item / BI;
            float v[T];
            if (n0 + kk < nend && i0 + i < Ci) {
                load_group<T, IO>(x + (n0 + kk) * (int64_t)Ci * T + (int64_t)(i0 + i) * T, v);
                dft_fwd<T>(v, tw);
            } else {
#pragma unroll
                for (int p = 0; p < T; ++p) v[p] = 0.f;
            }
#pragma unroll
            for (int p = 0; p < T; ++p) xs[p][kk][i] = v[p];
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = 0; kk < BK; ++kk) {
            float a[T][TO], b[T][TI];
#pragma unroll
            for (int p = 0; p < T; ++p) {
                lds_vec<TO>(&gs[p][kk][to * TO], a[p]);
                lds_vec<TI>(&xs[p][kk][ti * TI], b[p]);
            }
            plane_mac<T, TO, TI, true>(acc, a, b);
#pragma unroll
            for (int q = 0; q < TO; ++q) dbacc[q] += a[0][q];     // db = sum_n Re dY^_0
        }
        __syncthreads();
    }

    const size_t plane_stride = (size_t)Co * Ci;
    float* dst = part + (size_t)split * T * plane_stride;
#pragma unroll
    for (int a = 0; a < TO; ++a) {
        const int o = o0 + to * TO + a;
        if (o >= Co) continue;
#pragma unroll
        for (int b = 0; b < TI; ++b) {
            const int i = i0 + ti * TI + b;
            if (i >= Ci) continue;
#pragma unroll
            for (int p = 0; p < T; ++p) dst[p * plane_stride + (size_t)o * Ci + i] = acc[p][a][b];
        }
        if (blockIdx.y == 0 && ti == 0) db_part[(size_t)split * Co + o] = dbacc[a];
    }
}

// Weight gradient, phase 2: fixed-order sum over the splits, inverse DFT with its 1/T, dw[o][i][:].
// Block = 32 (o, i) pairs x T planes: thread (pair, plane) sums its plane over the splits (coalesced over the
// pairs), the planes meet in shared memory, and the first 32 threads run the inverse transform.
template <int T>
__global__ void __launch_bounds__(32 * T)
bwd_weight_finalize_kernel(const float* __restrict__ part, const float* __restrict__ db_part, int splits, int Ci,
                           int Co, bool correlation, float* __restrict__ dw, float* __restrict__ db, bool accumulate) {
    __shared__ float planes[T][33];
    __shared__ float2 tw[T];
    fill_twiddles<T>(tw);
    asm volatile("griddepcontrol.wait;" ::: "memory");         // launched to overlap the tail of the kernel that writes `part`
    const int pair = threadIdx.x & 31, p = threadIdx.x >> 5;
    const int idx = blockIdx.x * 32 + pair;
    const size_t plane_stride = (size_t)Co * Ci;
    // db: the first blocks also reduce the bias partials (one thread per output channel)
    {
        const int o = blockIdx.x * blockDim.x + threadIdx.x;
        if (o < Co && db != nullptr) {
            float s = 0.f;
            for (int sp = 0; sp < splits; ++sp) s += db_part[(size_t)sp * Co + o];
            db[o] = accumulate ? db[o] + s : s;                  // later token blocks add to the earlier ones
        }
    }
    float acc = 0.f;
    if (idx < Ci * Co) {
        // four running sums (split index mod 4), combined in a fixed order: the result does not depend on timing, and
        // eight loads are in flight per thread instead of one dependent chain
        const float* src = part + (size_t)p * plane_stride + idx;
        const size_t step = (size_t)T * plane_stride;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        int sp = 0;
#pragma unroll 2
        for (; sp + 4 <= splits; sp += 4) {
            a0 += __ldg(src + (size_t)sp * step);
            a1 += __ldg(src + (size_t)(sp + 1) * step);
            a2 += __ldg(src + (size_t)(sp + 2) * step);
            a3 += __ldg(src + (size_t)(sp + 3) * step);
        }
        for (; sp < splits; ++sp) a0 += __ldg(src + (size_t)sp * step);
        acc = (a0 + a1) + (a2 + a3);
    }
    const bool imag = plane_is_imag<T>(p);
    acc *= plane_inverse_scale<T>(p);
    if (imag && correlation) acc = -acc;
    planes[p][pair] = acc;
    __syncthreads();
    if (p == 0 && idx < Ci * Co) {
        float v[T];
#pragma unroll
        for (int q = 0; q < T; ++q) v[q] = planes[q][pair];
        dft_inv<T>(v, tw);
#pragma unroll
        for (int r = 0; r < T; ++r) dw[(size_t)idx * T + r] = accumulate ? dw[(size_t)idx * T + r] + v[r] : v[r];
    }
}

// Enough blocks of 32*T threads to cover the (o, i) pairs (32 per block) and, with one thread each, the Co bias sums.
inline int finalize_blocks(int T, int Ci, int Co) {
    const int by_pairs = (Ci * Co + 31) / 32, by_bias = (Co + 32 * T - 1) / (32 * T);
    return by_pairs > by_bias ? by_pairs : by_bias;
}

template <typename F>
cudaError_t dispatch_T(int T, F&& f) {
    switch (T) {                                  // the orders supported_T() lists
        case 1: return f(std::integral_constant<int, 1>{});
        case 2: return f(std::integral_constant<int, 2>{});
        case 3: return f(std::integral_constant<int, 3>{});
        case 4: return f(std::integral_constant<int, 4>{});
        case 5: return f(std::integral_constant<int, 5>{});
        case 6: return f(std::integral_constant<int, 6>{});
        case 7: return f(std::integral_constant<int, 7>{});
        case 8: return f(std::integral_constant<int, 8>{});
        case 12: return f(std::integral_constant<int, 12>{});
        case 16: return f(std::integral_constant<int, 16>{});
        case 32: return f(std::integral_constant<int, 32>{});
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_plan_weights(int T, eql_dtype_t dtype, bool correlation, const void* w, const void* bias,
                                int Ci, int Co, float* planes_fwd, float* planes_bwd, float* bias_f32,
                                cudaStream_t stream) {
    const int total = Ci * Co > Co ? Ci * Co : Co;
    const int threads = 128, blocks = (total + threads - 1) / threads;
    return dispatch_T(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        float* bdst = bias ? bias_f32 : nullptr;
        if (dtype == EQL_FP32)
            plan_weights_kernel<TT, float><<<blocks, threads, 0, stream>>>(
                (const float*)w, (const float*)bias, Ci, Co, correlation, planes_fwd, planes_bwd, bdst);
        else if (dtype == EQL_BF16)
            plan_weights_kernel<TT, __nv_bfloat16><<<blocks, threads, 0, stream>>>(
                (const __nv_bfloat16*)w, (const __nv_bfloat16*)bias, Ci, Co, correlation, planes_fwd, planes_bwd, bdst);
        else
            plan_weights_kernel<TT, __half><<<blocks, threads, 0, stream>>>(
                (const __half*)w, (const __half*)bias, Ci, Co, correlation, planes_fwd, planes_bwd, bdst);
        return cudaGetLastError();
    });
}

cudaError_t launch_direct_linear(int T, eql_dtype_t dtype, const void* in, void* out, int64_t N,
                                 int Cin, int Cout, const float* planes, const float* bias_f32,
                                 cudaStream_t stream, int act) {
    return dispatch_T(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        using C = DirectCfg<TT>;
        constexpr int BM = 16 * C::TM, BN = 16 * C::TN;
        dim3 grid((unsigned)((N + BM - 1) / BM), (unsigned)((Cout + BN - 1) / BN));
        if (dtype == EQL_FP32)
            direct_linear_kernel<TT, float><<<grid, kThreads, 0, stream>>>(
                (const float*)in, (float*)out, N, Cin, Cout, planes, bias_f32, act);
        else if (dtype == EQL_BF16)
            direct_linear_kernel<TT, __nv_bfloat16><<<grid, kThreads, 0, stream>>>(
                (const __nv_bfloat16*)in, (__nv_bfloat16*)out, N, Cin, Cout, planes, bias_f32, act);
        else
            direct_linear_kernel<TT, __half><<<grid, kThreads, 0, stream>>>(
                (const __half*)in, (__half*)out, N, Cin, Cout, planes, bias_f32, act);
        return cudaGetLastError();
    });
}

BwdWeightSplit direct_bwd_weight_split(int T, int Ci, int Co, int64_t N) {
    const int TO = T <= 4 ? 8 : T <= 16 ? 4 : 2, TI = T <= 8 ? 4 : 2, BK = T <= 8 ? 8 : 4;       // DirectCfg<T>
    const int64_t tiles = (int64_t)((Co + 16 * TO - 1) / (16 * TO)) * ((Ci + 16 * TI - 1) / (16 * TI));
    int64_t want = (kNumSMs + tiles - 1) / tiles;                // about one block per SM: fewer partial spectra to write and re-read
    const int64_t chunks = (N + BK - 1) / BK;
    if (want > chunks) want = chunks;
    if (want < 1) want = 1;
    if (want > 65535) want = 65535;
    BwdWeightSplit s;
    s.tokens_per_split = ((chunks + want - 1) / want) * BK;
    s.splits = (int)((N + s.tokens_per_split - 1) / s.tokens_per_split);
    if (s.splits < 1) s.splits = 1;
    s.scratch_bytes = align_up((size_t)s.splits * ((size_t)T * Co * Ci + Co) * sizeof(float), kWsAlign);
    return s;
}

cudaError_t launch_bwd_weight_finalize(int T, bool correlation, const float* scratch, int splits, int Ci, int Co,
                                       float* dw, float* db, cudaStream_t stream, bool accumulate) {
    const float* part = scratch;
    const float* db_part = scratch + (size_t)splits * T * Co * Ci;
    return dispatch_T(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        return launch_overlapped(bwd_weight_finalize_kernel<TT>, dim3(finalize_blocks(TT, Ci, Co)), dim3(32 * TT), 0, stream,
                                 part, db_part, splits, Ci, Co, correlation, dw, db, accumulate);
    });
}

cudaError_t launch_direct_bwd_weight(int T, eql_dtype_t dtype, bool correlation, const void* x, const void* dy,
                                     float* dw, float* db, int64_t N, int Ci, int Co,
                                     const BwdWeightSplit& split, float* scratch, cudaStream_t stream) {
    float* part = scratch;
    float* db_part = scratch + (size_t)split.splits * T * Co * Ci;
    return dispatch_T(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        using C = DirectCfg<TT>;
        constexpr int BO = 16 * C::TM, BI = 16 * C::TN;
        dim3 grid((Co + BO - 1) / BO, (Ci + BI - 1) / BI, split.splits);
        if (dtype == EQL_FP32)
            direct_bwd_weight_kernel<TT, float><<<grid, kThreads, 0, stream>>>(
                (const float*)x, (const float*)dy, N, Ci, Co, split.tokens_per_split, part, db_part);
        else if (dtype == EQL_BF16)
            direct_bwd_weight_kernel<TT, __nv_bfloat16><<<grid, kThreads, 0, stream>>>(
                (const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, N, Ci, Co, split.tokens_per_split, part, db_part);
        else
            direct_bwd_weight_kernel<TT, __half><<<grid, kThreads, 0, stream>>>(
                (const __half*)x, (const __half*)dy, N, Ci, Co, split.tokens_per_split, part, db_part);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        return launch_overlapped(bwd_weight_finalize_kernel<TT>, dim3(finalize_blocks(TT, Ci, Co)), dim3(32 * TT), 0, stream,
                                 (const float*)part, (const float*)db_part, split.splits, Ci, Co, correlation, dw, db, false);
    });
}

}  // namespace eql
