// EQ-Linear for the dihedral group D_T (rotations and reflections of a T-gon, order L = 2T) on the CUDA cores.
//
// The paper's Algorithm 1 diagonalises the cyclic group convolution with the DFT; its Conclusion names reflections as
// the next group.  For a non-abelian group the same three steps hold with the group's irreducible representations in
// place of the frequencies:
//     step 1   f^(rho) = sum_g f(g) rho(g)                  (a d x d real matrix per irrep rho of dimension d)
//     step 2   y^(rho)[n, o] = sum_i x^(rho)[n, i] . w^(rho)[o, i]      (d x d matrix products: block GEMMs)
//     step 4   y(g) = 1/|G| sum_rho d_rho tr(rho(g)^T y^(rho))
// D_T has two (T odd) or four (T even) one-dimensional irreps and (T-1)/2 resp. T/2-1 two-dimensional ones
// (rho_k(r^t) = rotation by 2 pi k t / T, rho_k(s) = diag(1, -1)); all are real.  The L = 2T matrix entries are this
// file's "planes"; per (token, input channel, output channel) step 2 costs one product per one-dimensional irrep and
// eight per two-dimensional one, 4T - 4 (T even) against the dense layer's 4 T^2.
// Layer:  y[n, o, g] = b[o] + sum_i sum_h w[o, i, h^-1 g] x[n, i, h],  g = f*T + t <-> r^t s^f.
//
// Kernels (same dataflow as the cyclic CUDA-core kernels): transform at load, plane products in registers, inverse
// transform + bias in the epilogue; the weight gradient as split partial spectra + a fixed-order finalize kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "eql_internal.h"
#include "rdft.cuh"

namespace eql {
namespace {

__device__ __forceinline__ float dto_f32(float v) { return v; }
__device__ __forceinline__ float dto_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ float dto_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename IO> __device__ __forceinline__ IO dfrom_f32(float v);
template <> __device__ __forceinline__ float dfrom_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half dfrom_f32<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 dfrom_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Plane order: 0 = trivial irrep, 1 = sign of the reflection, (T even: 2 = sign of the rotation, 3 = product of both),
// then for k = 1 .. K2 the four entries (0,0), (0,1), (1,0), (1,1) of rho_k.
template <int T> struct Dih {
    static constexpr int L = 2 * T;
    static constexpr int N1 = (T % 2 == 0) ? 4 : 2;          // one-dimensional irreps
    static constexpr int K2 = (T % 2 == 0) ? T / 2 - 1 : (T - 1) / 2;   // two-dimensional irreps
    static_assert(N1 + 4 * K2 == L, "sum of squared dimensions = group order");
    // d_rho / |G| of the irrep plane c belongs to (folded into the spectral weight)
    static __host__ __device__ constexpr float inverse_scale(int c) { return (c < N1 ? 1.0f : 2.0f) / (float)L; }
    // plane of the TRANSPOSED block (data gradient: dX^ = dY^ . W^T)
    static __host__ __device__ constexpr int transposed(int c) {
        return c < N1 ? c : (((c - N1) & 3) == 1 ? c + 1 : ((c - N1) & 3) == 2 ? c - 1 : c);
    }
};

// basis[c][g] = value at g of the matrix entry that plane c stands for; filled once per block.
template <int T>
__device__ __forceinline__ void fill_basis(float (*basis)[2 * T]) {
    using D = Dih<T>;
    constexpr int L = D::L;
    for (int idx = threadIdx.x; idx < L * L; idx += blockDim.x) {
        const int c = idx / L, g = idx % L, f = g / T, t = g % T;
        float v;
        if (c == 0) v = 1.f;
        else if (c == 1) v = f ? -1.f : 1.f;
        else if (c < D::N1) v = ((t & 1) ? -1.f : 1.f) * ((c == 3 && f) ? -1.f : 1.f);
        else {
            const int k = (c - D::N1) / 4 + 1, e = (c - D::N1) & 3;
            float sn, cs;
            sincospif(2.0f * (float)((k * t) % T) / (float)T, &sn, &cs);
            // rho_k(r^t) = [[cs, -sn], [sn, cs]];  rho_k(r^t s) = that times diag(1, -1)
            const float m[4] = {cs, f ? sn : -sn, sn, f ? -cs : cs};
            v = m[e];
        }
        basis[c][g] = v;
    }
    __syncthreads();
}

// v (group samples) -> planes, and planes -> group samples (the transposed table; scales live in the weight)
template <int T>
__device__ __forceinline__ void dih_forward(float* v, const float (*basis)[2 * T]) {
    constexpr int L = 2 * T;
    float out[L];
#pragma unroll
    for (int c = 0; c < L; ++c) {
        float a = 0.f;
#pragma unroll
        for (int g = 0; g < L; ++g) a = fmaf(basis[c][g], v[g], a);
        out[c] = a;
    }
#pragma unroll
    for (int c = 0; c < L; ++c) v[c] = out[c];
}
template <int T>
__device__ __forceinline__ void dih_inverse(float* v, const float (*basis)[2 * T]) {
    constexpr int L = 2 * T;
    float out[L];
#pragma unroll
    for (int g = 0; g < L; ++g) {
        float a = 0.f;
#pragma unroll
        for (int c = 0; c < L; ++c) a = fmaf(basis[c][g], v[c], a);
        out[g] = a;
    }
#pragma unroll
    for (int g = 0; g < L; ++g) v[g] = out[g];
}

// acc[c][i][j] += (a (.) b)[c]:  GRAD = false: Y = A . B per irrep block (forward; data gradient with the transposed
// weight planes);  GRAD = true: dW = B^T . A with a = dY^ (rows i of acc = output channels), b = X^ (columns = input channels).
template <int T, int TM, int TN, bool GRAD>
__device__ __forceinline__ void dih_mac(float (&acc)[2 * T][TM][TN], const float (&a)[2 * T][TM], const float (&b)[2 * T][TN]) {
    using D = Dih<T>;
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) {
#pragma unroll
            for (int c = 0; c < D::N1; ++c) acc[c][i][j] = fmaf(a[c][i], b[c][j], acc[c][i][j]);
#pragma unroll
            for (int k = 0; k < D::K2; ++k) {
                const int q = D::N1 + 4 * k;                     // planes q .. q+3 = entries 00, 01, 10, 11
                if constexpr (!GRAD) {
                    acc[q][i][j]     = fmaf(a[q][i],     b[q][j],     fmaf(a[q + 1][i], b[q + 2][j], acc[q][i][j]));
                    acc[q + 1][i][j] = fmaf(a[q][i],     b[q + 1][j], fmaf(a[q + 1][i], b[q + 3][j], acc[q + 1][i][j]));
                    acc[q + 2][i][j] = fmaf(a[q + 2][i], b[q][j],     fmaf(a[q + 3][i], b[q + 2][j], acc[q + 2][i][j]));
                    acc[q + 3][i][j] = fmaf(a[q + 2][i], b[q + 1][j], fmaf(a[q + 3][i], b[q + 3][j], acc[q + 3][i][j]));
                } else {                                         // dW = X^T . dY with X = b, dY = a
                    acc[q][i][j]     = fmaf(b[q][j],     a[q][i],     fmaf(b[q + 2][j], a[q + 2][i], acc[q][i][j]));
                    acc[q + 1][i][j] = fmaf(b[q][j],     a[q + 1][i], fmaf(b[q + 2][j], a[q + 3][i], acc[q + 1][i][j]));
                    acc[q + 2][i][j] = fmaf(b[q + 1][j], a[q][i],     fmaf(b[q + 3][j], a[q + 2][i], acc[q + 2][i][j]));
                    acc[q + 3][i][j] = fmaf(b[q + 1][j], a[q + 1][i], fmaf(b[q + 3][j], a[q + 3][i], acc[q + 3][i][j]));
                }
            }
        }
}

template <int T> struct DihCfg {                                 // by register budget: L * TM * TN accumulators per thread
    static constexpr int L = 2 * T;
    static constexpr int TM = L <= 8 ? 4 : L <= 12 ? 4 : 2;
    static constexpr int TN = L <= 8 ? 4 : 2;
    static constexpr int BK = L <= 8 ? 8 : 4;
};
constexpr int kDihThreads = 256;
constexpr int kDihPad = 4;

// ================================================================================================
// Spectral weight: one thread per (o, i).  planes_fwd[c][i][o] = d_c/|G| * W^_c[o][i];
// planes_bwd[c][o][i] = the same with every 2 x 2 block transposed (data gradient: dX^ = dY^ . W^T).
template <int T, typename IO>
__global__ void dih_plan_weights_kernel(const IO* __restrict__ w, const IO* __restrict__ bias, int Ci, int Co,
                                        float* __restrict__ pf, float* __restrict__ pb, float* __restrict__ bias_f32) {
    using D = Dih<T>;
    constexpr int L = D::L;
    __shared__ float basis[L][L];
    fill_basis<T>(basis);
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < Co && bias_f32 != nullptr) bias_f32[idx] = dto_f32(bias[idx]);
    if (idx >= Ci * Co) return;
    const int o = idx / Ci, i = idx - o * Ci;
    float v[L];
#pragma unroll
    for (int g = 0; g < L; ++g) v[g] = dto_f32(w[(size_t)idx * L + g]);
    dih_forward<T>(v, basis);
#pragma unroll
    for (int c = 0; c < L; ++c) {
        const float f = v[c] * D::inverse_scale(c);
        pf[((size_t)c * Ci + i) * Co + o] = f;
        pb[((size_t)D::transposed(c) * Co + o) * Ci + i] = f;
    }
}

// ================================================================================================
// Forward / data gradient: out = inverse( forward(in) (.) planes ) + bias.  Block tile BM tokens x BN output channels.
template <int T, typename IO>
__global__ void __launch_bounds__(kDihThreads)
dih_linear_kernel(const IO* __restrict__ in, IO* __restrict__ out, int64_t N, int Cin, int Cout,
                  const float* __restrict__ planes, const float* __restrict__ bias, int act) {
    using C = DihCfg<T>;
    constexpr int L = 2 * T, TM = C::TM, TN = C::TN, BK = C::BK, BM = 16 * TM, BN = 16 * TN;
    __shared__ __align__(16) float xs[L][BK][BM + kDihPad];
    __shared__ __align__(16) float ws[L][BK][BN + kDihPad];
    __shared__ float basis[L][L];
    fill_basis<T>(basis);

    const int tid = threadIdx.x, tm = tid & 15, tn = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;
    float acc[L][TM][TN];
#pragma unroll
    for (int c = 0; c < L; ++c)
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) acc[c][i][j] = 0.f;

    for (int k0 = 0; k0 < Cin; k0 += BK) {
        for (int item = tid; item < BM * BK; item += kDihThreads) {
            const int kk = item % BK, m = item / BK;
            float v[L];
            const int64_t row = m0 + m;
            if (row < N && k0 + kk < Cin) {
                const IO* p = in + row * (int64_t)Cin * L + (int64_t)(k0 + kk) * L;
#pragma unroll
                for (int g = 0; g < L; ++g) v[g] = dto_f32(__ldg(p + g));
                dih_forward<T>(v, basis);
            } else {
#pragma unroll
                for (int c = 0; c < L; ++c) v[c] = 0.f;
            }
#pragma unroll
            for (int c = 0; c < L; ++c) xs[c][kk][m] = v[c];
        }
        for (int idx = tid; idx < L * BK * BN; idx += kDihThreads) {
            const int n = idx % BN, kk = (idx / BN) % BK, c = idx / (BN * BK);
            float f = 0.f;
            if (k0 + kk < Cin && n0 + n < Cout) f = __ldg(planes + ((size_t)c * Cin + k0 + kk) * Cout + n0 + n);
            ws[c][kk][n] = f;
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = 0; kk < BK; ++kk) {
            float a[L][TM], b[L][TN];
#pragma unroll
            for (int c = 0; c < L; ++c) {
#pragma unroll
                for (int i = 0; i < TM; ++i) a[c][i] = xs[c][kk][tm * TM + i];
#pragma unroll
                for (int j = 0; j < TN; ++j) b[c][j] = ws[c][kk][tn * TN + j];
            }
            dih_mac<T, TM, TN, false>(acc, a, b);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t row = m0 + tm * TM + i;
        if (row >= N) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int n = n0 + tn * TN + j;
            if (n >= Cout) continue;
            float v[L];
#pragma unroll
            for (int c = 0; c < L; ++c) v[c] = acc[c][i][j];
            if (bias != nullptr) v[0] += __ldg(bias + n);          // a constant over the group lives in the trivial irrep
            dih_inverse<T>(v, basis);
            IO* q = out + row * (int64_t)Cout * L + (int64_t)n * L;
#pragma unroll
            for (int g = 0; g < L; ++g) {
                float r = v[g];
                if (act) r = 0.5f * r * (1.0f + erff(r * 0.70710678118654752440f));   // GELU
                q[g] = dfrom_f32<IO>(r);
            }
        }
    }
}

// ================================================================================================
// Weight gradient, phase 1: per token range, dW^_c[o][i] += (X^^T . dY^)_c.  Block tile BO x BI channels, all planes.
template <int T, typename IO>
__global__ void __launch_bounds__(kDihThreads)
dih_bwd_weight_kernel(const IO* __restrict__ x, const IO* __restrict__ dy, int64_t N, int Ci, int Co,
                      int64_t tokens_per_split, float* __restrict__ part, float* __restrict__ db_part) {
    using C = DihCfg<T>;
    constexpr int L = 2 * T, TO = C::TM, TI = C::TN, BK = C::BK, BO = 16 * TO, BI = 16 * TI;
    __shared__ __align__(16) float gs[L][BK][BO + kDihPad];
    __shared__ __align__(16) float xs[L][BK][BI + kDihPad];
    __shared__ float basis[L][L];
    fill_basis<T>(basis);
    const int tid = threadIdx.x, to = tid & 15, ti = tid >> 4;
    const int o0 = blockIdx.x * BO, i0 = blockIdx.y * BI, split = blockIdx.z;
    const int64_t nbeg = (int64_t)split * tokens_per_split;
    const int64_t nend = (nbeg + tokens_per_split < N) ? nbeg + tokens_per_split : N;
    float acc[L][TO][TI];
    float dbacc[TO];
#pragma unroll
    for (int c = 0; c < L; ++c)
#pragma unroll
        for (int a = 0; a < TO; ++a)
#pragma unroll
            for (int b = 0; b < TI; ++b) acc[c][a][b] = 0.f;
#pragma unroll
    for (int a = 0; a < TO; ++a) dbacc[a] = 0.f;

    for (int64_t n0 = nbeg; n0 < nend; n0 += BK) {
        for (int item = tid; item < (BO + BI) * BK; item += kDihThreads) {
            const bool is_y = item < BO * BK;
            const int loc = is_y ? item : item - BO * BK;
            const int width = is_y ? BO : BI;
            const int ch = loc % width, kk = loc / width;
            const int chan = (is_y ? o0 : i0) + ch, nchan = is_y ? Co : Ci;
            float v[L];
            if (n0 + kk < nend && chan < nchan) {
                const IO* p = (is_y ? dy : x) + (n0 + kk) * (int64_t)nchan * L + (int64_t)chan * L;
#pragma unroll
                for (int g = 0; g < L; ++g) v[g] = dto_f32(__ldg(p + g));
                dih_forward<T>(v, basis);
            } else {
#pragma unroll
                for (int c = 0; c < L; ++c) v[c] = 0.f;
            }
            if (is_y) {
#pragma unroll
                for (int c = 0; c < L; ++c) gs[c][kk][ch] = v[c];
            } else {
#pragma unroll
                for (int c = 0; c < L; ++c) xs[c][kk][ch] = v[c];
            }
        }
        __syncthreads();
#pragma unroll 2
        for (int kk = 0; kk < BK; ++kk) {
            float a[L][TO], b[L][TI];
#pragma unroll
            for (int c = 0; c < L; ++c) {
#pragma unroll
                for (int q = 0; q < TO; ++q) a[c][q] = gs[c][kk][to * TO + q];
#pragma unroll
                for (int q = 0; q < TI; ++q) b[c][q] = xs[c][kk][ti * TI + q];
            }
            dih_mac<T, TO, TI, true>(acc, a, b);
#pragma unroll
            for (int q = 0; q < TO; ++q) dbacc[q] += a[0][q];     // db = sum over tokens of the trivial-irrep plane of dy
        }
        __syncthreads();
    }
    const size_t plane_stride = (size_t)Co * Ci;
    float* dst = part + (size_t)split * L * plane_stride;
#pragma unroll
    for (int a = 0; a < TO; ++a) {
        const int o = o0 + to * TO + a;
        if (o >= Co) continue;
#pragma unroll
        for (int b = 0; b < TI; ++b) {
            const int i = i0 + ti * TI + b;
            if (i >= Ci) continue;
#pragma unroll
            for (int c = 0; c < L; ++c) dst[c * plane_stride + (size_t)o * Ci + i] = acc[c][a][b];
        }
        if (blockIdx.y == 0 && ti == 0) db_part[(size_t)split * Co + o] = dbacc[a];
    }
}

// Weight gradient, phase 2: fixed-order sum over the splits, d_c/|G|, transposed table -> dw[o][i][:], db[o].
template <int T>
__global__ void __launch_bounds__(256)
dih_finalize_kernel(const float* __restrict__ part, const float* __restrict__ db_part, int splits, int Ci, int Co,
                    float* __restrict__ dw, float* __restrict__ db) {
    using D = Dih<T>;
    constexpr int L = D::L;
    __shared__ float basis[L][L];
    fill_basis<T>(basis);
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < Co && db != nullptr) {
        float s = 0.f;
        for (int sp = 0; sp < splits; ++sp) s += db_part[(size_t)sp * Co + idx];
        db[idx] = s;
    }
    if (idx >= Ci * Co) return;
    const size_t plane_stride = (size_t)Co * Ci;
    float v[L];
#pragma unroll
    for (int c = 0; c < L; ++c) {
        float s = 0.f;
        for (int sp = 0; sp < splits; ++sp) s += __ldg(part + ((size_t)sp * L + c) * plane_stride + idx);
        v[c] = s * D::inverse_scale(c);
    }
    dih_inverse<T>(v, basis);
#pragma unroll
    for (int g = 0; g < L; ++g) dw[(size_t)idx * L + g] = v[g];
}

template <typename F>
cudaError_t dispatch_dih(int T, F&& f) {
    switch (T) {
        case 2: return f(std::integral_constant<int, 2>{});
        case 3: return f(std::integral_constant<int, 3>{});
        case 4: return f(std::integral_constant<int, 4>{});
        case 5: return f(std::integral_constant<int, 5>{});
        case 6: return f(std::integral_constant<int, 6>{});
        case 8: return f(std::integral_constant<int, 8>{});
        default: return cudaErrorInvalidValue;
    }
}
template <typename F>
cudaError_t dispatch_io(eql_dtype_t dtype, F&& f) {
    if (dtype == EQL_FP32) return f(float{});
    if (dtype == EQL_BF16) return f(__nv_bfloat16{});
    return f(__half{});
}

}  // namespace

bool dihedral_supported_T(int T) { return T == 2 || T == 3 || T == 4 || T == 5 || T == 6 || T == 8; }

int64_t dihedral_macs_per_pair(int T) {                             // step-2 products per (token, input, output channel)
    const int n1 = (T % 2 == 0) ? 4 : 2, k2 = (T % 2 == 0) ? T / 2 - 1 : (T - 1) / 2;
    return n1 + 8 * k2;
}

cudaError_t launch_dihedral_plan_weights(int T, eql_dtype_t dtype, const void* w, const void* bias, int Ci, int Co,
                                         float* planes_fwd, float* planes_bwd, float* bias_f32, cudaStream_t stream) {
    const int total = Ci * Co > Co ? Ci * Co : Co;
    const int threads = 128, blocks = (total + threads - 1) / threads;
    return dispatch_dih(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        return dispatch_io(dtype, [&](auto io) {
            using IO = decltype(io);
            dih_plan_weights_kernel<TT, IO><<<blocks, threads, 0, stream>>>((const IO*)w, (const IO*)bias, Ci, Co, planes_fwd,
                                                                            planes_bwd, bias ? bias_f32 : nullptr);
            return cudaGetLastError();
        });
    });
}

cudaError_t launch_dihedral_linear(int T, eql_dtype_t dtype, const void* in, void* out, int64_t N, int Cin, int Cout,
                                   const float* planes, const float* bias_f32, cudaStream_t stream, int act) {
    return dispatch_dih(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        using C = DihCfg<TT>;
        dim3 grid((unsigned)((N + 16 * C::TM - 1) / (16 * C::TM)), (unsigned)((Cout + 16 * C::TN - 1) / (16 * C::TN)));
        return dispatch_io(dtype, [&](auto io) {
            using IO = decltype(io);
            dih_linear_kernel<TT, IO><<<grid, kDihThreads, 0, stream>>>((const IO*)in, (IO*)out, N, Cin, Cout, planes, bias_f32, act);
            return cudaGetLastError();
        });
    });
}

BwdWeightSplit dihedral_bwd_weight_split(int T, int Ci, int Co, int64_t N) {
    const int L = 2 * T, TO = L <= 12 ? 4 : 2, TI = L <= 8 ? 4 : 2, BK = L <= 8 ? 8 : 4;       // DihCfg<T>
    const int64_t tiles = (int64_t)((Co + 16 * TO - 1) / (16 * TO)) * ((Ci + 16 * TI - 1) / (16 * TI));
    int64_t want = (kNumSMs + tiles - 1) / tiles;
    const int64_t chunks = (N + BK - 1) / BK;
    if (want > chunks) want = chunks;
    if (want < 1) want = 1;
    if (want > 65535) want = 65535;
    BwdWeightSplit s;
    s.tokens_per_split = ((chunks + want - 1) / want) * BK;
    s.splits = (int)((N + s.tokens_per_split - 1) / s.tokens_per_split);
    if (s.splits < 1) s.splits = 1;
    s.scratch_bytes = align_up((size_t)s.splits * ((size_t)L * Co * Ci + Co) * sizeof(float), kWsAlign);
    return s;
}

cudaError_t launch_dihedral_bwd_weight(int T, eql_dtype_t dtype, const void* x, const void* dy, float* dw, float* db,
                                       int64_t N, int Ci, int Co, const BwdWeightSplit& split, float* scratch,
                                       cudaStream_t stream) {
    float* part = scratch;
    float* db_part = scratch + (size_t)split.splits * 2 * T * Co * Ci;
    return dispatch_dih(T, [&](auto tc) {
        constexpr int TT = decltype(tc)::value;
        using C = DihCfg<TT>;
        dim3 grid((Co + 16 * C::TM - 1) / (16 * C::TM), (Ci + 16 * C::TN - 1) / (16 * C::TN), split.splits);
        cudaError_t e = dispatch_io(dtype, [&](auto io) {
            using IO = decltype(io);
            dih_bwd_weight_kernel<TT, IO><<<grid, kDihThreads, 0, stream>>>((const IO*)x, (const IO*)dy, N, Ci, Co,
                                                                            split.tokens_per_split, part, db_part);
            return cudaGetLastError();
        });
        if (e != cudaSuccess) return e;
        const int total = Ci * Co > Co ? Ci * Co : Co;
        dih_finalize_kernel<TT><<<(total + 255) / 256, 256, 0, stream>>>(part, db_part, split.splits, Ci, Co, dw, db);
        return cudaGetLastError();
    });
}

}  // namespace eql
