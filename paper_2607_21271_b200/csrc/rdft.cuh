// Real DFT / inverse real DFT of length T along the group axis, held entirely in registers (Algorithm 1, steps 1 and
// 4; Eq. 4 and Eq. 7; the T = 4 case reduces to Eq. 19 and Eq. 21).  Powers of two up to 32 run radix-2 butterflies;
// any other length (Algorithm 1 is stated for every cyclic group) is evaluated directly from a twiddle table
// (rdft_forward_table / rdft_inverse_table below).
//
// Real-packed plane order used everywhere in the library (T values in, T values out):
//   plane 0        : k = 0                    (real)
//   plane 2k-1, 2k : Re, Im of frequency k    for 0 < k < T/2
//   plane T-1      : k = T/2                  (real; even T only -- for odd T plane T-1 is Im of k = (T-1)/2)
//
// Forward:  X_k = sum_s x_s e^{-2 pi i k s / T}                 (unnormalised, Eq. 4)
// Inverse:  y_t = P_0 + (-1)^t P_{T-1} + sum_{0<k<T/2} ( P_{2k-1} cos(2 pi k t/T) - P_{2k} sin(2 pi k t/T) )
//           i.e. the inverse DFT of Eq. 7 / Eq. 15 for planes that were pre-scaled by 1/T (real
//           frequencies) and 2/T (complex frequencies).  The library folds those scales into the
//           spectral weight, so the inverse here is adds, subtracts and twiddle products only.
#pragma once

#include <utility>

#if defined(__CUDACC__)
#include <cuda_fp16.h>
#define EQL_HD __host__ __device__ __forceinline__
#else
#define EQL_HD inline
#endif

namespace eql {

// cos(2*pi*j/32), j = 0..8; sin(2*pi*j/32) = cos(2*pi*(8-j)/32).
template <int J32>
struct Tw32 {
    static_assert(J32 >= 0 && J32 <= 8, "twiddle index");
    static constexpr float value() {
        constexpr float t[9] = {1.0f,
                                0.98078528040323044913f,
                                0.92387953251128675613f,
                                0.83146961230254523708f,
                                0.70710678118654752440f,
                                0.55557023301960222474f,
                                0.38268343236508977173f,
                                0.19509032201612826785f,
                                0.0f};
        return t[J32];
    }
};

// Value types the butterflies run on: float (one channel) or, in device code, __half2 (two channels
// per instruction, every operation rounded to half precision).
template <typename V>
struct Num {
    static EQL_HD V cst(float c) { return V(c); }
};
#if defined(__CUDACC__)
template <>
struct Num<__half2> {
    static __device__ __forceinline__ __half2 cst(float c) { return __float2half2_rn(c); }
};
#endif

template <int N, class F, int... Is>
EQL_HD void static_for_impl(F&& f, std::integer_sequence<int, Is...>) {
    (f(std::integral_constant<int, Is>{}), ...);
}
// Calls f(integral_constant<int, 0>) ... f(integral_constant<int, N-1>) (compile-time indices).
template <int N, class F>
EQL_HD void static_for(F&& f) {
    static_for_impl<N>(static_cast<F&&>(f), std::make_integer_sequence<int, N>{});
}

// Half spectrum of a real sequence x[0], x[S], ..., x[(T-1)S]: re[k], im[k] for k = 0..T/2.
// Radix-2 decimation in time on half spectra: with E, O the half spectra of the even / odd samples,
//   X_k = E_k + w^k O_k,   X_{T/2-k} = conj(E_k - w^k O_k),   w = e^{-2 pi i / T},  k = 0..T/4.
template <int T, int S, typename V>
EQL_HD void rfft_half(const V* x, V* re, V* im) {
    const V zero = Num<V>::cst(0.f);
    if constexpr (T == 1) {
        re[0] = x[0]; im[0] = zero;
    } else if constexpr (T == 2) {
        re[0] = x[0] + x[S]; re[1] = x[0] - x[S];
        im[0] = zero; im[1] = zero;
    } else {
        constexpr int H = T / 2, Q = T / 4;
        V er[Q + 1], ei[Q + 1], orr[Q + 1], oi[Q + 1];
        rfft_half<H, 2 * S, V>(x, er, ei);
        rfft_half<H, 2 * S, V>(x + S, orr, oi);
        re[0] = er[0] + orr[0]; im[0] = zero;
        re[H] = er[0] - orr[0]; im[H] = zero;
        re[Q] = er[Q]; im[Q] = -orr[Q];                 // w^{T/4} = -i, and E_Q, O_Q are real
        static_for<(Q > 1 ? Q - 1 : 0)>([&](auto kk) {
            constexpr int k = decltype(kk)::value + 1;   // 0 < k < T/4
            constexpr int j = k * (32 / T);
            V tr, ti;
            if constexpr (2 * j == 8) {                  // k = T/8: cos = sin
                const V c = Num<V>::cst(Tw32<4>::value());
                tr = c * (orr[k] + oi[k]);
                ti = c * (oi[k] - orr[k]);
            } else {
                const V c = Num<V>::cst(Tw32<j>::value());
                const V s = Num<V>::cst(Tw32<8 - j>::value());
                tr = c * orr[k] + s * oi[k];             // (c - i s)(Or + i Oi)
                ti = c * oi[k] - s * orr[k];
            }
            re[k] = er[k] + tr;     im[k] = ei[k] + ti;
            re[H - k] = er[k] - tr; im[H - k] = ti - ei[k];
        });
    }
}

// Forward real DFT, in place: v[0..T) group samples -> v[0..T) real-packed planes.
template <int T, typename V = float>
EQL_HD void rdft_forward(V* v) {
    if constexpr (T == 1) {
    } else {
        V re[T / 2 + 1], im[T / 2 + 1];
        rfft_half<T, 1, V>(v, re, im);
        v[0] = re[0];
        v[T - 1] = re[T / 2];
        static_for<T / 2 - 1>([&](auto kk) {
            constexpr int k = decltype(kk)::value + 1;
            v[2 * k - 1] = re[k];
            v[2 * k] = im[k];
        });
    }
}

// Inverse on the scaled half spectrum (real frequencies x1, complex frequencies x2, see the header):
// y[0], y[S], ... y[(T-1)S] from re[k], im[k], k = 0..T/2.  Decimation in time run backwards:
//   A_k = X_k + conj(X_{T/2-k}) -> even samples,  B_k = (X_k - conj(X_{T/2-k})) w^{-k} -> odd samples.
template <int T, int S>
EQL_HD void irfft_half(const float* re, const float* im, float* y) {
    if constexpr (T == 1) {
        y[0] = re[0];
    } else if constexpr (T == 2) {
        y[0] = re[0] + re[1];
        y[S] = re[0] - re[1];
    } else {
        constexpr int H = T / 2, Q = T / 4;
        float ar[Q + 1], ai[Q + 1], br[Q + 1], bi[Q + 1];
        ar[0] = re[0] + re[H]; ai[0] = 0.f;
        br[0] = re[0] - re[H]; bi[0] = 0.f;
        ar[Q] = re[Q];  ai[Q] = 0.f;                     // the sub-transforms' k = T/4 planes are real
        br[Q] = -im[Q]; bi[Q] = 0.f;
        static_for<(Q > 1 ? Q - 1 : 0)>([&](auto kk) {
            constexpr int k = decltype(kk)::value + 1;
            constexpr int j = k * (32 / T);
            ar[k] = re[k] + re[H - k];
            ai[k] = im[k] - im[H - k];
            const float dr = re[k] - re[H - k];
            const float di = im[k] + im[H - k];
            if constexpr (2 * j == 8) {
                constexpr float c = Tw32<4>::value();
                br[k] = c * (dr - di);
                bi[k] = c * (di + dr);
            } else {
                constexpr float c = Tw32<j>::value();
                constexpr float s = Tw32<8 - j>::value();
                br[k] = c * dr - s * di;                 // (dr + i di)(c + i s)
                bi[k] = c * di + s * dr;
            }
        });
        irfft_half<H, 2 * S>(ar, ai, y);
        irfft_half<H, 2 * S>(br, bi, y + S);
    }
}

// Inverse real DFT, in place: v[0..T) real-packed pre-scaled planes -> v[0..T) group samples.
template <int T>
EQL_HD void rdft_inverse(float* v) {
    if constexpr (T == 1) {
    } else {
        float re[T / 2 + 1], im[T / 2 + 1];
        re[0] = v[0]; im[0] = 0.f;
        re[T / 2] = v[T - 1]; im[T / 2] = 0.f;
        static_for<T / 2 - 1>([&](auto kk) {
            constexpr int k = decltype(kk)::value + 1;
            re[k] = v[2 * k - 1];
            im[k] = v[2 * k];
        });
        irfft_half<T, 1>(re, im, v);
    }
}

// Scale that turns a true (unnormalised) spectrum plane into the pre-scaled plane rdft_inverse expects.
template <int T>
EQL_HD float plane_inverse_scale(int plane) {
    return (plane == 0 || (T % 2 == 0 && plane == T - 1)) ? (1.0f / T) : (2.0f / T);
}
// Plane p holds the imaginary part of a complex frequency (the planes that change sign under conjugation).
template <int T>
EQL_HD bool plane_is_imag(int plane) {
    return plane > 0 && plane % 2 == 0;          // for even T the last plane (k = T/2, real) has an odd index
}

constexpr bool rdft_has_butterflies(int T) { return T >= 1 && T <= 32 && (T & (T - 1)) == 0; }

// ---- any length: direct evaluation with a table tw[j] = (cos, sin)(2 pi j / T), j = 0..T-1 (shared or global memory).
// The loops are fully unrolled for a compile-time T, so every table index is a constant.
template <int T>
EQL_HD void rdft_forward_table(float* v, const float2* tw) {
    float out[T];
    float s0 = 0.f;
    static_for<T>([&](auto ss) { s0 += v[decltype(ss)::value]; });
    out[0] = s0;
    static_for<(T - 1) / 2>([&](auto kk) {
        constexpr int k = decltype(kk)::value + 1;
        float re = 0.f, im = 0.f;
        static_for<T>([&](auto ss) {
            constexpr int s = decltype(ss)::value, j = (k * s) % T;
            re += v[s] * tw[j].x;
            im -= v[s] * tw[j].y;                        // e^{-2 pi i k s / T}
        });
        out[2 * k - 1] = re;
        out[2 * k] = im;
    });
    if constexpr (T % 2 == 0) {
        float a = 0.f;
        static_for<T>([&](auto ss) { constexpr int s = decltype(ss)::value; a += (s % 2) ? -v[s] : v[s]; });
        out[T - 1] = a;
    }
    static_for<T>([&](auto ss) { v[decltype(ss)::value] = out[decltype(ss)::value]; });
}
// Inverse on pre-scaled planes (see the header of this file).
template <int T>
EQL_HD void rdft_inverse_table(float* v, const float2* tw) {
    float out[T];
    static_for<T>([&](auto tt) {
        constexpr int t = decltype(tt)::value;
        float y = v[0];
        if constexpr (T % 2 == 0) y += (t % 2) ? -v[T - 1] : v[T - 1];
        static_for<(T - 1) / 2>([&](auto kk) {
            constexpr int k = decltype(kk)::value + 1, j = (k * t) % T;
            y += v[2 * k - 1] * tw[j].x - v[2 * k] * tw[j].y;
        });
        out[t] = y;
    });
    static_for<T>([&](auto tt) { v[decltype(tt)::value] = out[decltype(tt)::value]; });
}

}  // namespace eql
