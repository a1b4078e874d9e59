// Device helpers shared by the tcgen05 kernels: half2 packing and the "slab row" transform
// (128 bytes = 64 consecutive fp16 elements of one token, read from a 128B-swizzled TMA slab,
// group DFT of the 64/T channels they hold, planes rounded to fp16 once and packed channel-pairwise).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstring>

#include "rdft.cuh"

namespace eql {

__device__ __forceinline__ float2 unpack_h2(uint32_t u) {
    __half2 h;
    memcpy(&h, &u, 4);
    return __half22float2(h);
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);
    uint32_t u;
    memcpy(&u, &h, 4);
    return u;
}

// The 16-bit I/O flavours of the tensor-core kernels: IEEE half and bfloat16 (same byte geometry, different
// conversions and UMMA operand format code).  The float specialisation only lets shared code compile.
template <typename IO> struct H16;
template <> struct H16<__half> {
    static constexpr uint32_t kUmmaFormat = 0u;
    static constexpr bool kIsHalf = true;
    static __device__ __forceinline__ float2 unpack(uint32_t u) { return unpack_h2(u); }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) { return pack_h2(lo, hi); }
    static __device__ __forceinline__ __half narrow(float v) { return __float2half_rn(v); }
};
template <> struct H16<__nv_bfloat16> {
    static constexpr uint32_t kUmmaFormat = 1u;
    static constexpr bool kIsHalf = false;
    static __device__ __forceinline__ float2 unpack(uint32_t u) {          // bf16 -> f32 is a 16-bit shift
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        uint32_t u;
        memcpy(&u, &h, 4);
        return u;
    }
    static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
};
template <> struct H16<float> {
    static constexpr uint32_t kUmmaFormat = 0u;
    static constexpr bool kIsHalf = false;
    static __device__ __forceinline__ float2 unpack(uint32_t) { return make_float2(0.f, 0.f); }
    static __device__ __forceinline__ uint32_t pack(float, float) { return 0u; }
    static __device__ __forceinline__ float narrow(float v) { return v; }
};

// Exact GELU, x * Phi(x) with the error function (the activation after fc1 in a ViT MLP block), for the forward
// kernels' optional fused epilogue.
__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f)); }

// row_base: start of this token's 128-byte row inside a slab written by TMA with 128B swizzle
// (slab base 1024-byte aligned, rows 128 bytes apart); r: row index inside the slab.
// wd[0..32) = the row's 64 halves in logical order.
__device__ __forceinline__ void load_slab_row(const uint8_t* row_base, int r, uint32_t (&wd)[32]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 c = *reinterpret_cast<const uint4*>(row_base + ((j ^ (r & 7)) << 4));
        wd[4 * j] = c.x; wd[4 * j + 1] = c.y; wd[4 * j + 2] = c.z; wd[4 * j + 3] = c.w;
    }
}

// Group DFT of the 64/T channels held in wd.
// packed[p][cp] = (plane p of channel 2cp, plane p of channel 2cp+1) as half2.
// plane0[c] (optional, float) = k = 0 plane of channel c (the sum over the group axis).
// HALF_MATH = false: butterflies in float, each plane rounded to half once.
// HALF_MATH = true : two channels per instruction in packed half arithmetic (every butterfly output rounded
//                    to half; about twice as cheap, error stays well inside the FP16 parity bar).
template <int T, bool WANT_PLANE0, bool HALF_MATH = false, typename IO = __half>
__device__ __forceinline__ void dft_words(const uint32_t (&wd)[32], uint32_t (&packed)[T][(64 / T) / 2], float* plane0) {
    static_assert(!HALF_MATH || H16<IO>::kIsHalf, "packed-half butterflies exist for IEEE half only");
    constexpr int NCH = 64 / T;
#pragma unroll
    for (int cp = 0; cp < NCH / 2; ++cp) {
        if constexpr (HALF_MATH) {
            __half2 v[T];
#pragma unroll
            for (int t = 0; t < T; t += 2) {
                const uint32_t wa = wd[((2 * cp) * T + t) / 2], wb = wd[((2 * cp + 1) * T + t) / 2];
                const uint32_t lo = __byte_perm(wa, wb, 0x5410);      // (a[t],   b[t])
                const uint32_t hi = __byte_perm(wa, wb, 0x7632);      // (a[t+1], b[t+1])
                memcpy(&v[t], &lo, 4);
                memcpy(&v[t + 1], &hi, 4);
            }
            rdft_forward<T, __half2>(v);
            if constexpr (WANT_PLANE0) {
                const float2 f = __half22float2(v[0]);
                plane0[2 * cp] = f.x; plane0[2 * cp + 1] = f.y;
            }
#pragma unroll
            for (int p = 0; p < T; ++p) memcpy(&packed[p][cp], &v[p], 4);
        } else {
            float v0[T], v1[T];
#pragma unroll
            for (int t = 0; t < T; t += 2) {
                const float2 a = H16<IO>::unpack(wd[((2 * cp) * T + t) / 2]);
                const float2 b = H16<IO>::unpack(wd[((2 * cp + 1) * T + t) / 2]);
                v0[t] = a.x; v0[t + 1] = a.y;
                v1[t] = b.x; v1[t + 1] = b.y;
            }
            rdft_forward<T>(v0);
            rdft_forward<T>(v1);
            if constexpr (WANT_PLANE0) { plane0[2 * cp] = v0[0]; plane0[2 * cp + 1] = v1[0]; }
#pragma unroll
            for (int p = 0; p < T; ++p) packed[p][cp] = H16<IO>::pack(v0[p], v1[p]);
        }
    }
}

// Group DFT of the 32/T float channels held in wd (a 128-byte slab row of an FP32 tensor), in place:
// afterwards wd[c*T + p] is plane p of channel c.
template <int T>
__device__ __forceinline__ void dft_words_f32(uint32_t (&wd)[32]) {
    constexpr int NCH = 32 / T;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        float v[T];
#pragma unroll
        for (int t = 0; t < T; ++t) v[t] = __uint_as_float(wd[c * T + t]);
        rdft_forward<T>(v);
#pragma unroll
        for (int t = 0; t < T; ++t) wd[c * T + t] = __float_as_uint(v[t]);
    }
}

// 3xTF32 split of a float: hi = v rounded to TF32 (10 mantissa bits), lo = (v - hi) rounded to TF32;
// hi*hi + hi*lo + lo*hi reproduces the float product to ~2^-22 (the tensor core itself would truncate, so both
// parts are rounded here).
__device__ __forceinline__ uint32_t round_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ void split_tf32(float v, uint32_t& hi, uint32_t& lo) {
    hi = round_tf32(v);
    lo = round_tf32(v - __uint_as_float(hi));
}

// Stores W 32-bit words of one plane as one contiguous run.
// W = 8 -> two 16-byte stores `second_half_stride` bytes apart, 4 -> one 16-byte store, 2 -> 8 bytes, 1 -> 4 bytes.
template <int NCH>
__device__ __forceinline__ void store_plane_run(uint8_t* d, const uint32_t* pk, int second_half_stride, uint32_t xor_mask = 0u) {
    if constexpr (NCH == 16) {
        *reinterpret_cast<uint4*>(d) = make_uint4(pk[0] ^ xor_mask, pk[1] ^ xor_mask, pk[2] ^ xor_mask, pk[3] ^ xor_mask);
        *reinterpret_cast<uint4*>(d + second_half_stride) =
            make_uint4(pk[4] ^ xor_mask, pk[5] ^ xor_mask, pk[6] ^ xor_mask, pk[7] ^ xor_mask);
    } else if constexpr (NCH == 8) {
        *reinterpret_cast<uint4*>(d) = make_uint4(pk[0] ^ xor_mask, pk[1] ^ xor_mask, pk[2] ^ xor_mask, pk[3] ^ xor_mask);
    } else if constexpr (NCH == 4) {
        *reinterpret_cast<uint2*>(d) = make_uint2(pk[0] ^ xor_mask, pk[1] ^ xor_mask);
    } else {
        *reinterpret_cast<uint32_t*>(d) = pk[0] ^ xor_mask;
    }
}

}  // namespace eql
