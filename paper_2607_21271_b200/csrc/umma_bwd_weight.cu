// Weight gradient on the tcgen05 tensor cores (FP32 accumulation in TMEM; FP16 inputs with kind::f16, FP32 inputs
// with kind::tf32 and the 3xTF32 hi/lo split: hi*hi + hi*lo + lo*hi):
//   dW^_k[o, i] = sum_n dY^_k[n, o] * conj(X^_k[n, i])     for every retained frequency k,
// a GEMM whose reduction dimension is the token index.  One CTA owns an (input-channel tile,
// output-channel tile) block of all T real-packed planes for one token range; the per-range partial
// spectra go to scratch [split][T][Co][Ci] and the finalize kernel sums them in a fixed order and
// applies the inverse group DFT (with its 1/T).
//
//   TMA (2-D, 128B swizzle)   16-token slabs of x and dy              -> shared raw slots
//   12 transform warps        group DFT (Eq. 4) in registers, fp16    -> shared MN-major operand tiles
//                             (x^ planes; dy^ planes, with -Re dy^ stored once more per complex k)
//   1 thread                  tcgen05.mma: A = x^ plane (M = input channels), B = dy^ planes
//                             real k:     D_k          += X_k^T G_k
//                             complex k: [Re | Im] dW^ += Xr^T [Gr | Gi] + Xi^T [Gi | -Gr]
//   12 warps (after the loop) tcgen05.ld -> partial spectra in scratch;  db partials from plane k = 0
//
// All mbarrier waits are bounded (see ptx_sm100.cuh); on a time-out the CTA drains and returns.
#include <cuda_fp16.h>

#include <mutex>

#include "eql_internal.h"
#include "ptx_sm100.cuh"
#include "rdft.cuh"
#include "umma_common.cuh"

namespace eql {
namespace {

constexpr int kChunkTok = 16;                 // tokens per pipeline stage = one UMMA K step
constexpr int kSlab = kChunkTok * 128;        // bytes of one raw slab [16 tokens x 128 B]
constexpr int kMaxXSlabs = 16, kMaxYSlabs = 8;
constexpr int kRawSlot = (kMaxXSlabs + kMaxYSlabs) * kSlab;      // 48 KB
constexpr int kThreadsBw = 512;
constexpr int kTmemColsBw = 512;
constexpr int kRawSlots = 2, kStages = 2;
constexpr int kWarpTma = 0, kWarpMmaBw = 1, kWarpDftX0 = 4, kWarpDftY0 = 12;
constexpr int kNumDft = 12;

struct BwParams {
    float* part;                 // [splits][T][Co][Ci]
    float* db_part;              // [splits][Co]
    int* status;
    int64_t N;
    int Ci, Co, CiT, CoT, nCiTiles, nCoTiles, nXs, nYs;
    int splits;
    int64_t chunks_per_split;    // 16-token chunks per token range
    int xhat_bytes, stage_bytes;
    int x_part_bytes, y_part_bytes;   // FP32: bytes of the TF32 "hi" copy of x^ / dy^ inside a stage; the "lo" copy follows it
    int stages;                  // operand stages (2; 1 where the hi/lo copies of FP32 leave no room for two)
    int raw_slots;               // raw slots of 48 KB (2; 1 where a large FP32 stage leaves room for one only)
    int y_slab0;                 // first slab of dy inside a raw slot (kMaxXSlabs, or nXs in the packed layout)
    int x3d, y3d;                // tensor maps are 3-D (64 elements, rows, slab index): one load per chunk and tensor
    int part_tma;                // the partial spectra can be written with TMA tensor stores (row pitch a multiple of 16 bytes)
};


struct BwBarriers {
    uint64_t full_raw[kRawSlots], empty_raw[kRawSlots];
    uint64_t full_ab[kStages], empty_ab[kStages];
    uint64_t full_d, mma_done;
    uint32_t tmem_base;
    int abort_flag;
};

template <int T, typename IO>
__global__ void __launch_bounds__(kThreadsBw, 1)
umma_bwd_weight_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                       const __grid_constant__ CUtensorMap tmap_part, const BwParams prm) {
    constexpr int E = sizeof(IO);                 // 2: half inputs, 4: float inputs (3xTF32)
    constexpr int EPR = 128 / E;                  // elements per 128-byte raw row
    constexpr int NCH = EPR / T;                  // channels per raw row
    // Operand tiles of a 16-token chunk.  FP16: MN-major (channels contiguous, as they come out of the transform),
    // 32 bytes per channel.  FP32: the tensor core transposes 32-bit operands only in a swizzle mode of its own, so
    // the TF32 tiles are written K-major (tokens contiguous): core matrix = 8 channels x 4 tokens (128 B), the four
    // core matrices of a channel group kF32Lbo = 144 bytes apart (16 bytes of padding keep the scattered 4-byte
    // stores of a half warp on distinct banks), channel groups kF32Sbo = 576 bytes apart: 72 bytes per channel.
    constexpr int kF32Lbo = 144, kF32Sbo = 4 * kF32Lbo;
    constexpr int TOKB = E == 2 ? kChunkTok * E : kF32Sbo / 8;   // bytes per channel of one tile
    extern __shared__ uint8_t smem_raw_base[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~(uintptr_t)1023);
    BwBarriers* bar = reinterpret_cast<BwBarriers*>(smem);
    uint8_t* raw = smem + 1024;                                  // kRawSlots x 48 KB
    uint8_t* stages = raw + prm.raw_slots * kRawSlot;            // prm.stages x stage_bytes (+ 8 KB slack after the last)
    const int NST = prm.stages, NRAW = prm.raw_slots;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &bar->abort_flag;
    int* status = prm.status;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kRawSlots; ++i) { ptx::mbar_init(&bar->full_raw[i], 1); ptx::mbar_init(&bar->empty_raw[i], kNumDft); }
        for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&bar->full_ab[i], kNumDft); ptx::mbar_init(&bar->empty_ab[i], 1); }
        ptx::mbar_init(&bar->full_d, 1);
        ptx::mbar_init(&bar->mma_done, 1);
        bar->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_x);
        ptx::prefetch_tensormap(&tmap_dy);
    }
    if (warp == kWarpMmaBw) {
        ptx::tmem_alloc(&bar->tmem_base, kTmemColsBw);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bar->tmem_base;
    // This kernel may have been scheduled while the kernel before it in the stream is still finishing: everything above
    // (barriers, tensor memory) overlapped that; nothing below may run before its results are visible.  The kernel
    // behind this one gets the same head start.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    // unit -> (token range, input-channel tile, output-channel tile); output tile fastest so that the
    // CTAs sharing the same x rows run at the same time
    const int co_tile = blockIdx.x % prm.nCoTiles;
    const int ci_tile = (blockIdx.x / prm.nCoTiles) % prm.nCiTiles;
    const int split = blockIdx.x / (prm.nCoTiles * prm.nCiTiles);
    const int64_t total_chunks = (prm.N + kChunkTok - 1) / kChunkTok;
    const int64_t chunk0 = (int64_t)split * prm.chunks_per_split;
    int64_t nchunks = total_chunks - chunk0;
    if (nchunks > prm.chunks_per_split) nchunks = prm.chunks_per_split;
    if (nchunks < 0) nchunks = 0;
    const int CiT = prm.CiT, CoT = prm.CoT;

    if (warp == kWarpTma) {
        if (lane == 0) {
            bool ok = true;
            int64_t c = 0;
            const uint32_t bytes = (uint32_t)(prm.nXs + prm.nYs) * kSlab;
            for (; c < nchunks; ++c) {
                const int slot = NRAW == 2 ? (int)(c & 1) : 0;
                ok = ptx::mbar_wait(&bar->empty_raw[slot], (uint32_t)((NRAW == 2 ? (c >> 1) : c) & 1) ^ 1, abort_flag, status, 201);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx(&bar->full_raw[slot], bytes);
                const int row = (int)((chunk0 + c) * kChunkTok);
                uint8_t* dst = raw + slot * kRawSlot;
                // One 3-D box [slab][16 rows][64 elements] per tensor where the row length is a whole number of
                // slabs; otherwise one 2-D box per slab (the same shared-memory layout either way).
                if (prm.x3d) {
                    ptx::tma_load_3d(dst, &tmap_x, 0, row, ci_tile * CiT * T / EPR, &bar->full_raw[slot]);
                } else {
                    for (int s = 0; s < prm.nXs; ++s)
                        ptx::tma_load_2d(dst + s * kSlab, &tmap_x, ci_tile * CiT * T + s * EPR, row, &bar->full_raw[slot]);
                }
                if (prm.y3d) {
                    ptx::tma_load_3d(dst + prm.y_slab0 * kSlab, &tmap_dy, 0, row, co_tile * CoT * T / EPR, &bar->full_raw[slot]);
                } else {
                    for (int s = 0; s < prm.nYs; ++s)
                        ptx::tma_load_2d(dst + (prm.y_slab0 + s) * kSlab, &tmap_dy, co_tile * CoT * T + s * EPR, row,
                                         &bar->full_raw[slot]);
                }
            }
            if (!ok) {
                const int64_t lo = c > NRAW ? c - NRAW : 0;
                for (int64_t d = lo; d < c; ++d)
                    ptx::mbar_wait(&bar->full_raw[NRAW == 2 ? (d & 1) : 0], (uint32_t)((NRAW == 2 ? (d >> 1) : d) & 1), abort_flag, status, 211, false);
            }
        }
    } else if (warp == kWarpMmaBw) {
        if (lane == 0) {
            bool ok = true;
            constexpr uint32_t kMnMajor = (1u << 15) | (1u << 16);       // both operands MN-major
            constexpr uint32_t kFmt = H16<IO>::kUmmaFormat;                // half or bfloat16 operands
            const uint32_t idesc_real = E == 2 ? (ptx::umma_idesc_f16_f32(128, CoT, kFmt) | kMnMajor) : ptx::umma_idesc_tf32_f32(128, CoT);
            const uint32_t idesc_cplx = E == 2 ? (ptx::umma_idesc_f16_f32(128, 2 * CoT, kFmt) | kMnMajor) : ptx::umma_idesc_tf32_f32(128, 2 * CoT);
            const uint32_t a_plane = (uint32_t)CiT * TOKB, b_tile = (uint32_t)CoT * TOKB;
            // FP16, MN-major no-swizzle tiles: lbo = stride between 8-token groups (128 B), sbo = stride between 8-channel groups
            // (256 B).  FP32, K-major no-swizzle tiles: lbo = stride between 4-token core matrices, sbo = between 8-channel groups.
            auto mma = [](uint32_t d, uint32_t a_addr, uint32_t b_addr, uint32_t idesc, uint32_t accumulate) {
                if constexpr (E == 2)
                    ptx::umma_f16(d, ptx::umma_smem_desc(a_addr, 128, 256), ptx::umma_smem_desc(b_addr, 128, 256), idesc, accumulate);
                else
                    ptx::umma_tf32(d, ptx::umma_smem_desc(a_addr, kF32Lbo, kF32Sbo), ptx::umma_smem_desc(b_addr, kF32Lbo, kF32Sbo), idesc, accumulate);
            };
            constexpr int KSTEPS = E == 2 ? 1 : 2;                       // a 16-token chunk is one K step of halves, two of TF32
            constexpr int PASSES = E == 2 ? 1 : 3;                       // 3xTF32: hi*hi, hi*lo, lo*hi
            for (int64_t c = 0; c < nchunks; ++c) {
                // NST is 1 or 2: stage and phase parity without a division
                const int st = NST == 2 ? (int)(c & 1) : 0;
                const uint32_t sph = (uint32_t)((NST == 2 ? (c >> 1) : c) & 1);
                ok = ptx::mbar_wait(&bar->full_ab[st], sph, abort_flag, status, 202);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t stage0 = ptx::smem_u32(stages + st * prm.stage_bytes);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
#pragma unroll
                    for (int pass = 0; pass < PASSES; ++pass) {
                        const uint32_t a0 = stage0 + (pass == 2 ? prm.x_part_bytes : 0) + ks * 2 * kF32Lbo;   // 8 tokens = 2 core matrices
                        const uint32_t b0 = stage0 + prm.xhat_bytes + (pass == 1 ? prm.y_part_bytes : 0) + ks * 2 * kF32Lbo;
                        const uint32_t acc = (c > 0 || ks > 0 || pass > 0) ? 1u : 0u;
                        mma(tmem_base, a0, b0, idesc_real, acc);
#pragma unroll
                        for (int f = 1; f < T / 2; ++f) {
                            const uint32_t d = tmem_base + (uint32_t)((2 * f - 1) * CoT);
                            const uint32_t bt = b0 + (uint32_t)(1 + 3 * (f - 1)) * b_tile;      // tiles Gr | Gi | -Gr
                            mma(d, a0 + (2 * f - 1) * a_plane, bt, idesc_cplx, acc);             // Xr^T [Gr | Gi]
                            mma(d, a0 + (2 * f) * a_plane, bt + b_tile, idesc_cplx, 1u);         // Xi^T [Gi | -Gr]
                        }
                        mma(tmem_base + (uint32_t)((T - 1) * CoT), a0 + (T - 1) * a_plane,
                            b0 + (uint32_t)(1 + 3 * (T / 2 - 1)) * b_tile, idesc_real, acc);
                    }
                }
                ptx::umma_commit(&bar->empty_ab[st]);
            }
            if (ok) ptx::umma_commit(&bar->full_d);
            ptx::umma_commit(&bar->mma_done);
            ptx::mbar_wait(&bar->mma_done, 0, abort_flag, status, 213, false);
        }
    } else if (warp >= kWarpDftX0) {
        // ------------------------------------------------------------ transform warps
        // A half warp takes one slab of a chunk.  Fixed layout: warps 4-11 the (up to 16) slabs of x, warps 12-15 the (up
        // to 8) slabs of dy.  Packed layout (y_slab0 = nXs, an even number): the slabs of dy follow those of x directly, so
        // a layer with few input channels can give more half warps - and a wider output tile - to dy.
        const bool packed_slabs = prm.y_slab0 != kMaxXSlabs;
        const int hw0 = 2 * (warp - kWarpDftX0);                 // first half warp of this warp
        const bool is_y = packed_slabs ? hw0 >= prm.nXs : warp >= kWarpDftY0;
        const int wi = packed_slabs ? (is_y ? (hw0 - prm.nXs) >> 1 : hw0 >> 1) : (is_y ? warp - kWarpDftY0 : warp - kWarpDftX0);
        const int half = lane >> 4, row = lane & 15;
        const int slab = 2 * wi + half;
        const bool active = slab < (is_y ? prm.nYs : prm.nXs);
        float dbacc[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) dbacc[i] = 0.f;
        bool ok = true;
        for (int64_t c = 0; c < nchunks; ++c) {
            const int slot = NRAW == 2 ? (int)(c & 1) : 0, st = NST == 2 ? (int)(c & 1) : 0;
            const uint32_t sph = (uint32_t)((NST == 2 ? (c >> 1) : c) & 1);
            ok = ptx::mbar_wait(&bar->full_raw[slot], (uint32_t)((NRAW == 2 ? (c >> 1) : c) & 1), abort_flag, status, 203);
            ok = ok && ptx::mbar_wait(&bar->empty_ab[st], sph ^ 1, abort_flag, status, 204);
            if (!ok) break;
            uint32_t wd[32];
            if (active)
                load_slab_row(raw + slot * kRawSlot + ((is_y ? prm.y_slab0 : 0) + slab) * kSlab + row * 128, row, wd);
            // The rows are in registers: order these generic-proxy reads before the async-proxy (TMA) refill of
            // the slot, then release it so that the refill overlaps the transform.
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->empty_raw[slot]);
            if (active) {
                const int mn0 = slab * NCH;                      // first channel of this slab inside the tile
                // FP16, MN-major tile: (channel mn, token k) at (mn/8)*256 + (k/8)*128 + (k%8)*16 + (mn%8)*2
                // FP32, K-major tile:  (channel mn, token k) at (mn/8)*576 + (k/4)*144 + (mn%8)*16 + (k%4)*4
                const int off = E == 2 ? (mn0 >> 3) * 256 + (row >> 3) * 128 + (row & 7) * 16 + (mn0 & 7) * 2
                                       : (row >> 2) * kF32Lbo + (row & 3) * 4;
                uint8_t* stage = stages + st * prm.stage_bytes;
                const int a_plane = CiT * TOKB, tb = CoT * TOKB;
                if constexpr (E == 2) {
                    uint32_t packed[T][NCH / 2];
                    float p0[NCH];
                    // dy: butterflies in float, planes rounded to fp16 once (its k = 0 plane also feeds db, unrounded).
                    // x: packed-half butterflies, two channels per instruction.  x^ is recomputed by every
                    // output-channel tile, which makes its transform the largest share of this kernel's instructions
                    // (-10 % kernel time); the weight gradient averages the extra rounding over the token sum
                    // (measured max error 4.2e-4 instead of 3.1e-4 of the largest |dw|, bar 3e-3).
                    // (bfloat16 inputs: float butterflies for both -- a packed bfloat16 butterfly keeps 8 bits per rounding)
                    if (is_y) dft_words<T, true, false, IO>(wd, packed, p0);
                    else if constexpr (H16<IO>::kIsHalf) dft_words<T, false, true>(wd, packed, nullptr);
                    else dft_words<T, false, false, IO>(wd, packed, nullptr);
                    if (!is_y) {
#pragma unroll
                        for (int p = 0; p < T; ++p) store_plane_run<NCH>(stage + p * a_plane + off, packed[p], 256);
                    } else {
#pragma unroll
                        for (int i = 0; i < NCH; ++i) dbacc[i] += p0[i];
                        uint8_t* yb = stage + prm.xhat_bytes + off;
                        store_plane_run<NCH>(yb, packed[0], 256);
#pragma unroll
                        for (int f = 1; f < T / 2; ++f) {
                            uint8_t* t0 = yb + (1 + 3 * (f - 1)) * tb;
                            store_plane_run<NCH>(t0, packed[2 * f - 1], 256);                    // Gr
                            store_plane_run<NCH>(t0 + tb, packed[2 * f], 256);                   // Gi
                            store_plane_run<NCH>(t0 + 2 * tb, packed[2 * f - 1], 256, 0x80008000u);   // -Gr
                        }
                        store_plane_run<NCH>(yb + (1 + 3 * (T / 2 - 1)) * tb, packed[T - 1], 256);
                    }
                } else {
                    // FP32: group DFT in place (wd[c*T + p] = plane p of channel c), then every plane goes out twice:
                    // rounded to TF32 ("hi") and the TF32-rounded remainder ("lo"), one stage part after the other
                    dft_words_f32<T>(wd);
                    auto put = [&](uint8_t* dst, int part_bytes, int p, uint32_t sign) {
#pragma unroll
                        for (int c2 = 0; c2 < NCH; ++c2) {
                            uint32_t hi, lo;
                            split_tf32(__uint_as_float(wd[c2 * T + p] ^ sign), hi, lo);
                            const int mn = mn0 + c2;
                            uint8_t* e = dst + (mn >> 3) * kF32Sbo + (mn & 7) * 16;
                            *reinterpret_cast<uint32_t*>(e) = hi;
                            *reinterpret_cast<uint32_t*>(e + part_bytes) = lo;
                        }
                    };
                    if (!is_y) {
#pragma unroll
                        for (int p = 0; p < T; ++p) put(stage + p * a_plane + off, prm.x_part_bytes, p, 0u);
                    } else {
#pragma unroll
                        for (int i = 0; i < NCH; ++i) dbacc[i] += __uint_as_float(wd[i * T]);
                        uint8_t* yb = stage + prm.xhat_bytes + off;
                        put(yb, prm.y_part_bytes, 0, 0u);
#pragma unroll
                        for (int f = 1; f < T / 2; ++f) {
                            uint8_t* t0 = yb + (1 + 3 * (f - 1)) * tb;
                            put(t0, prm.y_part_bytes, 2 * f - 1, 0u);                            // Gr
                            put(t0 + tb, prm.y_part_bytes, 2 * f, 0u);                           // Gi
                            put(t0 + 2 * tb, prm.y_part_bytes, 2 * f - 1, 0x80000000u);          // -Gr
                        }
                        put(yb + (1 + 3 * (T / 2 - 1)) * tb, prm.y_part_bytes, T - 1, 0u);
                    }
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->full_ab[st]);
        }
        // db partial of this token range: sum over the 16 token rows of each half warp
        if (is_y) {
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                float v = dbacc[i];
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                const int co = co_tile * CoT + slab * NCH + i;
                if (ok && active && row == 0 && ci_tile == 0 && slab * NCH + i < CoT && co < prm.Co)
                    prm.db_part[(size_t)split * prm.Co + co] = v;
            }
        }
        // ------------------------------------------------------------ epilogue: TMEM -> partial spectra
        // all 12 warps: a warp reads the TMEM lane quadrant (warp & 3) and every third group of 16 columns
        if (ok) {
            const int quad = warp & 3;
            const int third = (warp - kWarpDftX0) >> 2;
            const int ci_local = quad * 32 + lane;
            const int ci = ci_tile * CiT + ci_local;
            const bool lane_ok = ci_local < CiT && ci < prm.Ci;
            if (nchunks > 0) ok = ptx::mbar_wait(&bar->full_d, 0, abort_flag, status, 205);
            if (ok) {
                ptx::tc_fence_after_sync();
                const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
                const size_t plane_stride = (size_t)prm.Co * prm.Ci;
                float* dst = prm.part + (size_t)split * T * plane_stride;
                // A quad whose 32 rows all belong to this input-channel tile goes out through shared memory and TMA
                // tensor stores ([16 output channels x 32 input channels] floats per store, two staging buffers per
                // warp in the idle raw slots; channels beyond C_in / C_out are clipped by the hardware).  Other quads
                // write their valid lanes directly.
                const bool via_tma = prm.part_tma != 0 && quad * 32 + 32 <= CiT;
                float* stg = reinterpret_cast<float*>(raw + (warp - kWarpDftX0) * 4096);
                int it = 0;
                for (int col = third * 16; col < T * CoT; col += 48, ++it) {
                    uint32_t v[16];
                    if (nchunks > 0) {
                        ptx::tmem_ld<16>(lane_base + (uint32_t)col, v);
                        ptx::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = 0u;
                    }
                    const int p = col / CoT, o0 = co_tile * CoT + col % CoT;
                    if (via_tma) {
                        float* buf = stg + (it & 1) * 512;
                        if (lane == 0) ptx::bulk_wait_group_read1();     // the store issued two iterations ago has read this buffer
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 16; ++j) buf[j * 32 + lane] = __uint_as_float(v[j]);
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0 && o0 < prm.Co) {
                            ptx::tma_store_3d(&tmap_part, ci_tile * CiT + quad * 32, o0, split * T + p, buf);
                            ptx::bulk_commit_group();
                        }
                    } else if (lane_ok) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (o0 + j < prm.Co) dst[p * plane_stride + (size_t)(o0 + j) * prm.Ci + ci] = __uint_as_float(v[j]);
                    }
                }
                if (via_tma && lane == 0) ptx::bulk_wait_group_read0();
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kWarpMmaBw) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemColsBw);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

bool encode_rows16(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows, int elem_bytes) {
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)cols * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)kChunkTok};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
               const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view of a [rows, cols] tensor whose row length is a multiple of 128 bytes:
// dim0 = 128 contiguous bytes of elements, dim1 = rows (stride = row pitch), dim2 = slab index (stride = 128 bytes).
// A box [128 B, 16, nslabs] lands in shared memory as nslabs consecutive [16 x 128 B] slabs.
bool encode_slabs3d(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows, int nslabs,
                    int elem_bytes) {
    const cuuint32_t epr = (cuuint32_t)(128 / elem_bytes);
    const cuuint64_t gdim[3] = {epr, (cuuint64_t)rows, (cuuint64_t)(cols / epr)};
    const cuuint64_t gstr[2] = {(cuuint64_t)cols * elem_bytes, 128};
    const cuuint32_t box[3] = {epr, (cuuint32_t)kChunkTok, (cuuint32_t)nslabs};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
               const_cast<void*>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shared memory outside the operand stages: barriers, alignment, two raw slots, and 8 KB of slack after the last stage
// (the UMMA reads 128 rows of every plane although only CiT are valid).
constexpr size_t bw_fixed_smem(int raw_slots) { return 1024 + 1024 + (size_t)raw_slots * kRawSlot + 8192; }
constexpr size_t kBwFixedSmem = bw_fixed_smem(kRawSlots);

// Bytes per channel of one operand tile of a 16-token chunk: FP16 MN-major 32; FP32 K-major with padded cores 72.
int bw_chan_bytes(int elem_bytes) { return elem_bytes == 2 ? kChunkTok * 2 : 72; }

size_t bw_stage_bytes(int T, int CiT, int CoT, int elem_bytes) {
    const int copies = elem_bytes == 4 ? 2 : 1;
    const int ytiles = 2 + 3 * (T / 2 - 1);
    const size_t x_part = (size_t)T * ((CiT + 7) / 8 * 8) * bw_chan_bytes(elem_bytes);
    const size_t y_part = (size_t)ytiles * CoT * bw_chan_bytes(elem_bytes);
    return align_up(copies * (x_part + y_part), 1024);
}

int balanced_tile(int C, int max_tile, int round) {
    const int n = (C + max_tile - 1) / max_tile;
    const int per = (C + n - 1) / n;
    return (per + round - 1) / round * round;
}

}  // namespace


bool umma_bwd_weight_supported(int T, eql_dtype_t dtype) {
    if (dtype == EQL_FP16 || dtype == EQL_BF16) return T == 4 || T == 8 || T == 16 || T == 32;
    return T == 4 || T == 8;            // FP32 (3xTF32): larger T leaves too few channels per tile
}

constexpr int64_t kMaxChunksPerSplitFp32 = 12, kMaxChunksPerSplitFp16 = 2048;
constexpr size_t kBlockScratchBudget = 30u << 20;          // FP32 token blocks: partial sums of one launch (below the 32 MiB built-in scratch)

UmmaBwdWeightShape umma_bwd_weight_shape(int T, int Ci, int Co, eql_dtype_t dtype, int64_t N, int num_sms) {
    UmmaBwdWeightShape s{};
    s.T = T; s.Ci = Ci; s.Co = Co;
    s.elem_bytes = dtype == EQL_FP32 ? 4 : 2;
    s.bf16 = dtype == EQL_BF16;
    const int epr = 128 / s.elem_bytes;                          // elements per raw slab row
    int max_cit = kMaxXSlabs * epr / T;                          // at most 16 raw slabs of x per chunk
    if (max_cit > 128) max_cit = 128;                            // UMMA M = 128 TMEM lanes
    int max_cot = kMaxYSlabs * epr / T;                          // at most 8 raw slabs of dy per chunk
    if (max_cot > kTmemColsBw / T) max_cot = kTmemColsBw / T;    // T planes x CoT fp32 TMEM columns
    s.CoT = balanced_tile(Co, max_cot, 16);
    s.nCoTiles = (Co + s.CoT - 1) / s.CoT;
    s.CiT = balanced_tile(Ci, max_cit, T == 4 ? 16 : 8);
    // FP32 keeps two copies (hi, lo) of every operand tile: shrink the input-channel tile until one stage fits
    while (kBwFixedSmem + bw_stage_bytes(T, s.CiT, s.CoT, s.elem_bytes) > 227 * 1024 && max_cit > 16) {
        max_cit -= 8;
        s.CiT = balanced_tile(Ci, max_cit, T == 4 ? 16 : 8);
    }
    s.nCiTiles = (Ci + s.CiT - 1) / s.CiT;
    s.nXs = (s.CiT * T + epr - 1) / epr;
    s.raw_slots = kRawSlots;
    s.y_slab0 = kMaxXSlabs;
    // FP32 layers with few input channels: the half warps that x leaves idle can transform dy (packed slab layout), which
    // allows a wider output-channel tile - fewer tiles means fewer CTAs repeating the transform of x and half as many
    // chunks per CTA at the same MMA count per chunk.  The larger stage may leave room for one raw slot only.
    if (dtype == EQL_FP32 && s.nXs % 2 == 0 && s.nXs < kMaxXSlabs + kMaxYSlabs) {
        int max_cot2 = (kMaxXSlabs + kMaxYSlabs - s.nXs) * epr / T;
        if (max_cot2 > kTmemColsBw / T) max_cot2 = kTmemColsBw / T;
        max_cot2 = max_cot2 / 16 * 16;
        if (max_cot2 >= 16) {
            const int cot2 = balanced_tile(Co, max_cot2, 16);
            const int n2 = (Co + cot2 - 1) / cot2;
            if (cot2 <= max_cot2 && n2 < s.nCoTiles) {
                for (int rs = kRawSlots; rs >= 1; --rs) {
                    if (bw_fixed_smem(rs) + bw_stage_bytes(T, s.CiT, cot2, s.elem_bytes) <= 227 * 1024) {
                        s.CoT = cot2; s.nCoTiles = n2; s.raw_slots = rs; s.y_slab0 = s.nXs;
                        break;
                    }
                }
            }
        }
    }
    s.nYs = (s.CoT * T + epr - 1) / epr;
    const int64_t tiles = (int64_t)s.nCiTiles * s.nCoTiles;
    const int64_t chunks = N > 0 ? (N + kChunkTok - 1) / kChunkTok : 1;
    int64_t want = num_sms / tiles;
    if (want < 1) want = 1;
    s.block_tokens = N > 0 ? N : 1;
    // The tensor core adds into its FP32 accumulator with truncation, so the error of a partial sum grows linearly
    // with the number of accumulation steps (measured: ~2.7e-7 of the largest |dw| per 16-token chunk, independent
    // of the layer shape).  A CTA therefore accumulates a bounded token range; the partial sums are added with
    // round-to-nearest by the finalize kernel.
    const int64_t cap = dtype == EQL_FP32 ? kMaxChunksPerSplitFp32 : kMaxChunksPerSplitFp16;
    int64_t launch_chunks = chunks;                              // chunks covered by one launch
    if (want * cap < chunks) {
        if (dtype == EQL_FP32) {
            // FP32 (12 chunks per accumulator): a launch of a few whole waves of CTAs covers a block of tokens, and the
            // blocks run one after the other into the same scratch, which stays within the built-in scratch array
            const size_t partial = ((size_t)T * Ci * Co + Co) * sizeof(float);
            int64_t waves = (int64_t)(kBlockScratchBudget / ((size_t)want * partial));
            if (waves < 1) waves = 1;
            if (waves > 8) waves = 8;
            const int64_t max_splits = want * waves;             // the same for every N: no block needs more scratch than the first
            const int64_t block = max_splits * cap;
            if (block < chunks) {
                launch_chunks = block;
                s.block_tokens = block * kChunkTok;
                want = max_splits;
            } else {
                const int64_t need = (chunks + cap - 1) / cap;
                const int64_t w = (need * tiles + num_sms - 1) / num_sms;      // whole waves of CTAs
                want = w * num_sms / tiles;
                if (want < need) want = need;
                if (want > max_splits) want = max_splits;
            }
        } else {
            // FP16 (the same effect against the 3e-3 bar only matters beyond ~10^4 chunks per accumulator): more splits
            const int64_t need = (chunks + cap - 1) / cap;
            const int64_t w = (need * tiles + num_sms - 1) / num_sms;
            want = w * num_sms / tiles;
            if (want < need) want = need;
        }
    }
    if (want > launch_chunks) want = launch_chunks;
    s.chunks_per_split = (launch_chunks + want - 1) / want;
    s.splits = (int)((launch_chunks + s.chunks_per_split - 1) / s.chunks_per_split);
    s.scratch_bytes = align_up((size_t)s.splits * ((size_t)T * Co * Ci + Co) * sizeof(float), kWsAlign);
    s.total_chunks = chunks;
    s.stash_bytes = s.elem_bytes == 2 ? align_up((size_t)s.nCiTiles * chunks * ((size_t)T * s.CiT * 32), kWsAlign) : 0;
    return s;
}

cudaError_t launch_umma_bwd_weight(const UmmaBwdWeightShape& s, const void* x, const void* dy, int64_t N,
                                   float* scratch, int* status, cudaStream_t stream) {
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return cudaErrorNotSupported;
    CUtensorMap mx, my;
    const int E = s.elem_bytes, epr = 128 / E, nsplit = E == 4 ? 2 : 1;
    const int64_t xcols = (int64_t)s.Ci * s.T, ycols = (int64_t)s.Co * s.T;
    const bool x3d = (xcols % epr == 0) && encode_slabs3d(enc, &mx, x, xcols, N, s.nXs, E);
    const bool y3d = (ycols % epr == 0) && encode_slabs3d(enc, &my, dy, ycols, N, s.nYs, E);
    if (!x3d && !encode_rows16(enc, &mx, x, xcols, N, E)) return cudaErrorInvalidValue;
    if (!y3d && !encode_rows16(enc, &my, dy, ycols, N, E)) return cudaErrorInvalidValue;
    // partial spectra [splits*T][Co][Ci] floats as a 3-D tensor for the epilogue's TMA stores (box 32 x 16 x 1)
    CUtensorMap mp;
    bool part_tma = (s.Ci % 4 == 0) && (reinterpret_cast<uintptr_t>(scratch) % 16 == 0);
    if (part_tma) {
        const cuuint64_t gdim[3] = {(cuuint64_t)s.Ci, (cuuint64_t)s.Co, (cuuint64_t)s.splits * s.T};
        const cuuint64_t gstr[2] = {(cuuint64_t)s.Ci * sizeof(float), (cuuint64_t)s.Ci * s.Co * sizeof(float)};
        const cuuint32_t box[3] = {32, 16, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        part_tma = enc(&mp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, scratch, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    if (!part_tma) mp = mx;                                     // unused by the kernel then; any valid map will do
    BwParams prm{};
    prm.x3d = x3d; prm.y3d = y3d; prm.part_tma = part_tma;
    prm.part = scratch;
    prm.db_part = scratch + (size_t)s.splits * s.T * s.Co * s.Ci;
    prm.status = status;
    prm.N = N; prm.Ci = s.Ci; prm.Co = s.Co; prm.CiT = s.CiT; prm.CoT = s.CoT;
    prm.nCiTiles = s.nCiTiles; prm.nCoTiles = s.nCoTiles; prm.nXs = s.nXs; prm.nYs = s.nYs;
    prm.splits = s.splits; prm.chunks_per_split = s.chunks_per_split;
    const int ytiles = 2 + 3 * (s.T / 2 - 1);
    const int chan_bytes = bw_chan_bytes(E);
    prm.x_part_bytes = s.T * ((s.CiT + 7) / 8 * 8) * chan_bytes;  // one copy of the x^ planes
    prm.y_part_bytes = ytiles * s.CoT * chan_bytes;              // one copy of the dy^ tiles
    prm.xhat_bytes = nsplit * prm.x_part_bytes;
    prm.stage_bytes = (int)bw_stage_bytes(s.T, s.CiT, s.CoT, E);
    prm.raw_slots = s.raw_slots; prm.y_slab0 = s.y_slab0;
    prm.stages = bw_fixed_smem(s.raw_slots) + 2 * (size_t)prm.stage_bytes <= 227 * 1024 ? 2 : 1;
    const size_t smem = bw_fixed_smem(s.raw_slots) + (size_t)prm.stages * prm.stage_bytes;
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
    const int grid = s.splits * s.nCiTiles * s.nCoTiles;

    auto go = [&](auto tc, auto io) -> cudaError_t {
        constexpr int TT = decltype(tc)::value;
        using IO = decltype(io);
        static SmemLimitOnce smem_limit;                      // per kernel instantiation
        if (cudaError_t e = smem_limit.ensure(umma_bwd_weight_kernel<TT, IO>, 227 * 1024); e != cudaSuccess) return e;
        return launch_overlapped(umma_bwd_weight_kernel<TT, IO>, dim3(grid), dim3(kThreadsBw), smem, stream, mx, my, mp, prm);
    };
    if (E == 4) {
        if (s.T == 4) return go(std::integral_constant<int, 4>{}, float{});
        if (s.T == 8) return go(std::integral_constant<int, 8>{}, float{});
        return cudaErrorInvalidValue;
    }
    if (s.bf16) {
        switch (s.T) {
            case 4: return go(std::integral_constant<int, 4>{}, __nv_bfloat16{});
            case 8: return go(std::integral_constant<int, 8>{}, __nv_bfloat16{});
            case 16: return go(std::integral_constant<int, 16>{}, __nv_bfloat16{});
            case 32: return go(std::integral_constant<int, 32>{}, __nv_bfloat16{});
            default: return cudaErrorInvalidValue;
        }
    }
    switch (s.T) {
        case 4: return go(std::integral_constant<int, 4>{}, __half{});
        case 8: return go(std::integral_constant<int, 8>{}, __half{});
        case 16: return go(std::integral_constant<int, 16>{}, __half{});
        case 32: return go(std::integral_constant<int, 32>{}, __half{});
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace eql
