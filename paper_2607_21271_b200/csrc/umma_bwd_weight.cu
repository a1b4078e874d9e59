// Weight gradient on the tcgen05 tensor cores (FP16 inputs, FP32 accumulation in TMEM):
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
    int x3d, y3d;                // tensor maps are 3-D (64 elements, rows, slab index): one load per chunk and tensor
};

// Optional timeline instrumentation (compiled only with -DEQL_TRACE): CTA 0 records clock64() stamps.
#ifdef EQL_TRACE
__device__ unsigned long long g_trace_bw[8192];
#define BW_STAMP(slot) do { if (blockIdx.x == 0 && (slot) < 8192) g_trace_bw[(slot)] = clock64(); } while (0)
#else
#define BW_STAMP(slot) do { } while (0)
#endif

struct BwBarriers {
    uint64_t full_raw[kRawSlots], empty_raw[kRawSlots];
    uint64_t full_ab[kStages], empty_ab[kStages];
    uint64_t full_d, mma_done;
    uint32_t tmem_base;
    int abort_flag;
};

template <int T>
__global__ void __launch_bounds__(kThreadsBw, 1)
umma_bwd_weight_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                       const BwParams prm) {
    constexpr int NCH = 64 / T;
    extern __shared__ uint8_t smem_raw_base[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~(uintptr_t)1023);
    BwBarriers* bar = reinterpret_cast<BwBarriers*>(smem);
    uint8_t* raw = smem + 1024;                                  // kRawSlots x 48 KB
    uint8_t* stages = raw + kRawSlots * kRawSlot;                // kStages x stage_bytes (+ 4 KB slack after the last)

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
                const int slot = (int)(c % kRawSlots);
                ok = ptx::mbar_wait(&bar->empty_raw[slot], (uint32_t)((c / kRawSlots) & 1) ^ 1, abort_flag, status, 201);
                if (!ok) break;
                BW_STAMP(3000 + (int)c);
                ptx::mbar_arrive_expect_tx(&bar->full_raw[slot], bytes);
                const int row = (int)((chunk0 + c) * kChunkTok);
                uint8_t* dst = raw + slot * kRawSlot;
                // One 3-D box [slab][16 rows][64 elements] per tensor where the row length is a whole number of
                // slabs; otherwise one 2-D box per slab (the same shared-memory layout either way).
                if (prm.x3d) {
                    ptx::tma_load_3d(dst, &tmap_x, 0, row, ci_tile * CiT * T / 64, &bar->full_raw[slot]);
                } else {
                    for (int s = 0; s < prm.nXs; ++s)
                        ptx::tma_load_2d(dst + s * kSlab, &tmap_x, ci_tile * CiT * T + s * 64, row, &bar->full_raw[slot]);
                }
                if (prm.y3d) {
                    ptx::tma_load_3d(dst + kMaxXSlabs * kSlab, &tmap_dy, 0, row, co_tile * CoT * T / 64, &bar->full_raw[slot]);
                } else {
                    for (int s = 0; s < prm.nYs; ++s)
                        ptx::tma_load_2d(dst + (kMaxXSlabs + s) * kSlab, &tmap_dy, co_tile * CoT * T + s * 64, row,
                                         &bar->full_raw[slot]);
                }
            }
            if (!ok) {
                const int64_t lo = c > kRawSlots ? c - kRawSlots : 0;
                for (int64_t d = lo; d < c; ++d)
                    ptx::mbar_wait(&bar->full_raw[d % kRawSlots], (uint32_t)((d / kRawSlots) & 1), abort_flag, status, 211, false);
            }
        }
    } else if (warp == kWarpMmaBw) {
        if (lane == 0) {
            bool ok = true;
            const uint32_t idesc_real = ptx::umma_idesc_f16_f32_mn_major(128, CoT);
            const uint32_t idesc_cplx = ptx::umma_idesc_f16_f32_mn_major(128, 2 * CoT);
            const uint32_t a_plane = (uint32_t)CiT * 32u, b_tile = (uint32_t)CoT * 32u;
            for (int64_t c = 0; c < nchunks; ++c) {
                const int st = (int)(c % kStages);
                BW_STAMP(1000 + 3 * (int)c);
                ok = ptx::mbar_wait(&bar->full_ab[st], (uint32_t)((c / kStages) & 1), abort_flag, status, 202);
                BW_STAMP(1000 + 3 * (int)c + 1);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t a0 = ptx::smem_u32(stages + st * prm.stage_bytes);
                const uint32_t b0 = a0 + prm.xhat_bytes;
                const uint32_t acc = c > 0 ? 1u : 0u;
                // MN-major no-swizzle: lbo = stride between 8-token groups (128 B), sbo = stride between 8-channel groups (256 B)
                ptx::umma_f16(tmem_base, ptx::umma_smem_desc(a0, 128, 256), ptx::umma_smem_desc(b0, 128, 256), idesc_real, acc);
#pragma unroll
                for (int f = 1; f < T / 2; ++f) {
                    const uint32_t d = tmem_base + (uint32_t)((2 * f - 1) * CoT);
                    const uint32_t bt = b0 + (uint32_t)(1 + 3 * (f - 1)) * b_tile;          // tiles Gr | Gi | -Gr
                    ptx::umma_f16(d, ptx::umma_smem_desc(a0 + (2 * f - 1) * a_plane, 128, 256),
                                  ptx::umma_smem_desc(bt, 128, 256), idesc_cplx, acc);       // Xr^T [Gr | Gi]
                    ptx::umma_f16(d, ptx::umma_smem_desc(a0 + (2 * f) * a_plane, 128, 256),
                                  ptx::umma_smem_desc(bt + b_tile, 128, 256), idesc_cplx, 1u);  // Xi^T [Gi | -Gr]
                }
                ptx::umma_f16(tmem_base + (uint32_t)((T - 1) * CoT), ptx::umma_smem_desc(a0 + (T - 1) * a_plane, 128, 256),
                              ptx::umma_smem_desc(b0 + (uint32_t)(1 + 3 * (T / 2 - 1)) * b_tile, 128, 256), idesc_real, acc);
                ptx::umma_commit(&bar->empty_ab[st]);
                BW_STAMP(1000 + 3 * (int)c + 2);
            }
            if (ok) ptx::umma_commit(&bar->full_d);
            ptx::umma_commit(&bar->mma_done);
            ptx::mbar_wait(&bar->mma_done, 0, abort_flag, status, 213, false);
        }
    } else if (warp >= kWarpDftX0) {
        // ------------------------------------------------------------ transform warps
        const bool is_y = warp >= kWarpDftY0;
        const int wi = is_y ? warp - kWarpDftY0 : warp - kWarpDftX0;
        const int half = lane >> 4, row = lane & 15;
        const int slab = 2 * wi + half;
        const bool active = slab < (is_y ? prm.nYs : prm.nXs);
        float dbacc[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) dbacc[i] = 0.f;
        bool ok = true;
        for (int64_t c = 0; c < nchunks; ++c) {
            const int slot = (int)(c % kRawSlots), st = (int)(c % kStages);
#ifdef EQL_TRACE
            const bool tr = lane == 0 && (warp == kWarpDftX0 || warp == kWarpDftY0);
            const int tb = (warp == kWarpDftX0 ? 4000 : 5000) + 6 * (int)c;
            if (tr) BW_STAMP(tb);
#endif
            ok = ptx::mbar_wait(&bar->full_raw[slot], (uint32_t)((c / kRawSlots) & 1), abort_flag, status, 203);
#ifdef EQL_TRACE
            if (tr) BW_STAMP(tb + 1);
#endif
            ok = ok && ptx::mbar_wait(&bar->empty_ab[st], (uint32_t)((c / kStages) & 1) ^ 1, abort_flag, status, 204);
#ifdef EQL_TRACE
            if (tr) BW_STAMP(tb + 2);
#endif
            if (!ok) break;
            uint32_t wd[32];
            if (active)
                load_slab_row(raw + slot * kRawSlot + ((is_y ? kMaxXSlabs : 0) + slab) * kSlab + row * 128, row, wd);
            // The rows are in registers: order these generic-proxy reads before the async-proxy (TMA) refill of
            // the slot, then release it so that the refill overlaps the transform.
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->empty_raw[slot]);
            if (active) {
                uint32_t packed[T][NCH / 2];
                float p0[NCH];
#ifdef EQL_ABLATE_DFT
#pragma unroll
                for (int p = 0; p < T; ++p)
#pragma unroll
                    for (int c2 = 0; c2 < NCH / 2; ++c2) packed[p][c2] = wd[(p * (NCH / 2) + c2) & 31];
#pragma unroll
                for (int i = 0; i < NCH; ++i) p0[i] = 0.f;
#else
                dft_words<T, true>(wd, packed, p0);
#endif
                const int mn0 = slab * NCH;                      // first channel of this slab inside the tile
                // MN-major tile: (channel mn, token k) at (mn/8)*256 + (k/8)*128 + (k%8)*16 + (mn%8)*2
                const int off = (mn0 >> 3) * 256 + (row >> 3) * 128 + (row & 7) * 16 + (mn0 & 7) * 2;
                uint8_t* stage = stages + st * prm.stage_bytes;
                if (!is_y) {
#pragma unroll
                    for (int p = 0; p < T; ++p) store_plane_run<NCH>(stage + p * CiT * 32 + off, packed[p], 256);
                } else {
#pragma unroll
                    for (int i = 0; i < NCH; ++i) dbacc[i] += p0[i];
                    uint8_t* yb = stage + prm.xhat_bytes + off;
                    const int tb = CoT * 32;
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
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->full_ab[st]);
#ifdef EQL_TRACE
            if (tr) BW_STAMP(tb + 3);
#endif
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
                for (int col = third * 16; col < T * CoT; col += 48) {
                    uint32_t v[16];
                    if (nchunks > 0) {
                        ptx::tmem_ld<16>(lane_base + (uint32_t)col, v);
                        ptx::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = 0u;
                    }
                    const int p = col / CoT, o0 = co_tile * CoT + col % CoT;
                    if (lane_ok) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (o0 + j < prm.Co) dst[p * plane_stride + (size_t)(o0 + j) * prm.Ci + ci] = __uint_as_float(v[j]);
                    }
                }
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

bool encode_rows16(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows) {
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)cols * sizeof(__half)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kChunkTok};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view of a [rows, cols] half tensor whose row length is a multiple of 64 elements:
// dim0 = 64 contiguous elements, dim1 = rows (stride = row pitch), dim2 = slab index (stride = 128 bytes).
// A box [64, 16, nslabs] lands in shared memory as nslabs consecutive [16 x 128 B] slabs.
bool encode_slabs3d(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows, int nslabs) {
    const cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
    const cuuint64_t gstr[2] = {(cuuint64_t)cols * sizeof(__half), 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)kChunkTok, (cuuint32_t)nslabs};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int balanced_tile(int C, int max_tile, int round) {
    const int n = (C + max_tile - 1) / max_tile;
    const int per = (C + n - 1) / n;
    return (per + round - 1) / round * round;
}

}  // namespace

#ifdef EQL_TRACE
extern "C" int eqlinear_debug_read_trace_bw(unsigned long long* dst, int n) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(dst, g_trace_bw, sizeof(unsigned long long) * (n < 8192 ? n : 8192));
}
#endif

bool umma_bwd_weight_supported(int T, eql_dtype_t dtype) {
    return dtype == EQL_FP16 && (T == 4 || T == 8 || T == 16 || T == 32);
}

UmmaBwdWeightShape umma_bwd_weight_shape(int T, int Ci, int Co, int64_t N, int num_sms) {
    UmmaBwdWeightShape s{};
    s.T = T; s.Ci = Ci; s.Co = Co;
    int max_cit = 1024 / T;                                      // at most 16 raw slabs of x per chunk
    if (max_cit > 128) max_cit = 128;                            // UMMA M = 128 TMEM lanes
    s.CiT = balanced_tile(Ci, max_cit, T == 4 ? 16 : 8);
    s.nCiTiles = (Ci + s.CiT - 1) / s.CiT;
    s.CoT = balanced_tile(Co, kTmemColsBw / T, 16);
    s.nCoTiles = (Co + s.CoT - 1) / s.CoT;
    s.nXs = s.CiT * T / 64;
    s.nYs = s.CoT * T / 64;
    const int64_t tiles = (int64_t)s.nCiTiles * s.nCoTiles;
    const int64_t chunks = N > 0 ? (N + kChunkTok - 1) / kChunkTok : 1;
    int64_t want = num_sms / tiles;
    if (want < 1) want = 1;
    if (want > chunks) want = chunks;
    s.chunks_per_split = (chunks + want - 1) / want;
    s.splits = (int)((chunks + s.chunks_per_split - 1) / s.chunks_per_split);
    s.scratch_bytes = align_up((size_t)s.splits * ((size_t)T * Co * Ci + Co) * sizeof(float), kWsAlign);
    return s;
}

cudaError_t launch_umma_bwd_weight(const UmmaBwdWeightShape& s, const void* x, const void* dy, int64_t N,
                                   float* scratch, int* status, cudaStream_t stream) {
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return cudaErrorNotSupported;
    CUtensorMap mx, my;
    const int64_t xcols = (int64_t)s.Ci * s.T, ycols = (int64_t)s.Co * s.T;
    const bool x3d = (xcols % 64 == 0) && encode_slabs3d(enc, &mx, x, xcols, N, s.nXs);
    const bool y3d = (ycols % 64 == 0) && encode_slabs3d(enc, &my, dy, ycols, N, s.nYs);
    if (!x3d && !encode_rows16(enc, &mx, x, xcols, N)) return cudaErrorInvalidValue;
    if (!y3d && !encode_rows16(enc, &my, dy, ycols, N)) return cudaErrorInvalidValue;
    BwParams prm{};
    prm.x3d = x3d; prm.y3d = y3d;
    prm.part = scratch;
    prm.db_part = scratch + (size_t)s.splits * s.T * s.Co * s.Ci;
    prm.status = status;
    prm.N = N; prm.Ci = s.Ci; prm.Co = s.Co; prm.CiT = s.CiT; prm.CoT = s.CoT;
    prm.nCiTiles = s.nCiTiles; prm.nCoTiles = s.nCoTiles; prm.nXs = s.nXs; prm.nYs = s.nYs;
    prm.splits = s.splits; prm.chunks_per_split = s.chunks_per_split;
    prm.xhat_bytes = s.T * s.CiT * 32;
    const int ytiles = 2 + 3 * (s.T / 2 - 1);
    prm.stage_bytes = (int)align_up((size_t)prm.xhat_bytes + (size_t)ytiles * s.CoT * 32, 1024);
    const size_t smem = 1024 + 1024 + (size_t)kRawSlots * kRawSlot + (size_t)kStages * prm.stage_bytes + 4096;
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
    const int grid = s.splits * s.nCiTiles * s.nCoTiles;

    auto go = [&](auto tc) -> cudaError_t {
        constexpr int TT = decltype(tc)::value;
        static unsigned long long attr_done = 0;
        int dev = 0;
        cudaGetDevice(&dev);
        if (!((attr_done >> (dev & 63)) & 1ull)) {
            cudaError_t e = cudaFuncSetAttribute(umma_bwd_weight_kernel<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            if (e != cudaSuccess) return e;
            attr_done |= 1ull << (dev & 63);
        }
        umma_bwd_weight_kernel<TT><<<grid, kThreadsBw, smem, stream>>>(mx, my, prm);
        return cudaGetLastError();
    };
    switch (s.T) {
        case 4: return go(std::integral_constant<int, 4>{});
        case 8: return go(std::integral_constant<int, 8>{});
        case 16: return go(std::integral_constant<int, 16>{});
        case 32: return go(std::integral_constant<int, 32>{});
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace eql
