// Weight gradient from a SAVED spectrum of x (FP16, tcgen05): the forward pass (or a pre-pass kernel) has written
// x^ -- the group DFT of x, rounded to fp16 -- as the operand image of this kernel, so the transform of x, which the
// plain weight-gradient kernel repeats for every output-channel tile, is not done here at all.
//
//   image: for every (input-channel tile, 16-token chunk) one blob of T planes, each an MN-major
//          [CiT channels x 16 tokens] tile: (channel mn, token k) at (mn/8)*256 + (k/8)*128 + (k%8)*16 + (mn%8)*2
//   bulk copies (1 thread)     x^ blob of every chunk                       -> ring of shared-memory slots
//   TMA (1 thread)             16-token slabs of dy                         -> raw slots
//   12 transform warps         three groups take the chunks round-robin: group DFT of dy (Eq. 4) in registers
//                              -> MN-major dy^ operand tiles (with -Re dy^ stored once more per complex frequency)
//   1 thread                   tcgen05.mma, A = x^ plane, B = dy^ planes    -> TMEM (all T planes of one tile pair)
//   12 warps (after the loop)  tcgen05.ld -> partial spectra (TMA tensor stores); db partials from plane k = 0
//
// Partials and the finalize kernel are those of umma_bwd_weight.cu.  All mbarrier waits are bounded.
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
constexpr int kMaxYSlabs = 8;
constexpr int kRawSlot = kMaxYSlabs * kSlab;  // 16 KB: the dy rows of one chunk
constexpr int kThreadsBw = 512;
constexpr int kTmemColsBw = 512;
// Three transform groups of four warps take the chunks round-robin; chunk c uses raw slot, operand stage and group
// c % 3, so every barrier is always waited on by the same threads (a parity wait is only unambiguous one phase ahead).
constexpr int kGroups = 3, kWarpsPerGroup = 4;
constexpr int kWarpTma = 0, kWarpMmaBw = 1, kWarpTmaX = 2, kWarpDft0 = 4;
constexpr int kMaxXSlots = 6;                 // ring of transformed-x blobs, filled ahead of the dy pipeline
constexpr int kMaxCoT = 128;

struct BwParams {
    float* part;                 // [splits][T][Co][Ci]
    float* db_part;              // [splits][Co]
    const uint8_t* ximage;       // transformed x, see xhat_image_kernel
    int* status;
    int64_t N;
    int Ci, Co, CiT, CoT, nCiTiles, nCoTiles, nYs;
    int splits;
    int64_t chunks_per_split;    // 16-token chunks per token range
    int64_t total_chunks;
    int xhat_bytes, stage_bytes;  // x^ blob of a chunk; dy^ operand tiles of a chunk
    int x_slots;                 // depth of the x^ ring
    int y3d;                     // dy tensor map is 3-D (64 elements, rows, slab index): one load per chunk
    int part_tma;                // the partial spectra can be written with TMA tensor stores
};


struct BwBarriers {
    uint64_t full_raw[kGroups], empty_raw[kGroups];
    uint64_t full_ab[kGroups], empty_ab[kGroups];
    uint64_t full_x[kMaxXSlots], empty_x[kMaxXSlots];   // ring of x^ blobs (bulk copies), freed by the MMAs that read them
    uint64_t full_d, mma_done;
    uint32_t tmem_base;
    int abort_flag;
    float db[kGroups][kMaxCoT];  // bias-gradient partial of this CTA's output channels, one row per transform group
};

// ------------------------------------------------------------------------------------------------
// Pre-pass: group DFT (Eq. 4) of x, rounded to fp16 once, written as the tensor-core operand image of the
// weight-gradient kernel: for every (input-channel tile, 16-token chunk) one blob of T planes, each an MN-major
// [CiT channels x 16 tokens] tile:  (channel mn, token k) at (mn/8)*256 + (k/8)*128 + (k%8)*16 + (mn%8)*2.
// The six output-channel tiles of the EQ-ViT-B layer then share one transform of x instead of repeating it.
// One half warp per 64-element slab of a token row, one token per lane; rows >= N and channels >= Ci are zero.
template <int T, typename IO>
__global__ void xhat_image_kernel(const IO* __restrict__ x, int64_t N, int Ci, int CiT, int nXs, int64_t total_chunks,
                                  uint8_t* __restrict__ image) {
    constexpr int NCH = 64 / T;
    const int64_t blob = blockIdx.x;                             // = ci_tile * total_chunks + chunk
    const int ci_tile = (int)(blob / total_chunks);
    const int64_t chunk = blob % total_chunks;
    const int hw = threadIdx.x >> 4, row = threadIdx.x & 15;
    if (hw >= nXs) return;
    const int64_t token = chunk * kChunkTok + row;
    const int64_t e0 = (int64_t)ci_tile * CiT * T + (int64_t)hw * 64;   // first element of this slab in the token row
    const int64_t row_elems = (int64_t)Ci * T;
    uint32_t wd[32];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (token < N && e0 + 8 * j < row_elems)
            v = __ldg(reinterpret_cast<const uint4*>(x + token * row_elems + e0 + 8 * j));
        wd[4 * j] = v.x; wd[4 * j + 1] = v.y; wd[4 * j + 2] = v.z; wd[4 * j + 3] = v.w;
    }
    uint32_t packed[T][NCH / 2];
    dft_words<T, false, false, IO>(wd, packed, nullptr);
    const int mn0 = hw * NCH;
    const int off = (mn0 >> 3) * 256 + (row >> 3) * 128 + (row & 7) * 16 + (mn0 & 7) * 2;
    uint8_t* dst = image + (size_t)blob * ((size_t)T * CiT * 32) + off;
#pragma unroll
    for (int p = 0; p < T; ++p) store_plane_run<NCH>(dst + (size_t)p * CiT * 32, packed[p], 256);
}

// MERGED (x^ ring as deep as the dy^ stages, i.e. three): chunk c uses stage c % 3 and ring slot c % 3, so one "full"
// barrier (the group's transform warps + the x^ copy) and one "empty" barrier (one commit) per chunk serve both, and
// the MMA-issuing thread - which paces this kernel - handles half as many barrier operations.
template <int T, bool MERGED, typename IO>
__global__ void __launch_bounds__(kThreadsBw, 1)
umma_bwd_weight_saved_kernel(const __grid_constant__ CUtensorMap tmap_dy, const __grid_constant__ CUtensorMap tmap_part,
                             const BwParams prm) {
    constexpr int NCH = 64 / T;
    extern __shared__ uint8_t smem_raw_base[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~(uintptr_t)1023);
    BwBarriers* bar = reinterpret_cast<BwBarriers*>(smem);
    uint8_t* raw = smem + 2048;                                  // kGroups x 16 KB of dy rows
    uint8_t* stages = raw + kGroups * kRawSlot;                  // kGroups x stage_bytes: dy^ operand tiles
    uint8_t* xring = stages + kGroups * prm.stage_bytes;         // x_slots x xhat_bytes (+ 4 KB slack after the last)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &bar->abort_flag;
    int* status = prm.status;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kGroups; ++i) {
            ptx::mbar_init(&bar->full_raw[i], 1);
            ptx::mbar_init(&bar->empty_raw[i], kWarpsPerGroup);
            ptx::mbar_init(&bar->full_ab[i], kWarpsPerGroup + (MERGED ? 1 : 0));   // the group's warps have stored dy^ (+ the x^ copy)
            ptx::mbar_init(&bar->empty_ab[i], 1);
        }
        for (int i = 0; i < kMaxXSlots; ++i) { ptx::mbar_init(&bar->full_x[i], 1); ptx::mbar_init(&bar->empty_x[i], 1); }
        ptx::mbar_init(&bar->full_d, 1);
        ptx::mbar_init(&bar->mma_done, 1);
        bar->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_dy);
    }
    if (threadIdx.x < kGroups * kMaxCoT) (&bar->db[0][0])[threadIdx.x] = 0.f;
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
    // CTAs sharing the same x^ blobs run at the same time
    const int co_tile = blockIdx.x % prm.nCoTiles;
    const int ci_tile = (blockIdx.x / prm.nCoTiles) % prm.nCiTiles;
    const int split = blockIdx.x / (prm.nCoTiles * prm.nCiTiles);
    const int64_t chunk0 = (int64_t)split * prm.chunks_per_split;
    int64_t nchunks = prm.total_chunks - chunk0;
    if (nchunks > prm.chunks_per_split) nchunks = prm.chunks_per_split;
    if (nchunks < 0) nchunks = 0;
    const int CiT = prm.CiT, CoT = prm.CoT;

    if (warp == kWarpTma) {
        if (lane == 0) {
            // ---- dy rows of every chunk -> raw slot of the chunk's group
            bool ok = true;
            int64_t ny = 0;
            const uint32_t ybytes = (uint32_t)prm.nYs * kSlab;
            int slot = 0;
            uint32_t eph = 1;                                    // parity to wait for on the slot's "empty" barrier
            for (int64_t c = 0; c < nchunks; ++c, ++ny) {
                if (c > 0 && ++slot == kGroups) { slot = 0; eph ^= 1u; }
                ok = ptx::mbar_wait(&bar->empty_raw[slot], eph, abort_flag, status, 201);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx(&bar->full_raw[slot], ybytes);
                const int row = (int)((chunk0 + c) * kChunkTok);
                uint8_t* dst = raw + slot * kRawSlot;
                // One 3-D box [slab][16 rows][64 elements] where the row length is a whole number of slabs;
                // otherwise one 2-D box per slab (the same shared-memory layout either way).
                if (prm.y3d) {
                    ptx::tma_load_3d(dst, &tmap_dy, 0, row, co_tile * CoT * T / 64, &bar->full_raw[slot]);
                } else {
                    for (int s = 0; s < prm.nYs; ++s)
                        ptx::tma_load_2d(dst + s * kSlab, &tmap_dy, co_tile * CoT * T + s * 64, row, &bar->full_raw[slot]);
                }
            }
            if (!ok)                                             // drain: every copy issued must land before the CTA may exit
                for (int64_t d = ny > kGroups ? ny - kGroups : 0; d < ny; ++d)
                    ptx::mbar_wait(&bar->full_raw[d % kGroups], (uint32_t)((d / kGroups) & 1), abort_flag, status, 211, false);
        }
    } else if (warp == kWarpTmaX) {
        if (lane == 0) {
            // ---- x^ blob of every chunk -> ring slot (freed when the MMAs that read it have retired)
            bool ok = true;
            int64_t nx = 0;
            const int XS = MERGED ? kGroups : prm.x_slots;
            uint64_t* const full_xb = MERGED ? bar->full_ab : bar->full_x;
            uint64_t* const empty_xb = MERGED ? bar->empty_ab : bar->empty_x;
            const uint8_t* xsrc = prm.ximage + ((size_t)ci_tile * prm.total_chunks + chunk0) * (size_t)prm.xhat_bytes;
            int slot = 0;
            uint32_t eph = 1;
            for (int64_t c = 0; c < nchunks; ++c, ++nx) {
                if (c > 0 && ++slot == XS) { slot = 0; eph ^= 1u; }
                ok = ptx::mbar_wait(&empty_xb[slot], eph, abort_flag, status, 206);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx(&full_xb[slot], (uint32_t)prm.xhat_bytes);
                ptx::bulk_load_1d(xring + slot * prm.xhat_bytes, xsrc + (size_t)c * prm.xhat_bytes, (uint32_t)prm.xhat_bytes,
                                  &full_xb[slot]);
            }
            if (!ok)
                for (int64_t d = nx > XS ? nx - XS : 0; d < nx; ++d)
                    ptx::mbar_wait(&full_xb[d % XS], (uint32_t)((d / XS) & 1), abort_flag, status, 212, false);
        }
    } else if (warp == kWarpMmaBw) {
        if (lane == 0) {
            bool ok = true;
            const uint32_t idesc_real = ptx::umma_idesc_f16_f32_mn_major(128, CoT, H16<IO>::kUmmaFormat);
            const uint32_t idesc_cplx = ptx::umma_idesc_f16_f32_mn_major(128, 2 * CoT, H16<IO>::kUmmaFormat);
            const uint32_t a_plane = (uint32_t)CiT * 32u, b_tile = (uint32_t)CoT * 32u;
            const int XS = MERGED ? kGroups : prm.x_slots;
            int st = 0, xs = 0;                                  // dy^ stage and x^ ring slot of the current chunk
            uint32_t sph = 0, xph = 0;                           // their phase parities
            if (nchunks > 0)
                ok = ptx::mbar_wait(&bar->full_ab[0], 0, abort_flag, status, 202) &&
                     (MERGED || ptx::mbar_wait(&bar->full_x[0], 0, abort_flag, status, 207));
            for (int64_t c = 0; c < nchunks && ok; ++c) {
                ptx::tc_fence_after_sync();
                const uint32_t a0 = ptx::smem_u32(xring + xs * prm.xhat_bytes);
                const uint32_t b0 = ptx::smem_u32(stages + st * prm.stage_bytes);
                const uint32_t acc = c > 0 ? 1u : 0u;
                int nst = st + 1, nxs = xs + 1;
                uint32_t nsph = sph, nxph = xph;
                if (nst == kGroups) { nst = 0; nsph ^= 1u; }
                if (nxs == XS) { nxs = 0; nxph ^= 1u; }
                // MN-major no-swizzle: lbo = stride between 8-token groups (128 B), sbo = stride between 8-channel groups (256 B);
                // the descriptors of the chunk's first tiles are built once and advanced by (byte offset >> 4)
                const uint64_t ad = ptx::umma_smem_desc(a0, 128, 256), bd = ptx::umma_smem_desc(b0, 128, 256);
                const uint64_t ap = a_plane >> 4, bt1 = b_tile >> 4;
                ptx::umma_f16(tmem_base, ad, bd, idesc_real, acc);
#pragma unroll
                for (int f = 1; f < T / 2; ++f) {
                    const uint32_t d = tmem_base + (uint32_t)((2 * f - 1) * CoT);
                    const uint64_t bt = bd + (uint64_t)(1 + 3 * (f - 1)) * bt1;             // tiles Gr | Gi | -Gr
                    ptx::umma_f16(d, ad + (2 * f - 1) * ap, bt, idesc_cplx, acc);            // Xr^T [Gr | Gi]
                    ptx::umma_f16(d, ad + (2 * f) * ap, bt + bt1, idesc_cplx, 1u);           // Xi^T [Gi | -Gr]
                    if (f == 1 && c + 1 < nchunks) {
                        // The next chunk's operands are checked here, while the tensor pipe still has this chunk's
                        // MMAs queued, so that the issue stream has no gap between chunks.
                        ok = ptx::mbar_wait(&bar->full_ab[nst], nsph, abort_flag, status, 202) &&
                             (MERGED || ptx::mbar_wait(&bar->full_x[nxs], nxph, abort_flag, status, 207));
                    }
                }
                ptx::umma_f16(tmem_base + (uint32_t)((T - 1) * CoT), ad + (T - 1) * ap,
                              bd + (uint64_t)(1 + 3 * (T / 2 - 1)) * bt1, idesc_real, acc);
                ptx::umma_commit(&bar->empty_ab[st]);
                if constexpr (!MERGED) ptx::umma_commit(&bar->empty_x[xs]);
                st = nst; xs = nxs; sph = nsph; xph = nxph;
            }
            if (ok) ptx::umma_commit(&bar->full_d);
            ptx::umma_commit(&bar->mma_done);
            ptx::mbar_wait(&bar->mma_done, 0, abort_flag, status, 213, false);
        }
    } else if (warp >= kWarpDft0) {
        // ------------------------------------------------------------ transform warps (dy only; x^ arrives transformed)
        const int wi = warp - kWarpDft0;
        const int g = wi / kWarpsPerGroup, wg = wi % kWarpsPerGroup;
        const int half = lane >> 4, row = lane & 15;
        const int slab = 2 * wg + half;                          // dy slab of the chunk this half warp owns
        const bool active = slab < prm.nYs;
        float dbacc[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) dbacc[i] = 0.f;
        bool ok = true;
        uint32_t ph = 0;                                         // phase parity of this group's slot and stage
        for (int64_t c = g; c < nchunks; c += kGroups, ph ^= 1u) {
            ok = ptx::mbar_wait(&bar->full_raw[g], ph, abort_flag, status, 203);
            if (!ok) break;
            uint32_t wd[32];
            if (active) load_slab_row(raw + g * kRawSlot + slab * kSlab + row * 128, row, wd);
            // The rows are in registers: order these generic-proxy reads before the async-proxy (TMA) refill of
            // the slot, then release it so that the refill overlaps the transform.
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->empty_raw[g]);
            uint32_t packed[T][NCH / 2];
            float p0[NCH];
            if (active) {
                dft_words<T, true, false, IO>(wd, packed, p0);
            }
            // the MMAs that read this stage three chunks ago must have retired
            ok = ptx::mbar_wait(&bar->empty_ab[g], ph ^ 1, abort_flag, status, 204);
            if (!ok) break;
            if (active) {
                const int mn0 = slab * NCH;                      // first channel of this slab inside the tile
                // MN-major tile: (channel mn, token k) at (mn/8)*256 + (k/8)*128 + (k%8)*16 + (mn%8)*2
                const int off = (mn0 >> 3) * 256 + (row >> 3) * 128 + (row & 7) * 16 + (mn0 & 7) * 2;
#pragma unroll
                for (int i = 0; i < NCH; ++i) dbacc[i] += p0[i];
                uint8_t* yb = stages + g * prm.stage_bytes + off;
                const int tb2 = CoT * 32;
                store_plane_run<NCH>(yb, packed[0], 256);
#pragma unroll
                for (int f = 1; f < T / 2; ++f) {
                    uint8_t* t0 = yb + (1 + 3 * (f - 1)) * tb2;
                    store_plane_run<NCH>(t0, packed[2 * f - 1], 256);                    // Gr
                    store_plane_run<NCH>(t0 + tb2, packed[2 * f], 256);                  // Gi
                    store_plane_run<NCH>(t0 + 2 * tb2, packed[2 * f - 1], 256, 0x80008000u);   // -Gr
                }
                store_plane_run<NCH>(yb + (1 + 3 * (T / 2 - 1)) * tb2, packed[T - 1], 256);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bar->full_ab[g]);
        }
        // db partial of this token range: sum over the 16 token rows of each half warp; the three groups' sums meet
        // in shared memory and are added in a fixed order at the end
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            float v = dbacc[i];
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            if (active && row == 0 && slab * NCH + i < kMaxCoT) bar->db[g][slab * NCH + i] = v;
        }
        // ------------------------------------------------------------ epilogue: TMEM -> partial spectra
        // all 12 warps: a warp reads the TMEM lane quadrant (warp & 3) and every third group of 16 columns
        if (ok) {
            const int quad = warp & 3;
            const int third = wi >> 2;
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
                // warp in the idle dy slots and stages); other quads write their valid lanes directly.
                const bool via_tma = prm.part_tma != 0 && quad * 32 + 32 <= CiT;
                float* stg = reinterpret_cast<float*>(raw + wi * 4096);
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
    if (bar->abort_flag == 0 && ci_tile == 0 && (int)threadIdx.x < CoT && co_tile * CoT + (int)threadIdx.x < prm.Co)
        prm.db_part[(size_t)split * prm.Co + co_tile * CoT + threadIdx.x] =
            (bar->db[0][threadIdx.x] + bar->db[1][threadIdx.x]) + bar->db[2][threadIdx.x];
    if (warp == kWarpMmaBw) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemColsBw);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn_saved() {
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

// dy as 2-D [rows, cols] half tensor, box 64 elements x 16 rows (one slab per load)
bool encode_dy_rows16(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows) {
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)cols * sizeof(__half)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kChunkTok};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// dy as 3-D view (64 elements, rows, slab index) where the row length is a multiple of 64 elements: a box
// [64, 16, nslabs] lands in shared memory as nslabs consecutive [16 x 128 B] slabs
bool encode_dy_slabs3d(EncodeTiledFn enc, CUtensorMap* map, const void* base, int64_t cols, int64_t rows, int nslabs) {
    const cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
    const cuuint64_t gstr[2] = {(cuuint64_t)cols * sizeof(__half), 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)kChunkTok, (cuuint32_t)nslabs};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace


// Pre-pass: the spectrum image of x for launch_umma_bwd_weight_saved (used when the forward pass that ran for this
// batch could not write it itself).
cudaError_t launch_xhat_image(const UmmaBwdWeightShape& s, const void* x, int64_t N, void* stash, cudaStream_t stream) {
    if (s.elem_bytes != 2) return cudaErrorInvalidValue;
    const int64_t blobs = (int64_t)s.nCiTiles * s.total_chunks;
    if (blobs > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int xthreads = (s.nXs * 16 + 31) / 32 * 32;
    switch (s.T) {
#define EQL_XHAT(TT)                                                                                                        \
    case TT:                                                                                                               \
        if (s.bf16) xhat_image_kernel<TT, __nv_bfloat16><<<(unsigned)blobs, xthreads, 0, stream>>>(                        \
            (const __nv_bfloat16*)x, N, s.Ci, s.CiT, s.nXs, s.total_chunks, (uint8_t*)stash);                              \
        else xhat_image_kernel<TT, __half><<<(unsigned)blobs, xthreads, 0, stream>>>(                                      \
            (const __half*)x, N, s.Ci, s.CiT, s.nXs, s.total_chunks, (uint8_t*)stash);                                     \
        break;
        EQL_XHAT(4) EQL_XHAT(8) EQL_XHAT(16) EQL_XHAT(32)
#undef EQL_XHAT
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_umma_bwd_weight_saved(const UmmaBwdWeightShape& s, const void* stash, const void* dy, int64_t N,
                                         float* scratch, int* status, cudaStream_t stream) {
    if (s.elem_bytes != 2) return cudaErrorInvalidValue;
    EncodeTiledFn enc = encode_fn_saved();
    if (enc == nullptr) return cudaErrorNotSupported;
    CUtensorMap my, mp;
    const int64_t ycols = (int64_t)s.Co * s.T;
    const bool y3d = (ycols % 64 == 0) && encode_dy_slabs3d(enc, &my, dy, ycols, N, s.nYs);
    if (!y3d && !encode_dy_rows16(enc, &my, dy, ycols, N)) return cudaErrorInvalidValue;
    // partial spectra [splits*T][Co][Ci] floats as a 3-D tensor for the epilogue's TMA stores (box 32 x 16 x 1)
    bool part_tma = (s.Ci % 4 == 0) && (reinterpret_cast<uintptr_t>(scratch) % 16 == 0);
    if (part_tma) {
        const cuuint64_t gdim[3] = {(cuuint64_t)s.Ci, (cuuint64_t)s.Co, (cuuint64_t)s.splits * s.T};
        const cuuint64_t gstr[2] = {(cuuint64_t)s.Ci * sizeof(float), (cuuint64_t)s.Ci * s.Co * sizeof(float)};
        const cuuint32_t box[3] = {32, 16, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        part_tma = enc(&mp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, scratch, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    if (!part_tma) mp = my;                                     // unused by the kernel then; any valid map will do
    BwParams prm{};
    prm.y3d = y3d; prm.part_tma = part_tma;
    prm.part = scratch;
    prm.db_part = scratch + (size_t)s.splits * s.T * s.Co * s.Ci;
    prm.ximage = (const uint8_t*)stash;
    prm.status = status;
    prm.N = N; prm.Ci = s.Ci; prm.Co = s.Co; prm.CiT = s.CiT; prm.CoT = s.CoT;
    prm.nCiTiles = s.nCiTiles; prm.nCoTiles = s.nCoTiles; prm.nYs = s.nYs;
    prm.splits = s.splits; prm.chunks_per_split = s.chunks_per_split; prm.total_chunks = s.total_chunks;
    prm.xhat_bytes = s.T * s.CiT * 32;
    const int ytiles = 2 + 3 * (s.T / 2 - 1);
    prm.stage_bytes = (int)align_up((size_t)ytiles * s.CoT * 32, 1024);
    const size_t fixed = 1024 + 2048 + (size_t)kGroups * kRawSlot + (size_t)kGroups * prm.stage_bytes + 4096;
    prm.x_slots = kGroups;                                           // three slots: the merged-barrier variant
    while (prm.x_slots > 2 && fixed + (size_t)prm.x_slots * prm.xhat_bytes > 227 * 1024) --prm.x_slots;
    const size_t smem = fixed + (size_t)prm.x_slots * prm.xhat_bytes;
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
    const int grid = s.splits * s.nCiTiles * s.nCoTiles;

    const bool merged = prm.x_slots == kGroups;
    auto go2 = [&](auto tc, auto mg) -> cudaError_t {
        constexpr int TT = decltype(tc)::value;
        constexpr bool MG = decltype(mg)::value;
        static SmemLimitOnce smem_limit[2];                   // per kernel instantiation
        if (s.bf16) {
            if (cudaError_t e = smem_limit[1].ensure(umma_bwd_weight_saved_kernel<TT, MG, __nv_bfloat16>, 227 * 1024); e != cudaSuccess) return e;
            return launch_overlapped(umma_bwd_weight_saved_kernel<TT, MG, __nv_bfloat16>, dim3(grid), dim3(kThreadsBw), smem, stream, my, mp, prm);
        }
        if (cudaError_t e = smem_limit[0].ensure(umma_bwd_weight_saved_kernel<TT, MG, __half>, 227 * 1024); e != cudaSuccess) return e;
        return launch_overlapped(umma_bwd_weight_saved_kernel<TT, MG, __half>, dim3(grid), dim3(kThreadsBw), smem, stream, my, mp, prm);
    };
    auto go = [&](auto tc) -> cudaError_t { return merged ? go2(tc, std::true_type{}) : go2(tc, std::false_type{}); };
    switch (s.T) {
        case 4: return go(std::integral_constant<int, 4>{});
        case 8: return go(std::integral_constant<int, 8>{});
        case 16: return go(std::integral_constant<int, 16>{});
        case 32: return go(std::integral_constant<int, 32>{});
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace eql
