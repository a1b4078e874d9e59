// Fused EQ-Linear forward / data-gradient with the transformed activations RESIDENT in shared memory (16-bit I/O: IEEE
// half or bfloat16; FP32 accumulation in TMEM, T = 4 or 8).  Used where the spectrum of one token tile fits on chip
// (C_in * T * 2 bytes * 512/T tokens <= ~150 KB), i.e. the layers with few input channels.
//
// Compared with the streaming kernel (umma_linear.cu) the roles of the two operands are exchanged: the
// accumulator holds OUTPUT CHANNELS on the 128 TMEM lanes and (plane, token) on the columns,
//     D_p[o, n] = sum_i w^_p[o, i] x^_p[n, i]          A = spectral weight tile [128 channels x 16], B = x^ tile [tokens x 16].
// A work unit is (tile of 512/T tokens, tile of 128 output channels); a CTA owns a contiguous range of units in
// token-major order, so the group DFT (Eq. 4) of a token tile is computed once and reused by all of its
// output-channel tiles, and only the spectral weights stream through a ring.
//
//   TMA (2-D, 128B swizzle)     raw rows of x, 32 tokens x 128 B per item         -> one ring slot per transform warp
//   transform warps             group DFT in registers, planes rounded to fp16    -> resident x^ tiles (K-major, 32B swizzle)
//   TMA (1-D bulk)              spectral-weight image of (channel tile, 16-channel chunk) -> weight ring
//   1 thread                    tcgen05.mma kind::f16; complex frequency (Eq. 5) as
//                                   [Re|Im] += Wr [Xr|Xi],   Re += (-Wi) Xi (A negated by the instruction),   Im += Wi Xr
//   12 warps (16 for T = 4)     tcgen05.ld, bias on plane k = 0, inverse DFT (Eq. 7), fp16 rounding; a thread owns one
//                               output channel, so a warp writes 32 channels x T elements of a token as one contiguous run
//
// The transform of the next token tile runs while the MMAs of the current tile's last channel tile are in flight
// (each x^ chunk is rewritten as soon as the MMAs that read it have retired).
//
// Two compile-time variants.  Resident mode: all chunks of a token tile stay in shared memory (several channel tiles).
// Ring mode (one channel tile, any C_in): three x^ chunk buffers and three weight slots used as rings with ONE
// full/empty barrier pair per chunk for both; this is the variant the data gradient of a wide-output layer runs.
//
// Every wait on an mbarrier is bounded: on a time-out the CTA raises an abort flag, records a status code for the
// host, drains its outstanding copies and MMAs, frees its TMEM and returns.
#include <cuda_fp16.h>

#include <cstring>
#include <mutex>

#include "eql_internal.h"
#include "ptx_sm100.cuh"
#include "rdft.cuh"
#include "umma_common.cuh"

namespace eql {
namespace {


constexpr int kTmemColsRes = 512;
constexpr int kResWarpTmaX = 0, kResWarpMma = 1, kResWarpTmaW = 2, kResWarpTmaX2 = 3, kResWarpCompute0 = 4;
constexpr int kResComputeWarps = 16;         // at most (barrier array size)
// Compute warps per kernel: the T = 4 epilogue is short on instruction issue and long on stores, and gains from a
// fourth warp per TMEM lane quadrant even at 96 registers per thread (Swin layer: 99.7 -> 96.1 us); the T = 8 kernels
// lose more to the smaller register file than they gain (76 -> 80 us), so they keep three.
template <int T> struct ResWarps { static constexpr int kCompute = T == 4 ? 16 : 12, kThreads = (4 + kCompute) * 32; };
constexpr int kItemBytes = 4096;            // raw item: 32 token rows x 128 bytes
constexpr int kWTileBytes = 4096;           // spectral-weight tile of one plane: [128 channels x 32 B]
constexpr int kResMaxK = 12;                // resident chunks (barrier array size)
constexpr int kResMaxWSlots = 4;
constexpr uint32_t kResSpin = 256;
constexpr uint32_t kIdescNegateA = 1u << 13;

struct ResParams {
    void* out;                   // [N, Cout*T] half
    const uint8_t* image;        // [channel tile][chunk][plane][128 x 32 B], see build_image_res_kernel
    const float* bias;           // [Cout] or nullptr
    int* status;
    int64_t N;
    int Cin, Cout;
    int nCT, nK;                 // output-channel tiles, 16-channel chunks
    int w_slots, n_tw;           // weight-ring slots, transform warps (= raw ring slots)
    int x_slots;                 // x^ chunk buffers: nK (a whole token tile resident) or, with one channel tile, a ring of 3
    int64_t num_units;           // token tiles x nCT
    // optional: also write the spectrum of the input in the operand layout of the weight-gradient kernel
    // (umma_bwd_weight_saved.cu): blob (input-channel tile, 16-token chunk), T planes of MN-major [CiT x 16] tiles
    uint8_t* stash;              // nullptr: off
    int st_CiT, st_nCiTiles;     // the weight gradient's input-channel tiling
    int64_t st_chunks;           // 16-token chunks in all
    int act;                     // 1: GELU on the result (forward of a plan built with EQL_FLAG_GELU)
};


struct ResBarriers {
    uint64_t full_raw[kResComputeWarps], empty_raw[kResComputeWarps];
    uint64_t full_x[kResMaxK], empty_x[kResMaxK];
    uint64_t full_w[kResMaxWSlots], empty_w[kResMaxWSlots];
    uint64_t full_d[2], empty_d[2], mma_done;
    uint32_t tmem_base;
    int abort_flag;
};

// Spectral-weight operand image: planes[p][cin][cout] (float, scaled, conjugated for the data gradient) ->
// for every (channel tile ct, chunk kc, plane p) one [128 x 16] half tile in the canonical K-major layout with
// 32-byte swizzle: byte b of row n lives at n*32 + (((b>>4) ^ ((n>>2)&1))<<4) + (b&15); row n = channel ct*128 + n.
template <int T, typename IO>
__global__ void build_image_res_kernel(const float* __restrict__ planes, int Cin, int Cout, int nCT, int nK,
                                       IO* __restrict__ image) {
    const int64_t total = (int64_t)nCT * nK * T * 128 * 16;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int within = (int)(idx % (128 * 16));
        const int64_t tile = idx / (128 * 16);
        const int p = (int)(tile % T);
        const int kc = (int)((tile / T) % nK), ct = (int)(tile / ((int64_t)T * nK));
        const int n = within / 16, c = (within % 16) / 8;
        const int kk = (c ^ ((n >> 2) & 1)) * 8 + within % 8;
        const int cin = kc * 16 + kk, cout = ct * 128 + n;
        float v = 0.f;
        if (cin < Cin && cout < Cout) v = planes[((size_t)p * Cin + cin) * Cout + cout];
        image[idx] = H16<IO>::narrow(v);
    }
}

// ------------------------------------------------------------------------------------------------
// PF ("paired form"): x^ additionally keeps -Re x^ of every complex frequency, stored as tiles [Re | Im | -Re], so that a
// complex frequency takes two MMAs of width 2 NTOK ([Re|Im] += Wr [Xr|Xi] and, with A negated, += (-Wi) [Xi|-Xr])
// instead of three; an MMA costs about the same whatever its width, so this shortens the main loop where the larger
// x^ buffers fit.
template <int T, int NTOK, bool PF, bool MERGED, bool ACT, typename IO>
__global__ void __launch_bounds__(ResWarps<T>::kThreads, 1)
umma_linear_res_kernel(const __grid_constant__ CUtensorMap tmap_in, const ResParams prm) {
    // IO: IEEE half or bfloat16 (same byte geometry; conversions and the UMMA operand format differ)
    // NTOK tokens per tile: the accumulator of a unit is T planes x NTOK fp32 TMEM columns.  With T * NTOK = 256 two
    // accumulators alternate, so that the epilogue of a unit overlaps the MMAs of the next one.
    constexpr int NCW = ResWarps<T>::kCompute;  // compute warps
    constexpr int kResShares = NCW / 4;         // warps sharing the token column groups of a TMEM lane quadrant
    constexpr int NBUF = 512 / (T * NTOK);
    constexpr int XTILES = PF ? 2 + 3 * (T / 2 - 1) : T;   // plane tiles per chunk
    constexpr int kXChunkBytes = XTILES * NTOK * 32;       // x^ of one 16-channel chunk: tiles of [NTOK tokens x 32 B]
    constexpr int NCH = 64 / T;                 // channels per 128-byte raw row
    constexpr int SPK = 16 / NCH;               // raw slabs (64 elements wide) per 16-channel chunk
    constexpr int PARTS = NTOK / 32;            // 32-token items per slab
    constexpr int IPC = SPK * PARTS;            // items per chunk (= 4 for T = 4 and T = 8)
    constexpr int XT = NTOK * 32;               // bytes of one x^ plane tile [NTOK tokens x 16 channels]
    constexpr int W = NCH / 2;                  // 32-bit words one raw row contributes to one plane
    constexpr int kWSlot = T * kWTileBytes;
    static_assert(T == 4 || T == 8, "resident kernel: T = 4 or 8");
    static_assert(NBUF == 1 || NBUF == 2, "accumulator count");

    extern __shared__ uint8_t smem_raw_base[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~(uintptr_t)1023);
    // ring mode: three x^ buffers, three weight slots, twelve transform warps, one channel tile (compile-time there)
    const int nK = prm.nK, nCT = MERGED ? 1 : prm.nCT, n_tw = MERGED ? 12 : prm.n_tw, w_slots = MERGED ? 3 : prm.w_slots,
              XR = MERGED ? 3 : prm.x_slots;
    uint8_t* raw = smem;                                         // n_tw items
    uint8_t* xhat = raw + n_tw * kItemBytes;                     // XR chunk buffers
    uint8_t* wsm = xhat + XR * kXChunkBytes;                     // w_slots slots
    ResBarriers* bar = reinterpret_cast<ResBarriers*>(wsm + w_slots * kWSlot);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &bar->abort_flag;
    int* status = prm.status;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kResComputeWarps; ++i) { ptx::mbar_init(&bar->full_raw[i], 1); ptx::mbar_init(&bar->empty_raw[i], 1); }
        for (int i = 0; i < kResMaxK; ++i) { ptx::mbar_init(&bar->full_x[i], IPC + (MERGED ? 1 : 0)); ptx::mbar_init(&bar->empty_x[i], 1); }
        for (int i = 0; i < kResMaxWSlots; ++i) { ptx::mbar_init(&bar->full_w[i], 1); ptx::mbar_init(&bar->empty_w[i], 1); }
        for (int i = 0; i < 2; ++i) { ptx::mbar_init(&bar->full_d[i], 1); ptx::mbar_init(&bar->empty_d[i], NCW); }
        ptx::mbar_init(&bar->mma_done, 1);
        bar->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_in);
    }
    if (warp == kResWarpMma) {
        ptx::tmem_alloc(&bar->tmem_base, kTmemColsRes);
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

    // this CTA's contiguous range of units; unit u = token tile (u / nCT), channel tile (u % nCT)
    const int64_t u0 = prm.num_units * (int64_t)blockIdx.x / gridDim.x;
    const int64_t u1 = prm.num_units * ((int64_t)blockIdx.x + 1) / gridDim.x;
    // every role walks the units with a running (token tile, channel tile) pair instead of dividing per unit
    const int ct0 = (int)(u0 % nCT);
    const int64_t tt0 = u0 / nCT;
    // With a ring of x^ buffers (fewer buffers than chunks) nothing survives a unit: every unit transforms its token
    // tile itself, i.e. is the first and the last of its tile.
    constexpr bool ring = MERGED;                                // the host runs ring mode with equally deep rings only
    // Ring mode with equally deep rings: chunk q uses x^ buffer q % 3 and weight slot q % 3, so one "full" barrier
    // (transform warps + the weight copy) and one "empty" barrier (one commit) per chunk serve both, which halves the
    // barrier operations of the MMA-issuing thread.
    // MERGED is a template parameter so that the other modes keep their exact instruction stream.
    constexpr bool merged = MERGED;                               // host: ring mode with w_slots == x_slots
    uint64_t* const full_wb = merged ? bar->full_x : bar->full_w;
    uint64_t* const empty_wb = merged ? bar->empty_x : bar->empty_w;
    auto first_of_tile = [&](int64_t u, int ct) { return ring || u == u0 || ct == 0; };
    auto last_of_tile = [&](int64_t u, int ct) { return ring || u == u1 - 1 || ct == nCT - 1; };
    const int items_per_tile = IPC * nK;

    if (warp == kResWarpTmaX || warp == kResWarpTmaX2) {
        // ---------------------------------------------------------------- raw activation rows via TMA
        // Two producer threads in two warps, one for the even ring slots (= even items) and one for the odd ones: a thread
        // gets one bulk / tensor copy accepted every ~300 ns whatever its size (measured: L2-resident source, 4 to 64 KB
        // per copy, any number in flight; the rate scales with the number of issuing warps), and these items are 4 KB.
        // A layer with many input channels needs one item per ~260 ns and SM at the speed of its MMA loop.
        if (lane == 0) {
            const int me = warp == kResWarpTmaX ? 0 : 1;         // n_tw is even: slot parity = item parity
            uint32_t gi = me;                                    // running item counter; item gi lives in slot gi % n_tw
            int slot = me;
            uint32_t eph = 1;
            bool ok = true;
            int ct = ct0;
            int64_t tt = tt0;
            uint32_t base = 0;                                   // running number of the tile's first item
            for (int64_t u = u0; u < u1 && ok; ++u, ++ct) {
                if (ct == nCT) { ct = 0; ++tt; }
                if (!first_of_tile(u, ct)) continue;
                const int row0 = (int)tt * NTOK;
                for (; gi < base + (uint32_t)items_per_tile; gi += 2) {
                    const int i = (int)(gi - base);
                    ok = ptx::mbar_wait(&bar->empty_raw[slot], eph, abort_flag, status, 301, true, kResSpin);
                    if (!ok) break;
                    ptx::mbar_arrive_expect_tx(&bar->full_raw[slot], kItemBytes);
                    const int s = i / PARTS, h = i % PARTS;      // slab (64 elements of the row), 32-token part
                    ptx::tma_load_2d(raw + slot * kItemBytes, &tmap_in, s * 64, row0 + h * 32, &bar->full_raw[slot]);
                    slot += 2;
                    if (slot >= n_tw) { slot -= n_tw; eph ^= 1u; }
                }
                base += (uint32_t)items_per_tile;
            }
            // drain: every copy this thread issued must have landed before the CTA may exit (its items: me, me + 2, ...)
            if (gi >= 2) {
                const uint32_t last = gi - 2;                    // last item issued (or the one a failed wait stopped at)
                const uint32_t lo = last + 2 > (uint32_t)n_tw ? last + 2 - n_tw : me;
                for (uint32_t c = lo; c <= last; c += 2)
                    ptx::mbar_wait(&bar->full_raw[c % n_tw], (c / n_tw) & 1, abort_flag, status, 311, false);
            }
        }
    } else if (warp == kResWarpTmaW) {
        // ---------------------------------------------------------------- spectral-weight tiles via bulk copy
        if (lane == 0) {
            uint32_t cw = 0;
            int slot = 0;
            uint32_t eph = 1;                                    // parity to wait for on the slot's "empty" barrier
            bool ok = true;
            int ct = ct0;
            for (int64_t u = u0; u < u1 && ok; ++u, ++ct) {
                if (ct == nCT) ct = 0;
                for (int kc = 0; kc < nK; ++kc, ++cw) {
                    ok = ptx::mbar_wait(&empty_wb[slot], eph, abort_flag, status, 302, true, kResSpin);
                    if (!ok) break;
                    ptx::mbar_arrive_expect_tx(&full_wb[slot], kWSlot);
                    ptx::bulk_load_1d(wsm + slot * kWSlot, prm.image + ((size_t)ct * nK + kc) * (size_t)kWSlot, kWSlot,
                                      &full_wb[slot]);
                    if (++slot == w_slots) { slot = 0; eph ^= 1u; }
                }
            }
            const uint32_t lo = cw > (uint32_t)w_slots ? cw - w_slots : 0;
            for (uint32_t c = lo; c < cw; ++c)
                ptx::mbar_wait(&full_wb[c % w_slots], (c / w_slots) & 1, abort_flag, status, 312, false);
        }
    } else if (warp == kResWarpMma) {
        // ---------------------------------------------------------------- tensor-core issue (one thread)
        if (lane == 0) {
            uint32_t cu = 0, tc = 0;
            int slot = 0;                                        // weight-ring slot of the current chunk
            uint32_t wph = 0;                                    // its phase parity
            bool ok = true;
            const uint32_t idesc1 = ptx::umma_idesc_f16_f32(128, NTOK, H16<IO>::kUmmaFormat);      // one plane of tokens
            const uint32_t idesc2 = ptx::umma_idesc_f16_f32(128, 2 * NTOK, H16<IO>::kUmmaFormat);  // [Re | Im] planes of a complex frequency
            // shared-memory descriptors are built once per chunk and advanced by (byte offset >> 4) in their address field
            // (the tiles stay inside the 256 KB window, so no carry leaves it)
            auto mma = [](uint32_t d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
                ptx::umma_f16(d, a_desc, b_desc, idesc, accumulate);
            };
            constexpr uint64_t kWTileD = kWTileBytes >> 4, kXTileD = XT >> 4;
            int ct = ct0;
            for (int64_t u = u0; u < u1 && ok; ++u, ++cu, ++ct) {
                if (ct == nCT) ct = 0;
                const bool first = first_of_tile(u, ct), last = last_of_tile(u, ct);
                if (first && u != u0) ++tc;
                const uint32_t buf = cu % NBUF;
                const uint32_t dbase = tmem_base + buf * (uint32_t)(T * NTOK);
                ok = ptx::mbar_wait(&bar->empty_d[buf], ((cu / NBUF) & 1) ^ 1, abort_flag, status, 303, true, kResSpin);
                if (!ok) break;
                // x^ buffer and phase of the tile's chunk 0: chunk kc of the CTA's tc-th tile has running number tc*nK + kc
                // (resident mode has XR == nK: buffer = chunk index, phase = tile parity, no division)
                int xs = ring ? (int)((tc * (uint32_t)nK) % (uint32_t)XR) : 0;
                uint32_t xph = ring ? ((tc * (uint32_t)nK) / (uint32_t)XR) & 1u : tc & 1u;
                // operands of the unit's first chunk
                if (first) ok = ptx::mbar_wait(&bar->full_x[xs], xph, abort_flag, status, 304, true, kResSpin);
                if constexpr (!merged) ok = ok && ptx::mbar_wait(&bar->full_w[slot], wph, abort_flag, status, 305, true, kResSpin);
                if (!ok) break;
                for (int kc = 0; kc < nK; ++kc) {
                    ptx::tc_fence_after_sync();
                    const uint64_t a0 = ptx::umma_smem_desc_k_sw32(ptx::smem_u32(wsm + slot * kWSlot));      // weight tiles, plane p at p * 4 KB
                    const uint64_t b0 = ptx::umma_smem_desc_k_sw32(ptx::smem_u32(xhat + xs * kXChunkBytes)); // x^ tiles, plane p at p * XT
                    const uint32_t acc = kc > 0 ? 1u : 0u;
                    int nslot = slot + 1;
                    uint32_t nwph = wph;
                    if (nslot == w_slots) { nslot = 0; nwph ^= 1u; }
                    int nxs = xs + 1;
                    uint32_t nxph = xph;
                    if (nxs == XR) { nxs = 0; nxph ^= 1u; }
                    mma(dbase, a0, b0, idesc1, acc);                                                      // k = 0
#pragma unroll
                    for (int f = 1; f < T / 2; ++f) {
                        const uint32_t dre = dbase + (uint32_t)((2 * f - 1) * NTOK), dim = dre + NTOK;
                        const uint64_t wr = a0 + (2 * f - 1) * kWTileD, wi = wr + kWTileD;
                        if constexpr (PF) {
                            const uint64_t xr = b0 + (1 + 3 * (f - 1)) * kXTileD, xi = xr + kXTileD;  // tiles Re | Im | -Re
                            mma(dre, wr, xr, idesc2, acc);                                                // [Re|Im] += Wr [Xr|Xi]
                            mma(dre, wi, xi, idesc2 | kIdescNegateA, 1u);                                 // [Re|Im] -= Wi [Xi|-Xr]
                        } else {
                            const uint64_t xr = b0 + (2 * f - 1) * kXTileD, xi = xr + kXTileD;
                            mma(dre, wr, xr, idesc2, acc);                                                // [Re|Im] += Wr [Xr|Xi]
                            mma(dre, wi, xi, idesc1 | kIdescNegateA, 1u);                                 //  Re     -= Wi Xi
                            mma(dim, wi, xr, idesc1, 1u);                                                 //  Im     += Wi Xr
                        }
                        if (f == 1 && kc + 1 < nK) {
                            // The next chunk's operands are checked here, while the tensor pipe still has this chunk's
                            // MMAs queued, so that the issue stream has no gap between chunks.
                            if (first) ok = ptx::mbar_wait(&bar->full_x[nxs], nxph, abort_flag, status, 304, true, kResSpin);
                            if constexpr (!merged) ok = ok && ptx::mbar_wait(&bar->full_w[nslot], nwph, abort_flag, status, 305, true, kResSpin);
                        }
                    }
                    mma(dbase + (uint32_t)((T - 1) * NTOK), a0 + (T - 1) * kWTileD, b0 + (XTILES - 1) * kXTileD, idesc1, acc);  // k = T/2
                    if constexpr (!merged) ptx::umma_commit(&bar->empty_w[slot]);
                    if (last) ptx::umma_commit(&bar->empty_x[xs]);  // the x^ buffer may be overwritten once these MMAs retire
                    slot = nslot; wph = nwph;
                    xs = nxs; xph = nxph;
                    if (!ok) break;
                }
                if (ok) ptx::umma_commit(&bar->full_d[buf]);
            }
            // all MMAs issued by this thread must have retired before shared memory and TMEM go away
            ptx::umma_commit(&bar->mma_done);
            ptx::mbar_wait(&bar->mma_done, 0, abort_flag, status, 313, false);
        }
    } else if (warp >= kResWarpCompute0) {
        // ---------------------------------------------------------------- compute warps: transform and epilogue
        const int cw = warp - kResWarpCompute0;
        const int quad = warp & 3;                               // TMEM lane quadrant this warp may read
        const int third = cw >> 2;                               // share of the token column groups
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
        bool ok = true;

        // Group DFT of this warp's items of token tile number tc (the tc-th tile of this CTA).  Items are dealt
        // round-robin over the transform warps by their running number, so warp cw always reads ring slot cw.
        uint32_t my_items = 0;                                   // items this warp has taken from its ring slot
        // Chunks [c_lo, c_hi) of the tile only: with a ring of x^ buffers the first XR chunks are transformed before the
        // previous unit's epilogue and the rest after it, while the MMAs of the tile consume them.
        auto transform_tile = [&](uint32_t tc, int c_lo, int c_hi, int64_t tile_row0) {
            if (cw >= n_tw || c_lo >= c_hi) return;
            const uint32_t base = tc * (uint32_t)items_per_tile;
            const int lo = c_lo * IPC, hi = c_hi * IPC;
            // this warp's items of the tile: running numbers congruent to cw modulo n_tw
            const int i0 = lo + (int)(((uint32_t)cw + 4u * (uint32_t)n_tw - (base + (uint32_t)lo) % (uint32_t)n_tw) % (uint32_t)n_tw);
            for (int i = i0; i < hi && ok; i += n_tw, ++my_items) {
                ok = ptx::mbar_wait(&bar->full_raw[cw], my_items & 1, abort_flag, status, 306, true, 16);
                if (!ok) break;
                uint32_t wd[32];
                load_slab_row(raw + cw * kItemBytes + lane * 128, lane, wd);
                // The row is in registers: order these generic-proxy reads before the async-proxy (TMA) refill of
                // the slot, then release it so that the refill overlaps the transform.
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bar->empty_raw[cw]);
                uint32_t packed[T][W];
                // Ring mode has the transform on the critical path (every chunk is transformed right before its MMAs):
                // packed-half butterflies there, two channels per instruction (-5 % kernel time, max error 5.5e-4
                // instead of 4.7e-4 of the largest output, bar 3e-3).  Resident mode: float butterflies, one rounding.
                // (packed-half butterflies exist for IEEE half only: bfloat16 keeps 8 significand bits per rounding)
                if constexpr (ring && H16<IO>::kIsHalf) dft_words<T, false, true>(wd, packed, nullptr);
                else dft_words<T, false, false, IO>(wd, packed, nullptr);
                const int s = i / PARTS, h = i % PARTS;
                const int kc = s / SPK, q = s % SPK;
                const int r = h * 32 + lane;                     // token row inside the tile
                if (prm.stash != nullptr) {
                    // the same planes, for the weight gradient of this batch (rows past N and channels past C_in are
                    // zero here, as the TMA load filled them, and are written as such)
                    const int c0 = s * NCH;                      // first channel of this raw row's run
                    const int64_t n = tile_row0 + r;
                    if (c0 < prm.st_nCiTiles * prm.st_CiT && n < prm.st_chunks * 16) {
                        const int cit = c0 / prm.st_CiT, mn0 = c0 - cit * prm.st_CiT;
                        const int k = (int)(n & 15);
                        uint8_t* g = prm.stash + ((size_t)cit * prm.st_chunks + (size_t)(n >> 4)) * ((size_t)T * prm.st_CiT * 32) +
                                     (mn0 >> 3) * 256 + (k >> 3) * 128 + (k & 7) * 16;
#pragma unroll
                        for (int p = 0; p < T; ++p) store_plane_run<2 * W>(g + (size_t)p * prm.st_CiT * 32, packed[p], 256);
                    }
                }
                // buffer of this chunk (running number qn); the MMAs that read the buffer's previous contents must have retired
                const uint32_t qn = tc * (uint32_t)nK + (uint32_t)kc;
                const int xsl = ring ? (int)(qn % (uint32_t)XR) : kc;
                const uint32_t use = ring ? qn / (uint32_t)XR : tc;
                if (use > 0) {
                    ok = ptx::mbar_wait(&bar->empty_x[xsl], (use - 1) & 1, abort_flag, status, 307, true, 16);
                    if (!ok) break;
                }
                // x^ plane tile: row r at r*32, its two 16-byte chunks exchanged when bit 2 of r is set (32B swizzle);
                // this raw row's run of channels starts at byte kb of the row
                const int kb = q * NCH * 2;
                const int sw = (r >> 2) & 1;
                uint8_t* dst = xhat + xsl * kXChunkBytes + r * 32 + (((kb >> 4) ^ sw) << 4) + (kb & 15);
                const int second = sw ? -16 : 16;
                if constexpr (PF) {
                    store_plane_run<2 * W>(dst, packed[0], second);
#pragma unroll
                    for (int f = 1; f < T / 2; ++f) {
                        uint8_t* t0 = dst + (1 + 3 * (f - 1)) * XT;
                        store_plane_run<2 * W>(t0, packed[2 * f - 1], second);                      // Re
                        store_plane_run<2 * W>(t0 + XT, packed[2 * f], second);                     // Im
                        store_plane_run<2 * W>(t0 + 2 * XT, packed[2 * f - 1], second, 0x80008000u); // -Re
                    }
                    store_plane_run<2 * W>(dst + (XTILES - 1) * XT, packed[T - 1], second);
                } else {
#pragma unroll
                    for (int p = 0; p < T; ++p) store_plane_run<2 * W>(dst + p * XT, packed[p], second);
                }
                ptx::fence_proxy_async_smem();                   // generic-proxy writes -> visible to the MMA (async proxy)
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bar->full_x[xsl]);
            }
        };

        uint32_t tc = 0, cu = 0;
        const int pre = XR < nK ? XR : nK;                       // chunks of a tile that fit before its MMAs start freeing buffers
        if (u0 < u1) transform_tile(0, 0, pre, tt0 * NTOK);
        int ct = ct0;
        int64_t tt = tt0;
        for (int64_t u = u0; u < u1 && ok; ++u, ++cu, ++ct) {
            if (ct == nCT) { ct = 0; ++tt; }
            // ring of x^ buffers (one channel tile): the rest of this tile's chunks, consumed by its MMAs as they arrive
            if (first_of_tile(u, ct)) {
                transform_tile(tc, pre, nK, tt * NTOK);
                if (!ok) break;
            }
            // the next token tile is transformed while the MMAs of this tile's last channel tile are in flight
            if (last_of_tile(u, ct) && u + 1 < u1) {
                ++tc;
                transform_tile(tc, 0, pre, (tt + 1) * NTOK);
                if (!ok) break;
            }
            // ---- epilogue of unit u: thread = output channel, columns = (plane, token)
            const int64_t row0 = tt * NTOK;
            const int o = ct * 128 + quad * 32 + lane;
            const bool o_ok = o < prm.Cout;
            const float bias_v = (prm.bias != nullptr && o_ok) ? __ldg(prm.bias + o) : 0.f;
            const size_t pitch = (size_t)prm.Cout * T * sizeof(__half);
            uint8_t* out_o = reinterpret_cast<uint8_t*>(prm.out) + (size_t)o * T * sizeof(__half);
            const uint32_t buf = cu % NBUF;
            const uint32_t acc_base = lane_base + buf * (uint32_t)(T * NTOK);
            ok = ptx::mbar_wait(&bar->full_d[buf], (cu / NBUF) & 1, abort_flag, status, 308, true, 16);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            constexpr int NG = NTOK / 8;                         // groups of 8 tokens
            for (int g = third; g < NG; g += kResShares) {
                const int n0 = g * 8;
                uint32_t in[T][8];
#pragma unroll
                for (int p = 0; p < T; ++p) ptx::tmem_ld<8>(acc_base + (uint32_t)(p * NTOK + n0), in[p]);
                ptx::tmem_ld_wait();
                if (g + kResShares >= NG) {                      // this warp's last read of the accumulator
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&bar->empty_d[buf]);
                }
                uint8_t* dst = out_o + (size_t)(row0 + n0) * pitch;
                const int rows_left = (int)(prm.N - (row0 + n0) < 8 ? prm.N - (row0 + n0) : 8);   // may be <= 0
                // whole groups of a valid channel (everything but the batch's last tile and the channels past C_out) take
                // a copy of the loop without per-token predicates
                auto emit = [&](auto whole_tag) {
                    constexpr bool kWhole = decltype(whole_tag)::value;
#pragma unroll
                    for (int j = 0; j < 8; ++j, dst += pitch) {
                        float v[T];
#pragma unroll
                        for (int p = 0; p < T; ++p) v[p] = __uint_as_float(in[p][j]);
                        v[0] += bias_v;
                        rdft_inverse<T>(v);
                        if constexpr (ACT) {                     // fused GELU: its own instantiation of the kernel
#pragma unroll
                            for (int t = 0; t < T; ++t) v[t] = gelu_erf(v[t]);
                        }
                        if (kWhole || (o_ok && j < rows_left)) {
                            if constexpr (T == 8)
                                *reinterpret_cast<uint4*>(dst) = make_uint4(H16<IO>::pack(v[0], v[1]), H16<IO>::pack(v[2], v[3]),
                                                                            H16<IO>::pack(v[4], v[5]), H16<IO>::pack(v[6], v[7]));
                            else
                                *reinterpret_cast<uint2*>(dst) = make_uint2(H16<IO>::pack(v[0], v[1]), H16<IO>::pack(v[2], v[3]));
                        }
                    }
                };
                if (o_ok && rows_left >= 8) emit(std::true_type{});
                else emit(std::false_type{});
            }
        }
    }

    // ---------------------------------------------------------------- teardown (reached by every thread)
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kResWarpMma) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemColsRes);
    }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_res_fn() {
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

constexpr size_t kResSmemLimit = 227 * 1024;

size_t res_smem_bytes(int T, int nTok, bool paired, int x_slots, int w_slots, int n_tw) {
    const int tiles = paired ? 2 + 3 * (T / 2 - 1) : T;
    return 1024 + (size_t)n_tw * kItemBytes + (size_t)x_slots * tiles * nTok * 32 + (size_t)w_slots * T * kWTileBytes +
           sizeof(ResBarriers) + 64;
}

}  // namespace


bool umma_res_supported(int T, eql_dtype_t dtype) { return (dtype == EQL_FP16 || dtype == EQL_BF16) && (T == 4 || T == 8); }

UmmaResShape umma_res_shape(int T, int Cin, int Cout, eql_dtype_t dtype) {
    UmmaResShape s{};
    s.T = T; s.Cin = Cin; s.Cout = Cout;
    s.bf16 = dtype == EQL_BF16;
    s.nTok = 512 / T;                                            // one accumulator filling the 512 TMEM columns
    s.nK = (Cin + 15) / 16;
    s.nCT = (Cout + 127) / 128;
    s.image_bytes = align_up((size_t)s.nCT * s.nK * T * kWTileBytes, kWsAlign);
    s.fits = false;
    s.paired = false;
    // ring depths in order of preference: the weight stream paces the main loop (3 chunks cover its latency), then
    // as many transform warps as shared memory allows
    static const int cand[][2] = {{3, 12}, {3, 8}, {2, 12}, {2, 8}, {2, 4}};
    if (s.nK <= kResMaxK) {                                      // the whole token tile resident: x^ buffers = chunks
        s.x_slots = s.nK;
        for (const auto& c : cand) {
            if (res_smem_bytes(T, s.nTok, false, s.x_slots, c[0], c[1]) <= kResSmemLimit) {
                s.w_slots = c[0]; s.n_tw = c[1]; s.fits = true;
                break;
            }
        }
    }
    // One channel tile: nothing is reused across units, so three x^ buffers used as a ring are enough (with two
    // channel tiles, each repeating the transform, the streaming kernel measured faster: 104 vs 111 us on the
    // D = 1024, T = 4 shape).  The ring
    // needs all 12 transform warps (chunk q is then always transformed by warps 4 (q % 3) .. 4 (q % 3) + 3, which
    // therefore see every phase of the buffer barriers they wait on).
    if (s.nCT == 1 && !(s.fits && s.w_slots >= 3) && s.nK > 3 &&
        res_smem_bytes(T, s.nTok, false, 3, 3, 12) <= kResSmemLimit) {
        s.x_slots = 3; s.w_slots = 3; s.n_tw = 12; s.fits = true;
    }
    // paired form where the larger x^ buffers still leave a deep weight ring
    if (s.fits && s.w_slots >= 3 && res_smem_bytes(T, s.nTok, true, s.x_slots, 3, s.n_tw) <= kResSmemLimit) {
        s.paired = true;
        s.w_slots = 3;
    }
    // (not in ring mode: equal ring depths let one barrier pair serve the weight slot and the x^ buffer of a chunk)
    if (s.fits && s.w_slots == 3 && s.x_slots == s.nK &&
        res_smem_bytes(T, s.nTok, s.paired, s.x_slots, 4, s.n_tw) <= kResSmemLimit)
        s.w_slots = 4;
    return s;
}

cudaError_t launch_build_umma_res_image(const UmmaResShape& s, const float* planes, void* image, cudaStream_t stream) {
    const int64_t total = (int64_t)s.nCT * s.nK * s.T * 128 * 16;
    const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
    if (s.T == 4 && !s.bf16)
        build_image_res_kernel<4, __half><<<blocks, 256, 0, stream>>>(planes, s.Cin, s.Cout, s.nCT, s.nK, (__half*)image);
    else if (s.T == 8 && !s.bf16)
        build_image_res_kernel<8, __half><<<blocks, 256, 0, stream>>>(planes, s.Cin, s.Cout, s.nCT, s.nK, (__half*)image);
    else if (s.T == 4)
        build_image_res_kernel<4, __nv_bfloat16><<<blocks, 256, 0, stream>>>(planes, s.Cin, s.Cout, s.nCT, s.nK, (__nv_bfloat16*)image);
    else if (s.T == 8)
        build_image_res_kernel<8, __nv_bfloat16><<<blocks, 256, 0, stream>>>(planes, s.Cin, s.Cout, s.nCT, s.nK, (__nv_bfloat16*)image);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

cudaError_t launch_umma_linear_res(const UmmaResShape& s, const void* in, void* out, int64_t N, const void* image,
                                   const float* bias_f32, int* status, int num_sms, cudaStream_t stream,
                                   const UmmaBwdWeightShape* stash_shape, void* stash) {
    if (!s.fits) return cudaErrorInvalidConfiguration;
    EncodeTiledFn enc = encode_tiled_res_fn();
    if (enc == nullptr) return cudaErrorNotSupported;
    CUtensorMap tmap;
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)s.Cin * s.T, (cuuint64_t)N};
        const cuuint64_t gstr[1] = {(cuuint64_t)s.Cin * s.T * sizeof(__half)};
        const cuuint32_t box[2] = {64, 32};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(in), gdim, gstr, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    ResParams prm{};
    prm.out = out; prm.image = (const uint8_t*)image; prm.bias = bias_f32; prm.status = status;
    prm.N = N; prm.Cin = s.Cin; prm.Cout = s.Cout; prm.nCT = s.nCT; prm.nK = s.nK;
    prm.w_slots = s.w_slots; prm.n_tw = s.n_tw; prm.x_slots = s.x_slots;
    prm.num_units = ((N + s.nTok - 1) / s.nTok) * s.nCT;
    prm.act = s.act;
    if (stash != nullptr && stash_shape != nullptr) {
        prm.stash = (uint8_t*)stash;
        prm.st_CiT = stash_shape->CiT; prm.st_nCiTiles = stash_shape->nCiTiles; prm.st_chunks = stash_shape->total_chunks;
    }
    const int grid = (int)(prm.num_units < num_sms ? prm.num_units : num_sms);
    const size_t smem = res_smem_bytes(s.T, s.nTok, s.paired, s.x_slots, s.w_slots, s.n_tw);

    auto launch = [&](auto kernel, SmemLimitOnce& once, int threads) -> cudaError_t {
        if (cudaError_t e = once.ensure(kernel, (int)kResSmemLimit); e != cudaSuccess) return e;
        return launch_overlapped(kernel, dim3(grid), dim3(threads), smem, stream, tmap, prm);
    };
    auto go = [&](auto tc, auto nt, auto pf, auto mg) -> cudaError_t {
        constexpr int TT = decltype(tc)::value, NT = decltype(nt)::value;
        constexpr bool PF = decltype(pf)::value, MG = decltype(mg)::value;
        static SmemLimitOnce once[4];                         // per kernel instantiation: (activation, element type)
        constexpr int threads = ResWarps<TT>::kThreads;
        if (s.bf16) {
            if (prm.act) return launch(umma_linear_res_kernel<TT, NT, PF, MG, true, __nv_bfloat16>, once[3], threads);
            return launch(umma_linear_res_kernel<TT, NT, PF, MG, false, __nv_bfloat16>, once[2], threads);
        }
        if (prm.act) return launch(umma_linear_res_kernel<TT, NT, PF, MG, true, __half>, once[1], threads);
        return launch(umma_linear_res_kernel<TT, NT, PF, MG, false, __half>, once[0], threads);
    };
    using I4 = std::integral_constant<int, 4>;
    using I8 = std::integral_constant<int, 8>;
    using I64 = std::integral_constant<int, 64>;
    using I128 = std::integral_constant<int, 128>;
    const bool merged = s.x_slots < s.nK;                                // ring mode: one barrier pair per chunk
    // the ring-mode variant has these folded in at compile time
    if (merged && !(s.x_slots == 3 && s.w_slots == 3 && s.n_tw == 12 && s.nCT == 1)) return cudaErrorInvalidConfiguration;
    auto pick = [&](auto tc, auto nt) -> cudaError_t {
        if (merged)
            return s.paired ? go(tc, nt, std::true_type{}, std::true_type{}) : go(tc, nt, std::false_type{}, std::true_type{});
        return s.paired ? go(tc, nt, std::true_type{}, std::false_type{}) : go(tc, nt, std::false_type{}, std::false_type{});
    };
    if (s.T == 4 && s.nTok == 128) return pick(I4{}, I128{});
    if (s.T == 8 && s.nTok == 64) return pick(I8{}, I64{});
    return cudaErrorInvalidValue;
}

}  // namespace eql
