// Fused EQ-Linear forward / data-gradient on the 5th-generation tensor cores (tcgen05 + TMEM): 16-bit I/O (IEEE half or
// bfloat16, kind::f16) or float I/O (kind::tf32 with the 3xTF32 split), FP32 accumulation.  One persistent CTA per SM;
// a work unit is (128-token tile, output-channel tile).
//
//   TMA (2-D, 128B swizzle)      raw rows of x            -> shared "slabs" [128 rows x 128 B]
//   12 compute warps, phase 1    group DFT (Eq. 4) in registers, planes rounded to the operand type once
//                                -> shared A operands, one [128 x 16] K-major tile per real-packed plane
//   TMA (1-D bulk)               spectral-weight image of this (tile, 16-channel chunk) -> shared B operands
//   1 thread                     tcgen05.mma kind::f16: one product per real frequency, and the complex
//                                product of Eq. 5 as the real 2x2 block [Xr|Xi] x [[Wr,Wi],[-Wi,Wr]] -> TMEM
//   12 compute warps, phase 2    tcgen05.ld, bias on plane k = 0, inverse DFT (Eq. 7) in registers, one rounding,
//                                [32 tokens x 128 B] staged in shared memory (the idle A-operand stages) and written
//                                with asynchronous, fully coalesced TMA tensor stores
//
// Frequency-domain data never leaves the SM (registers, shared memory, TMEM).  The data gradient is the
// same kernel run on dy with the conjugate-transposed weight image and no bias.
//
// CG = 2 ("CTA pair"; plans of wide layers, or EQL_FLAG_CTA_PAIR): the same kernel as a cluster of two CTAs on two SMs
// that work on two neighbouring token tiles and the same output-channel tile in lockstep.  One
// tcgen05.mma.cta_group::2 (M = 256) issued by the pair's leader covers both token tiles; its B operand -- the
// spectral weight tile -- is split in halves between the two CTAs, so each SM loads and holds only half of every
// weight tile (the L2 -> SM traffic of the weights halves).  Each CTA issues its own loads into its own shared memory;
// only mbarrier arrivals cross the pair: the peer's word that its stage of a chunk is full (one remote arrive per
// stage on the leader's barrier of that stage), the leader's commits to the peer's "empty" and "accumulator full"
// barriers (a second commit each, addressed to the peer), and the peer's epilogue warps releasing the accumulator to
// the leader.
// Measured on B200 (T = 4, 32 768 tokens, forward): 56.7 / 135 / 476 / 1964 us at 256 / 512 / 1024 / 2048 channels
// against 54.3 / 138 / 491 / 1937 us for the single-CTA form (data gradient at 2048: 1952 against 2168 us),
// bit-identical results.  The gain is small because these main loops run at the SM's shared-memory bandwidth
// (~112 KB cross shared memory per 16-channel chunk: raw rows in and out, x^ in, operand reads, weight refill; at
// 128 B per cycle that is the measured ~880 cycles per chunk), and of those bytes the pair form removes only half
// of the weight refill: each SM's shared memory still serves its half of B to BOTH tensor cores.
// (With release / acquire at cluster scope on the pair's barriers the form ran 1.7x slower: a cluster-scope release
// stalls the arriving thread ~1200 cycles, a cluster-scope acquire ~250.)
//
// Every wait on an mbarrier is bounded: on a time-out the CTA raises an abort flag, records a status
// code for the host, drains its outstanding copies and MMAs, frees its TMEM and returns.
#include <cuda_fp16.h>

#include <cstring>
#include <mutex>

#include "eql_internal.h"
#include "ptx_sm100.cuh"
#include "rdft.cuh"
#include "umma_common.cuh"

namespace eql {
namespace {

constexpr int kTileM = 128;            // tokens per tile = UMMA M = TMEM lanes
constexpr int kRowBytes = 32;           // operand row of one pipeline stage = one UMMA K step (16 halves / 8 floats)
constexpr int kSlabBytes = kTileM * 128;
constexpr int kThreadsUmma = 512;
constexpr int kTmemCols = 512;

// warp roles
constexpr int kWarpTmaX = 0, kWarpMma = 1, kWarpTmaB = 2, kWarpCompute0 = 4;
constexpr int kNumComputeWarps = 12;

template <int T, int E, int CG = 1> struct UmmaCfg;   // E = bytes per element of the I/O tensors (2: half, 4: float); CG: CTAs per MMA
// Ring depths.  The raw ring has 3 slots of SPS slabs (16 KB each) that complete on one barrier; with 3 slots every
// slot is always served by the same warp groups (slab number mod 3 selects the group).  SA transformed-operand
// stages (T*4 KB each, twice that for the hi/lo halves of FP32), SB weight-image slots.  Measured on the EQ-ViT-B
// shape: a raw slot is released only after its rows have been transformed and stored, so a deep raw ring (6 slabs)
// matters more than a third weight-image slot.
// EARLY: release a raw slot as soon as its rows are in registers (one more fence + arrive per item) instead of after
// the transformed rows have been stored; used where the raw ring cannot be deep.
// MAXCOT: output channels per tile (T*CoT fp32 TMEM columns <= 512, and the weight-image slot must fit).
// MERGED (needs SA == SB): chunk q uses operand stage q % SA AND weight slot q % SA, and one "full" barrier (transform
// warps + the weight copy's bytes) and one "empty" barrier (one commit) per chunk serve both.  The single thread that
// issues the MMAs then executes one wait and one commit per chunk instead of two each; each costs it ~200 cycles while
// the tensor core is streaming operands, and on wide layers that thread paces the kernel.
// KS: chunks (UMMA K steps) per operand stage and weight slot.  With two, the issuing thread's wait and commit are paid
// once per 32 reduced channels (the reduction is padded to a multiple of KS chunks with zero channels).
template <> struct UmmaCfg<2, 2, 1>  { static constexpr int SPS = 1, SA = 3, SB = 3, KS = 2, MAXCOT = 256; static constexpr bool EARLY = true, MERGED = true; };
template <> struct UmmaCfg<4, 2, 1>  { static constexpr int SPS = 1, SA = 2, SB = 2, KS = 2, MAXCOT = 128; static constexpr bool EARLY = true, MERGED = true; };
template <> struct UmmaCfg<8, 2, 1>  { static constexpr int SPS = 2, SA = 2, SB = 2, KS = 1, MAXCOT = 64;  static constexpr bool EARLY = false, MERGED = true; };
template <> struct UmmaCfg<16, 2, 1> { static constexpr int SPS = 1, SA = 2, SB = 1, KS = 1, MAXCOT = 32;  static constexpr bool EARLY = true, MERGED = false; };
template <> struct UmmaCfg<32, 2, 1> { static constexpr int SPS = 1, SA = 1, SB = 1, KS = 1, MAXCOT = 16;  static constexpr bool EARLY = true, MERGED = false; };
template <> struct UmmaCfg<4, 4, 1>  { static constexpr int SPS = 1, SA = 3, SB = 1, KS = 1, MAXCOT = 128; static constexpr bool EARLY = true, MERGED = false; };
template <> struct UmmaCfg<8, 4, 1>  { static constexpr int SPS = 1, SA = 2, SB = 1, KS = 1, MAXCOT = 48;  static constexpr bool EARLY = true, MERGED = false; };
// CTA pairs: a CTA holds half of every weight tile, which leaves room for deeper rings (measured: depths beyond these
// change nothing, for either form -- the rings are not what paces the kernel).
template <> struct UmmaCfg<4, 2, 2>  { static constexpr int SPS = 1, SA = 3, SB = 3, KS = 2, MAXCOT = 128; static constexpr bool EARLY = true, MERGED = true; };
template <> struct UmmaCfg<8, 2, 2>  { static constexpr int SPS = 2, SA = 2, SB = 2, KS = 1, MAXCOT = 64;  static constexpr bool EARLY = false, MERGED = true; };
constexpr int kRawSlots = 3;
constexpr uint32_t kSpin = 256;               // test_wait polls before a single-thread role falls back to try_wait

struct UmmaParams {
    void* out;                   // [N, Cout*T]
    const uint8_t* image;        // spectral-weight operand image, see build_image_kernel
    const float* bias;           // [Cout] or nullptr
    int* status;                 // device status word of the plan
    int64_t N;
    int Cin, Cout;
    int CoT, nTiles, nK, rowsB;
    int b_slot_bytes;            // bytes of one B ring slot (rowsB*32, twice that for FP32, rounded up to 128)
    int64_t num_units;
    int accumulate;              // out += result (TMA reduce-add) instead of out = result: later segments of a reduction
    int act;                     // 1: GELU on the result (forward of a plan built with EQL_FLAG_GELU)
};


struct SmemBarriers {
    uint64_t full_raw[6], empty_raw[6];
    uint64_t full_a[8], empty_a[8];      // SA <= 8
    uint64_t full_b[4], empty_b[4];      // SB <= 4 (unmerged rings)
    uint64_t full_d, empty_d, mma_done, staging_free;
    uint32_t tmem_base;
    int abort_flag;
};

// ------------------------------------------------------------------------------------------------
// Operand image of the spectral weight for the tensor-core kernel.
// planes[p][cin][cout] (float, already scaled by 1/T resp. 2/T, conjugated for the data gradient) ->
// for every (output tile, channel chunk of one UMMA K step) one blob of rowsB rows x 32 bytes in the canonical K-major
// layout with 32-byte swizzle: byte b of row n lives at n*32 + (((b>>4) ^ ((n>>2)&1))<<4) + (b&15).
// FP32 plans store two such blobs back to back: the TF32 "hi" parts and the "lo" remainders (3xTF32).
// Rows of a blob (CoT = output channels per tile):
//   [0, CoT)                         plane 0 (k = 0)
//   per complex frequency f (4*CoT): Wr | Wi   (multiplied by Re x^)   then   -Wi | Wr   (by Im x^)
//   [rowsB - CoT, rowsB)             plane T-1 (k = T/2)
//
// CTA-pair layout (pair != 0): every B tile (the rows one MMA reads) is split in halves, the first half of its rows
// for the leader CTA and the second for its peer, and a blob holds first everything the leader loads, then everything
// the peer loads: [half][hi | lo part][rowsB / 2 rows].  The halves of a real plane are its first and second CoT / 2
// output channels; the halves of a complex frequency's tiles [Wr | Wi] and [-Wi | Wr] are the rows that produce Re y^
// (leader) and Im y^ (peer).
template <int T, typename IO>
__global__ void build_image_kernel(const float* __restrict__ planes, int Cin, int Cout, int CoT, int nTiles, int nK,
                                   int rowsB, IO* __restrict__ image, int cin0, int CinTotal, int pair) {
    constexpr int E = sizeof(IO), KCH = kRowBytes / E, EPC = 16 / E, NSPLIT = E == 4 ? 2 : 1;
    const int64_t per_blob = (int64_t)NSPLIT * rowsB * KCH;
    const int64_t total = (int64_t)nTiles * nK * per_blob;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int within_all = (int)(idx % per_blob);
        const int64_t blob = idx / per_blob;
        const int kc = (int)(blob % nK), tile = (int)(blob / nK);
        int part, within, plane, local;
        float sign = 1.f;
        if (pair) {
            const int rowsH = rowsB / 2, H = CoT / 2;
            const int half = within_all / (NSPLIT * rowsH * KCH), rem = within_all % (NSPLIT * rowsH * KCH);
            part = rem / (rowsH * KCH);
            within = rem % (rowsH * KCH);
            const int n = within / KCH;                              // row inside this CTA's half of the blob
            if (n < H) {
                plane = 0; local = half * H + n;
            } else if (n >= rowsH - H) {
                plane = T - 1; local = half * H + n - (rowsH - H);
            } else {
                const int m = n - H, f = m / (2 * CoT) + 1, second = (m / CoT) & 1;   // second: the tile multiplied by Im x^
                local = m % CoT;
                if (!second) plane = half == 0 ? 2 * f - 1 : 2 * f;                  // Wr -> Re y^ | Wi -> Im y^
                else if (half == 0) { plane = 2 * f; sign = -1.f; }                 // -Wi -> Re y^
                else plane = 2 * f - 1;                                             // Wr -> Im y^
            }
        } else {
            part = within_all / (rowsB * KCH);
            within = within_all % (rowsB * KCH);
            const int n = within / KCH;
            if (n < CoT) {
                plane = 0; local = n;
            } else if (n >= rowsB - CoT) {
                plane = T - 1; local = n - (rowsB - CoT);
            } else {
                const int m = n - CoT, f = m / (4 * CoT) + 1, quarter = (m / CoT) & 3;
                local = m % CoT;
                if (quarter == 0) plane = 2 * f - 1;                     // Wr  -> Re y^
                else if (quarter == 1) plane = 2 * f;                    // Wi  -> Im y^
                else if (quarter == 2) { plane = 2 * f; sign = -1.f; }   // -Wi -> Re y^
                else plane = 2 * f - 1;                                  // Wr  -> Im y^
            }
        }
        // destination element `within` of the (half-)blob: row n, 16-byte chunk c, element e of the chunk; the chunk
        // holds k-half (c ^ bit 2 of n) (32-byte swizzle)
        const int n = within / KCH;
        const int c = (within % KCH) / EPC;
        const int kk = (c ^ ((n >> 2) & 1)) * EPC + within % EPC;
        const int cin = kc * KCH + kk, cout = tile * CoT + local;
        float v = 0.f;
        if (cin < Cin && cout < Cout) v = sign * planes[((size_t)plane * CinTotal + cin0 + cin) * Cout + cout];
        if constexpr (E == 2) {
            image[idx] = H16<IO>::narrow(v);
        } else {
            uint32_t hi, lo;
            split_tf32(v, hi, lo);
            image[idx] = __uint_as_float(part == 0 ? hi : lo);
        }
    }
}

// ------------------------------------------------------------------------------------------------
template <int T, typename IO, int CG, bool ACT>
__global__ void __launch_bounds__(kThreadsUmma, 1)
umma_linear_kernel(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_out,
                   const UmmaParams prm) {
    constexpr int E = sizeof(IO);               // 2: half I/O, kind::f16;  4: float I/O, kind::tf32 with the 3xTF32 split
    using Cfg = UmmaCfg<T, E, CG>;
    constexpr int SPS = Cfg::SPS, SA = Cfg::SA, SB = Cfg::SB, KS = Cfg::KS;
    constexpr bool PAIR = CG == 2, MERGED = Cfg::MERGED;
    static_assert(!MERGED || SA == SB, "one barrier pair per chunk needs equally deep rings");
    static_assert(!PAIR || MERGED, "the CTA-pair form is written for the merged rings");
    constexpr int SR = kRawSlots * SPS;         // slabs in the raw ring
    constexpr int EPR = 128 / E;                // elements per raw slab row (128 B)
    constexpr int NCH = EPR / T;                // channels per raw slab row
    constexpr int KCH = kRowBytes / E;          // channels per chunk = one UMMA K step (16 halves / 8 floats)
    constexpr int SPK = KCH >= NCH ? KCH / NCH : 1;   // slabs per chunk (= T/4; one slab holds both chunks of a stage at T = 2)
    constexpr int CPS = NCH > KCH ? NCH / KCH : 1;    // chunks per slab (2 at T = 2: a 128-byte row is 32 channels)
    static_assert(CPS == 1 || CPS == KS, "a slab that spans chunks must span exactly one stage");
    constexpr int SLABS_PER_STAGE = SPK * KS / CPS;
    constexpr int NSPLIT = E == 4 ? 2 : 1;      // operand copies: FP32 keeps TF32 hi parts and lo remainders
    constexpr int kAPart = T * 4096;            // T planes x [128 rows x 32 B]
    constexpr int kAChunk = kAPart * NSPLIT;    // one chunk's operand tiles
    constexpr int kAStage = kAChunk * KS;
    constexpr int W = NCH * E / 4;              // 32-bit words one slab row contributes to one plane

    extern __shared__ uint8_t smem_raw_base[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_base) + 1023) & ~(uintptr_t)1023);
    uint8_t* raw = smem;                                   // SR slabs
    uint8_t* xhat = raw + SR * kSlabBytes;                 // SA stages
    uint8_t* bsm = xhat + SA * kAStage;                    // SB slots
    SmemBarriers* bar = reinterpret_cast<SmemBarriers*>(bsm + SB * prm.b_slot_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = &bar->abort_flag;
    int* status = prm.status;

    // A unit is (token tile, channel tile); a pair takes two neighbouring token tiles per unit, one per CTA.
    const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < kRawSlots; ++i) { ptx::mbar_init(&bar->full_raw[i], 1); ptx::mbar_init(&bar->empty_raw[i], 4 * SPS); }
        // "full" of a stage: the transform warps; merged rings: + the weight copy (its producer's arrive.expect_tx);
        // pair, leader: + the peer CTA's word that its own stage is full
        const uint32_t full_count = 4 * SLABS_PER_STAGE + (MERGED ? 1 : 0) + ((PAIR && rank == 0) ? 1 : 0);
        for (int i = 0; i < SA; ++i) { ptx::mbar_init(&bar->full_a[i], full_count); ptx::mbar_init(&bar->empty_a[i], 1); }
        for (int i = 0; i < SB; ++i) { ptx::mbar_init(&bar->full_b[i], 1); ptx::mbar_init(&bar->empty_b[i], 1); }
        ptx::mbar_init(&bar->full_d, 1);
        ptx::mbar_init(&bar->empty_d, kNumComputeWarps * CG);    // pair: the leader's barrier takes both CTAs' warps
        ptx::mbar_init(&bar->mma_done, 1);
        ptx::mbar_init(&bar->staging_free, kNumComputeWarps);
        bar->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_in);
        ptx::prefetch_tensormap(&tmap_out);
    }
    if (warp == kWarpMma) {
        if constexpr (PAIR) { ptx::tmem_alloc_pair(&bar->tmem_base, kTmemCols); ptx::tmem_relinquish_pair(); }
        else { ptx::tmem_alloc(&bar->tmem_base, kTmemCols); ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if constexpr (PAIR) {                       // the peer's barriers must be initialised before anything arrives on them
        ptx::cluster_arrive();
        ptx::cluster_wait();
    }
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bar->tmem_base;
    // This kernel may have been scheduled while the kernel before it in the stream is still finishing: everything above
    // (barriers, tensor memory) overlapped that; nothing below may run before its results are visible.  The kernel
    // behind this one gets the same head start.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    const int nK = prm.nK, nTiles = prm.nTiles, CoT = prm.CoT, rowsB = prm.rowsB;
    const int64_t first = blockIdx.x / CG, stride = gridDim.x / CG;
    auto unit_row0 = [&](int64_t u) { return (int)(((u / nTiles) * CG + rank) * kTileM); };
    const int rowsH = rowsB / CG;                                // weight-image rows this CTA holds per (tile, chunk)
    // barriers of the weight ring: its own, or (merged rings) those of the operand stages
    uint64_t* const full_wb = MERGED ? bar->full_a : bar->full_b;
    uint64_t* const empty_wb = MERGED ? bar->empty_a : bar->empty_b;

    if (warp == kWarpTmaX) {
        // ---------------------------------------------------------------- raw activation rows via TMA
        if (lane == 0) {
            uint32_t cr = 0;                                     // running slab counter; slot phase = cr / SPS
            bool ok = true;
            for (int64_t u = first; u < prm.num_units && ok; u += stride) {
                const int row0 = unit_row0(u);
                for (int kc = 0; kc < nK && ok; kc += CPS) {
                    for (int q = 0; q < SPK; ++q, ++cr) {
                        const uint32_t ph = cr / SPS;            // slot phase counter
                        const int slot = ph % kRawSlots;
                        if (cr % SPS == 0) {
                            ok = ptx::mbar_wait(&bar->empty_raw[slot], ((ph / kRawSlots) & 1) ^ 1, abort_flag, status, 101, true, kSpin);
                            if (!ok) break;
                            ptx::mbar_arrive_expect_tx(&bar->full_raw[slot], SPS * kSlabBytes);
                        }
                        ptx::tma_load_2d(raw + (slot * SPS + cr % SPS) * kSlabBytes, &tmap_in, (kc * KCH + q * NCH) * T, row0,
                                         &bar->full_raw[slot]);
                    }
                }
            }
            // A slot phase must receive all SPS loads it was armed for, also at the very end of the work.
            if (ok) {
                while (cr % SPS != 0) {
                    const uint32_t ph = cr / SPS;
                    ptx::tma_load_2d(raw + ((ph % kRawSlots) * SPS + cr % SPS) * kSlabBytes, &tmap_in, 0, 0, &bar->full_raw[ph % kRawSlots]);
                    ++cr;
                }
            }
            // drain: every copy this thread issued must have landed before the CTA may exit
            {
                const uint32_t nph = (cr + SPS - 1) / SPS;
                const uint32_t lo = nph > (uint32_t)kRawSlots ? nph - kRawSlots : 0;
                for (uint32_t c = lo; c < nph; ++c)
                    ptx::mbar_wait(&bar->full_raw[c % kRawSlots], (c / kRawSlots) & 1, abort_flag, status, 111, false);
            }
        }
    } else if (warp == kWarpTmaB) {
        // ---------------------------------------------------------------- spectral-weight blobs via bulk copy
        if (lane == 0) {
            uint32_t cb = 0;
            bool ok = true;
            const uint32_t blob_bytes = (uint32_t)rowsH * kRowBytes * NSPLIT;       // pair: this CTA's half of the blob
            for (int64_t u = first; u < prm.num_units && ok; u += stride) {
                const int tile = (int)(u % nTiles);
                for (int kc = 0; kc < nK; kc += KS, ++cb) {          // one slot per stage: KS chunks
                    const int slot = cb % SB;
                    ok = ptx::mbar_wait(&empty_wb[slot], ((cb / SB) & 1) ^ 1, abort_flag, status, 102, true, kSpin);
                    if (!ok) break;
                    ptx::mbar_arrive_expect_tx(&full_wb[slot], KS * blob_bytes);
#pragma unroll
                    for (int sub = 0; sub < KS; ++sub)
                        ptx::bulk_load_1d(bsm + slot * prm.b_slot_bytes + sub * blob_bytes,
                                          prm.image + (((size_t)tile * nK + kc + sub) * CG + rank) * (size_t)blob_bytes, blob_bytes,
                                          &full_wb[slot]);
                }
            }
            if (!ok) {
                // giving up: the copies still in flight must land before this CTA's shared memory goes away (with merged
                // rings the phase also needs the transform warps, which may have given up too: the wait is bounded)
                const uint32_t lo = cb > (uint32_t)SB ? cb - SB : 0;
                for (uint32_t c = lo; c < cb; ++c)
                    ptx::mbar_wait(&full_wb[c % SB], (c / SB) & 1, abort_flag, status, 112, false);
            }
        }
    } else if (warp == kWarpMma) {
        // ---------------------------------------------------------------- tensor-core issue (one thread)
        if (lane == 0 && rank == 0) {
            uint32_t ca = 0, cb = 0, cu = 0;
            bool ok = true;
            constexpr int M = kTileM * CG;
            constexpr uint32_t kFmt = H16<IO>::kUmmaFormat;      // half or bfloat16 operands
            const uint32_t idesc_real = E == 2 ? ptx::umma_idesc_f16_f32(M, CoT, kFmt) : ptx::umma_idesc_tf32_f32(M, CoT);
            const uint32_t idesc_cplx = E == 2 ? ptx::umma_idesc_f16_f32(M, 2 * CoT, kFmt) : ptx::umma_idesc_tf32_f32(M, 2 * CoT);
            auto mma = [](uint32_t d, uint32_t a_addr, uint32_t b_addr, uint32_t idesc, uint32_t accumulate) {
                const uint64_t ad = ptx::umma_smem_desc_k_sw32(a_addr), bd = ptx::umma_smem_desc_k_sw32(b_addr);
                if constexpr (E == 2) {
                    if constexpr (PAIR) ptx::umma_f16_pair(d, ad, bd, idesc, accumulate);
                    else ptx::umma_f16(d, ad, bd, idesc, accumulate);
                } else {
                    if constexpr (PAIR) ptx::umma_tf32_pair(d, ad, bd, idesc, accumulate);
                    else ptx::umma_tf32(d, ad, bd, idesc, accumulate);
                }
            };
            // a barrier of this CTA and, in a pair, the barrier at the same place in the peer CTA
            auto commit_both = [&](uint64_t* b) {
                if constexpr (PAIR) {
                    ptx::umma_commit_pair(b);
                    ptx::umma_commit_pair_addr(ptx::map_to_cta(ptx::smem_u32(b), 1u));
                } else {
                    ptx::umma_commit(b);
                }
            };
            // Rows of this CTA's weight slot (pair: half tiles).  Real plane: CoT / CG rows; a complex frequency: two
            // tiles of 2 CoT / CG rows each.
            const uint32_t b_part = (uint32_t)rowsH * kRowBytes;
            const uint32_t rows_real = (uint32_t)(CoT / CG), rows_cplx = (uint32_t)(2 * CoT / CG);
            for (int64_t u = first; u < prm.num_units && ok; u += stride, ++cu) {
                ok = ptx::mbar_wait(&bar->empty_d, (cu & 1) ^ 1, abort_flag, status, 103, true, kSpin);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                for (int kc = 0; kc < nK; kc += KS, ++ca, ++cb) {    // ca, cb count stages
                    const int sa = ca % SA, sb = cb % SB;
                    // (pair: the peer's arrival on this barrier stands for shared memory of the peer CTA that the peer's own
                    // threads wrote and fenced; a wait with acquire at cluster scope instead costs ~250 cycles per chunk)
                    ok = ptx::mbar_wait(&bar->full_a[sa], (ca / SA) & 1, abort_flag, status, 104, true, kSpin);
                    if constexpr (!MERGED) ok = ok && ptx::mbar_wait(&bar->full_b[sb], (cb / SB) & 1, abort_flag, status, 105, true, kSpin);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // FP16: one pass.  FP32 (3xTF32): hi*hi, hi*lo, lo*hi accumulate into the same columns.
#pragma unroll
                    for (int sub = 0; sub < KS; ++sub)
#pragma unroll
                    for (int pass = 0; pass < (E == 4 ? 3 : 1); ++pass) {
                        const uint32_t a0 = ptx::smem_u32(xhat + sa * kAStage + sub * kAChunk) + (pass == 2 ? kAPart : 0);
                        const uint32_t b0 = ptx::smem_u32(bsm + sb * prm.b_slot_bytes) + sub * b_part * NSPLIT + (pass == 1 ? b_part : 0);
                        const uint32_t acc = (kc > 0 || sub > 0 || pass > 0) ? 1u : 0u;
                        // k = 0
                        mma(tmem_base, a0, b0, idesc_real, acc);
                        // complex frequencies: [Re y^ | Im y^] (+)= Re x^ [Wr|Wi] + Im x^ [-Wi|Wr]
#pragma unroll
                        for (int f = 1; f < T / 2; ++f) {
                            const uint32_t d = tmem_base + (uint32_t)((2 * f - 1) * CoT);
                            const uint32_t rb = rows_real + (uint32_t)(f - 1) * 2 * rows_cplx;
                            mma(d, a0 + (2 * f - 1) * 4096, b0 + rb * kRowBytes, idesc_cplx, acc);
                            mma(d, a0 + (2 * f) * 4096, b0 + (rb + rows_cplx) * kRowBytes, idesc_cplx, 1u);
                        }
                        // k = T/2
                        mma(tmem_base + (uint32_t)((T - 1) * CoT), a0 + (T - 1) * 4096,
                            b0 + ((uint32_t)rowsH - rows_real) * kRowBytes, idesc_real, acc);
                    }
                    commit_both(&bar->empty_a[sa]);
                    if constexpr (!MERGED) commit_both(&bar->empty_b[sb]);
                }
                if (ok) commit_both(&bar->full_d);
            }
            // all MMAs issued by this thread must have retired before shared memory and TMEM go away
            if constexpr (PAIR) ptx::umma_commit_pair(&bar->mma_done);
            else ptx::umma_commit(&bar->mma_done);
            ptx::mbar_wait(&bar->mma_done, 0, abort_flag, status, 113, false);
        } else if (PAIR && lane == 0) {
            // The peer CTA of a pair issues no MMA.  This thread tells the leader when this CTA's stage of a chunk
            // (transformed rows and weight half) is full, by arriving on the leader's barrier of the same stage; the
            // leader's commits release the stage in both CTAs.
            uint32_t ca = 0;
            bool ok = true;
            const uint32_t leader_full0 = ptx::map_to_cta(ptx::smem_u32(&bar->full_a[0]), 0u);
            for (int64_t u = first; u < prm.num_units && ok; u += stride) {
                for (int kc = 0; kc < nK; kc += KS, ++ca) {
                    ok = ptx::mbar_wait(&bar->full_a[ca % SA], (ca / SA) & 1, abort_flag, status, 116, true, kSpin);
                    if (!ok) break;
                    ptx::mbar_arrive_remote(leader_full0 + (ca % SA) * 8u);
                }
            }
        }
    } else if (warp >= kWarpCompute0) {
        // ---------------------------------------------------------------- compute warps: transform, then epilogue
        // Per unit every compute warp first transforms its share of the raw slab rows (group DFT -> A operands)
        // and then drains its share of the accumulator (inverse DFT -> global).  Work items of the transform
        // are (slab, 32-row quarter).
        constexpr int G = EPR / T;                               // channels per TMEM read group (128 output bytes per token)
        // The 12 warps form 3 groups of 4; raw slab number cr is transformed by group cr % 3, one 32-row quarter
        // per warp.  Because the ring has 3 slots, a slot is always served by the same groups, so each warp
        // sees every phase of the slot barriers it waits on, in order (a parity wait is only unambiguous one
        // phase ahead).  A warp's consecutive slabs are 3 apart, i.e. 3/SPK chunks, which must stay below SA
        // (a warp that stored into chunk c' has seen the commit of chunk c' - SA, so when it next waits for the
        // commit of chunk c - SA with c - c' <= SA the barrier is at most one phase behind).
        static_assert(kRawSlots == 3 && SPS <= 3, "raw slots must map to fixed warp groups");
        static_assert((3 + SLABS_PER_STAGE - 1) / SLABS_PER_STAGE <= SA, "empty_a parity wait would be ambiguous");
        const int cw = warp - kWarpCompute0;
        const int quad = warp & 3;                               // TMEM lane quadrant this warp may read
        const int group = cw >> 2;                               // transform group, and share of the epilogue's column groups
        const int third = group;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t ca = 0, cu = 0;
        bool ok = true;
        // the accumulator of this CTA has been read: tell the MMA-issuing thread (in a pair, the leader CTA's)
        const uint32_t empty_d_leader = PAIR ? ptx::map_to_cta(ptx::smem_u32(&bar->empty_d), 0u) : 0u;
        auto release_d = [&]() {
            if (PAIR && rank != 0) ptx::mbar_arrive_remote(empty_d_leader);
            else ptx::mbar_arrive(&bar->empty_d);
        };
        bool staging_pending = false;                            // previous unit's TMA stores may still be reading the stage
        uint8_t* staging = xhat + cw * 4096;                     // this warp's [32 tokens x 128 B] output stage (128B swizzle)
        for (int64_t u = first; u < prm.num_units && ok; u += stride, ++cu) {
            // ---- transform
            for (int kc = 0; kc < nK && ok; kc += CPS, ca += CPS) {   // ca counts chunks here; stage = chunk / KS
                const uint32_t stage = ca / KS;
                const int sa = stage % SA;
#pragma unroll 1
                for (int q = 0; q < SPK; ++q) {
                    const uint32_t cr = (ca / CPS) * SPK + q;    // running slab counter
                    if ((int)(cr % 3) != group) continue;
                    const uint32_t ph = cr / SPS;                // raw-ring slot phase this slab arrives in
                    const int slot = ph % kRawSlots;
                    ok = ptx::mbar_wait(&bar->full_raw[slot], (ph / kRawSlots) & 1, abort_flag, status, 106, true, 16);
                    if (!ok) break;
                    const int d = quad;                          // this warp's 32-row quarter of the slab
                    const int r = d * 32 + lane;
                    uint32_t wd[32];
                    load_slab_row(raw + (slot * SPS + cr % SPS) * kSlabBytes + r * 128, r, wd);
                    if constexpr (Cfg::EARLY) {
                        // The rows are in registers: order these generic-proxy reads before the async-proxy (TMA)
                        // refill of the slot, then release it so that the refill overlaps the transform.
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(&bar->empty_raw[slot]);
                    }
                    // A tile of a plane: row r at r*32, its two 16-byte chunks exchanged when bit 2 of r is set (32B swizzle);
                    // this slab row's run of channels starts at byte kb of the row
                    const int kb = q * NCH * E;
                    const int sw = (r >> 2) & 1;
                    uint8_t* dst = xhat + sa * kAStage + (ca % KS) * kAChunk + r * 32 + (((kb >> 4) ^ sw) << 4) + (kb & 15);
                    const int second = sw ? -16 : 16;            // where the other half of the same row lives (32-byte runs only)
                    uint32_t packed[E == 2 ? T : 1][E == 2 ? NCH / 2 : 1];
                    if constexpr (E == 2) {
                        dft_words<T, false, false, IO>(wd, packed, nullptr);
                    } else {
                        dft_words_f32<T>(wd);                    // wd[c*T + p] = plane p of channel c
                    }
                    ok = ptx::mbar_wait(&bar->empty_a[sa], ((stage / SA) & 1) ^ 1, abort_flag, status, 107, true, 16);
                    if (!ok) break;
                    if (staging_pending) {                       // the previous unit's output stage lives in the A-operand stages
                        ok = ptx::mbar_wait(&bar->staging_free, (cu - 1) & 1, abort_flag, status, 109, true, 16);
                        if (!ok) break;
                        staging_pending = false;
                    }
                    if constexpr (E == 2 && CPS == 2) {
                        // the row's 32 channels are the stage's two chunks: 16 channels (one full 32-byte operand row) each
#pragma unroll
                        for (int p = 0; p < T; ++p) {
                            store_plane_run<16>(dst + p * 4096, &packed[p][0], second);
                            store_plane_run<16>(dst + kAChunk + p * 4096, &packed[p][8], second);
                        }
                    } else if constexpr (E == 2) {
#pragma unroll
                        for (int p = 0; p < T; ++p) store_plane_run<2 * W>(dst + p * 4096, packed[p], second);
                    } else {
#pragma unroll
                        for (int p = 0; p < T; ++p) {
                            uint32_t hi[W], lo[W];
#pragma unroll
                            for (int c = 0; c < NCH; ++c) split_tf32(__uint_as_float(wd[c * T + p]), hi[c], lo[c]);
                            store_plane_run<2 * W>(dst + p * 4096, hi, second);
                            store_plane_run<2 * W>(dst + kAPart + p * 4096, lo, second);
                        }
                    }
                    ptx::fence_proxy_async_smem();               // generic-proxy writes -> visible to the MMA (async proxy)
                    __syncwarp();
                    // The same fence also orders this thread's earlier generic-proxy reads of the raw slab before the
                    // async-proxy (TMA) refill that the release below allows.
                    if (lane == 0) {
                        if constexpr (!Cfg::EARLY) ptx::mbar_arrive(&bar->empty_raw[slot]);
                        ptx::mbar_arrive(&bar->full_a[sa]);
                    }
                }
            }
            if (!ok) break;
            // ---- epilogue
            const int tile = (int)(u % nTiles);
            ok = ptx::mbar_wait(&bar->full_d, cu & 1, abort_flag, status, 108, true, 16);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const int ngroups = CoT / G;
            for (int gi = third; gi < ngroups; gi += 3) {
                const int c0 = gi * G;
                uint32_t in[T][G];
#pragma unroll
                for (int p = 0; p < T; ++p) ptx::tmem_ld<G>(lane_base + (uint32_t)(p * CoT + c0), in[p]);
                ptx::tmem_ld_wait();
                if (gi + 3 >= ngroups) {                         // this warp's last read of the accumulator
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) release_d();
                }
                const int co0 = tile * CoT + c0;
                uint32_t o[32];                                  // G channels x T elements = 128 bytes
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float v[T];
#pragma unroll
                    for (int p = 0; p < T; ++p) v[p] = __uint_as_float(in[p][g]);
                    if (prm.bias != nullptr && co0 + g < prm.Cout) v[0] += __ldg(prm.bias + co0 + g);
                    rdft_inverse<T>(v);
                    if constexpr (ACT) {                         // fused GELU: its own instantiation of the kernel
#pragma unroll
                        for (int t = 0; t < T; ++t) v[t] = gelu_erf(v[t]);
                    }
                    if constexpr (E == 2) {
#pragma unroll
                        for (int t = 0; t < T; t += 2) o[(g * T + t) / 2] = H16<IO>::pack(v[t], v[t + 1]);
                    } else {
#pragma unroll
                        for (int t = 0; t < T; ++t) o[g * T + t] = __float_as_uint(v[t]);
                    }
                }
                // stage the warp's 32 rows of 128 bytes (chunk j of row l at j ^ (l & 7): the tensor map's 128B swizzle) and
                // hand them to one asynchronous TMA store; rows >= N and channels >= Cout are clipped by the hardware
                if (lane == 0) ptx::bulk_wait_group_read0();     // previous group's stage has been read
                __syncwarp();
#pragma unroll
                for (int jj = 0; jj < 8; ++jj)
                    *reinterpret_cast<uint4*>(staging + lane * 128 + ((jj ^ (lane & 7)) << 4)) =
                        make_uint4(o[4 * jj], o[4 * jj + 1], o[4 * jj + 2], o[4 * jj + 3]);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && co0 < prm.Cout) {
                    if (prm.accumulate) ptx::tma_reduce_add_2d(&tmap_out, co0 * T, unit_row0(u) + quad * 32, staging);
                    else ptx::tma_store_2d(&tmap_out, co0 * T, unit_row0(u) + quad * 32, staging);
                    ptx::bulk_commit_group();
                }
            }
            // the A-operand stages double as the output stage: the next unit's transform may overwrite them only after
            // every warp's stores have read their source
            if (lane == 0) {
                ptx::bulk_wait_group_read0();
                ptx::mbar_arrive(&bar->staging_free);
            }
            staging_pending = true;
            if (third >= ngroups) {                              // fewer column groups than shares: nothing to read
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) release_d();
            }
        }
    }

    // ---------------------------------------------------------------- teardown (reached by every thread)
    ptx::tc_fence_before_sync();
    __syncthreads();
    if constexpr (PAIR) {                       // neither CTA may leave while the other can still signal it or read its memory
        ptx::cluster_arrive();
        ptx::cluster_wait();
    }
    if (warp == kWarpMma) {
        ptx::tc_fence_after_sync();
        if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
        else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
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

template <int T, int E, int CG>
size_t umma_smem_bytes(int b_slot_bytes) {
    using Cfg = UmmaCfg<T, E, CG>;
    return 1024 + (size_t)kRawSlots * Cfg::SPS * kSlabBytes + (size_t)Cfg::SA * Cfg::KS * T * 4096 * (E == 4 ? 2 : 1) +
           (size_t)Cfg::SB * b_slot_bytes + sizeof(SmemBarriers) + 64;
}

// Calls f(integral_constant<T>, element type tag) for the supported (T, dtype) pairs.
template <typename F>
cudaError_t dispatch_umma(int T, int elem_bytes, F&& f, bool bf16 = false) {
    if (elem_bytes == 2 && bf16) {
        switch (T) {
            case 2: return f(std::integral_constant<int, 2>{}, __nv_bfloat16{});
            case 4: return f(std::integral_constant<int, 4>{}, __nv_bfloat16{});
            case 8: return f(std::integral_constant<int, 8>{}, __nv_bfloat16{});
            case 16: return f(std::integral_constant<int, 16>{}, __nv_bfloat16{});
            case 32: return f(std::integral_constant<int, 32>{}, __nv_bfloat16{});
            default: return cudaErrorInvalidValue;
        }
    }
    if (elem_bytes == 2) {
        switch (T) {
            case 2: return f(std::integral_constant<int, 2>{}, __half{});
            case 4: return f(std::integral_constant<int, 4>{}, __half{});
            case 8: return f(std::integral_constant<int, 8>{}, __half{});
            case 16: return f(std::integral_constant<int, 16>{}, __half{});
            case 32: return f(std::integral_constant<int, 32>{}, __half{});
            default: return cudaErrorInvalidValue;
        }
    }
    switch (T) {
        case 4: return f(std::integral_constant<int, 4>{}, float{});
        case 8: return f(std::integral_constant<int, 8>{}, float{});
        default: return cudaErrorInvalidValue;
    }
}

int umma_chunks_per_stage(int T, int elem_bytes, bool pair) {
    int k = 1;
    dispatch_umma(T, elem_bytes, [&](auto tc, auto io) {
        constexpr int TT = decltype(tc)::value, EE = sizeof(decltype(io));
        k = UmmaCfg<TT, EE, 1>::KS;
        if constexpr (EE == 2 && (TT == 4 || TT == 8)) { if (pair) k = UmmaCfg<TT, EE, 2>::KS; }
        return cudaSuccess;
    });
    return k;
}

int umma_max_cot(int T, int elem_bytes) {
    int m = 0;
    dispatch_umma(T, elem_bytes, [&](auto tc, auto io) {
        m = UmmaCfg<decltype(tc)::value, sizeof(decltype(io)), 1>::MAXCOT;
        return cudaSuccess;
    });
    return m;
}

}  // namespace


bool umma_linear_supported(int T, eql_dtype_t dtype) {
    if (dtype == EQL_FP16 || dtype == EQL_BF16) return T == 2 || T == 4 || T == 8 || T == 16 || T == 32;
    return T == 4 || T == 8;            // FP32 (3xTF32): the hi/lo operand stages of larger T do not fit in shared memory
}

UmmaLinearShape umma_linear_shape(int T, int Cin, int Cout, eql_dtype_t dtype) {
    UmmaLinearShape s{};
    s.T = T; s.Cin = Cin; s.Cout = Cout;
    s.elem_bytes = dtype == EQL_FP32 ? 4 : 2;
    s.bf16 = dtype == EQL_BF16;
    const int max_cot = umma_max_cot(T, s.elem_bytes);           // T planes x CoT fp32 TMEM columns <= 512
    s.nTiles = (Cout + max_cot - 1) / max_cot;
    const int per = (Cout + s.nTiles - 1) / s.nTiles;
    const int gran = T == 2 ? 32 : 16;                          // the epilogue drains 128 output bytes (64 / T channels) at a time
    s.CoT = (per + gran - 1) / gran * gran;
    const int kch = kRowBytes / s.elem_bytes;                    // channels per chunk (one UMMA K step)
    const int ks = umma_chunks_per_stage(T, s.elem_bytes, false);   // (the same for the pair form of every T that has one)
    s.nK = ((Cin + kch - 1) / kch + ks - 1) / ks * ks;         // whole stages: the padding chunks hold zero channels
    s.rowsB = (2 * T - 2) * s.CoT;
    s.image_bytes = align_up((size_t)s.nTiles * s.nK * s.rowsB * kRowBytes * (s.elem_bytes == 4 ? 2 : 1), kWsAlign);
    s.cin0 = 0; s.CinTotal = Cin;
    return s;
}

int umma_reduction_segments(int Cin, eql_dtype_t dtype, int* seg_len) {
    if (dtype != EQL_FP32 || Cin <= kFp32SegmentChannels) { *seg_len = Cin; return 1; }
    const int want = (Cin + kFp32SegmentChannels - 1) / kFp32SegmentChannels;
    const int len = ((Cin + want - 1) / want + 15) / 16 * 16;
    *seg_len = len;
    return (Cin + len - 1) / len;
}

UmmaLinearShape umma_linear_segment(int T, int Cin, int Cout, eql_dtype_t dtype, int k, int seg_len) {
    const int c0 = k * seg_len;
    UmmaLinearShape s = umma_linear_shape(T, Cin - c0 < seg_len ? Cin - c0 : seg_len, Cout, dtype);
    s.cin0 = c0; s.CinTotal = Cin;
    return s;
}

size_t umma_linear_image_bytes(int T, int Cin, int Cout, eql_dtype_t dtype) {
    int len = 0;
    const int n = umma_reduction_segments(Cin, dtype, &len);
    size_t total = 0;
    for (int k = 0; k < n; ++k) total += umma_linear_segment(T, Cin, Cout, dtype, k, len).image_bytes;
    return total;
}

cudaError_t launch_build_umma_image(const UmmaLinearShape& s, const float* planes, void* image, cudaStream_t stream) {
    return dispatch_umma(s.T, s.elem_bytes, [&](auto tc, auto io) {
        constexpr int TT = decltype(tc)::value;
        using IO = decltype(io);
        const int64_t total = (int64_t)(s.image_bytes / sizeof(IO));
        const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
        build_image_kernel<TT, IO><<<blocks, 256, 0, stream>>>(planes, s.Cin, s.Cout, s.CoT, s.nTiles, s.nK, s.rowsB,
                                                                (IO*)image, s.cin0, s.CinTotal, s.pair ? 1 : 0);
        return cudaGetLastError();
    }, s.bf16);
}

cudaError_t launch_umma_linear(const UmmaLinearShape& s, const void* in, void* out, int64_t N, const void* image,
                               const float* bias_f32, int* status, int num_sms, cudaStream_t stream, bool accumulate) {
    if (accumulate && s.elem_bytes != 4) return cudaErrorInvalidValue;       // the reduce-add path exists for float outputs
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return cudaErrorNotSupported;
    const CUtensorMapDataType dt = s.elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    const cuuint32_t epr = 128 / s.elem_bytes;                   // elements per 128-byte slab row
    CUtensorMap tmap, tmap_out;
    const cuuint32_t estr[2] = {1, 1};
    {
        // a segment of the reduction sees only its own columns of the rows (the rest reads as zero fill)
        const cuuint64_t gdim[2] = {(cuuint64_t)s.Cin * s.T, (cuuint64_t)N};
        const cuuint64_t gstr[1] = {(cuuint64_t)s.CinTotal * s.T * s.elem_bytes};
        const cuuint32_t box[2] = {epr, (cuuint32_t)kTileM};
        const char* in_seg = (const char*)in + (size_t)s.cin0 * s.T * s.elem_bytes;
        if (enc(&tmap, dt, 2, const_cast<char*>(in_seg), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t odim[2] = {(cuuint64_t)s.Cout * s.T, (cuuint64_t)N};
        const cuuint64_t ostr[1] = {(cuuint64_t)s.Cout * s.T * s.elem_bytes};
        const cuuint32_t obox[2] = {epr, 32};
        if (enc(&tmap_out, dt, 2, out, odim, ostr, obox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    UmmaParams prm{};
    prm.out = out; prm.image = (const uint8_t*)image; prm.bias = bias_f32; prm.status = status;
    prm.N = N; prm.Cin = s.Cin; prm.Cout = s.Cout;
    prm.CoT = s.CoT; prm.nTiles = s.nTiles; prm.nK = s.nK; prm.rowsB = s.rowsB;
    const int cg = s.pair ? 2 : 1;
    prm.b_slot_bytes = (int)align_up((size_t)(s.rowsB / cg) * kRowBytes * (s.elem_bytes == 4 ? 2 : 1) *
                                         umma_chunks_per_stage(s.T, s.elem_bytes, s.pair), 256);
    const int64_t token_tiles = (N + kTileM - 1) / kTileM;
    prm.num_units = ((token_tiles + cg - 1) / cg) * s.nTiles;    // a pair takes two token tiles per unit
    prm.accumulate = accumulate ? 1 : 0;
    prm.act = s.act;

    return dispatch_umma(s.T, s.elem_bytes, [&](auto tc, auto io) {
        constexpr int TT = decltype(tc)::value;
        using IO = decltype(io);
        if (s.pair) {
            if constexpr (sizeof(IO) == 2 && (TT == 4 || TT == 8)) {
                const size_t smem = umma_smem_bytes<TT, 2, 2>(prm.b_slot_bytes);
                if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
                static SmemLimitOnce smem_limit[2];
                auto kernel = prm.act ? umma_linear_kernel<TT, IO, 2, true> : umma_linear_kernel<TT, IO, 2, false>;
                if (cudaError_t e = smem_limit[prm.act ? 1 : 0].ensure(kernel, 227 * 1024); e != cudaSuccess) return e;
                cudaLaunchConfig_t cfg{};
                cudaLaunchAttribute attr[2];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
                attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // see ptx::grid_dependency_wait
                attr[1].val.programmaticStreamSerializationAllowed = 1;
                cfg.blockDim = dim3(kThreadsUmma); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
                cfg.attrs = attr; cfg.numAttrs = 2;
                // persistent: as many pairs as can be resident at once (pairs need two SMs of one GPC), at most one per unit
                static std::atomic<int> max_pairs{0};
                int pairs = max_pairs.load(std::memory_order_relaxed);
                if (pairs == 0) {
                    cfg.gridDim = dim3(2 * (num_sms / 2));
                    if (cudaError_t e = cudaOccupancyMaxActiveClusters(&pairs, kernel, &cfg); e != cudaSuccess) return e;
                    if (pairs <= 0) return cudaErrorInvalidConfiguration;
                    if (pairs > num_sms / 2) pairs = num_sms / 2;
                    max_pairs.store(pairs, std::memory_order_relaxed);
                }
                if (prm.num_units < pairs) pairs = (int)prm.num_units;
                cfg.gridDim = dim3(2 * pairs);
                return cudaLaunchKernelEx(&cfg, kernel, tmap, tmap_out, prm);
            } else {
                return cudaErrorInvalidConfiguration;
            }
        } else {
            const int grid = (int)(prm.num_units < num_sms ? prm.num_units : num_sms);
            const size_t smem = umma_smem_bytes<TT, sizeof(IO), 1>(prm.b_slot_bytes);
            if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
            if (prm.act) {
                static SmemLimitOnce smem_limit_act;              // per kernel instantiation
                if (cudaError_t e = smem_limit_act.ensure(umma_linear_kernel<TT, IO, 1, true>, 227 * 1024); e != cudaSuccess) return e;
                return launch_overlapped(umma_linear_kernel<TT, IO, 1, true>, dim3(grid), dim3(kThreadsUmma), smem, stream, tmap, tmap_out, prm);
            }
            static SmemLimitOnce smem_limit;                      // per kernel instantiation
            if (cudaError_t e = smem_limit.ensure(umma_linear_kernel<TT, IO, 1, false>, 227 * 1024); e != cudaSuccess) return e;
            return launch_overlapped(umma_linear_kernel<TT, IO, 1, false>, dim3(grid), dim3(kThreadsUmma), smem, stream, tmap, tmap_out, prm);
        }
    }, s.bf16);
}

bool umma_linear_pair_supported(int T, eql_dtype_t dtype) { return (dtype == EQL_FP16 || dtype == EQL_BF16) && (T == 4 || T == 8); }

}  // namespace eql
