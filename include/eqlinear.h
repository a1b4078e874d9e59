/*
 * eqlinear.h -- C ABI of the Flash EQ-Linear hot path for NVIDIA B200 (sm_100a).
 *
 * The operator (Eq. 1 of the paper; circular-convolution reading of Eq. 3-5 and Eq. 19-21):
 *
 *     y[n, o, t] = bias[o] + sum_{i < C_in} sum_{s < T}  w[o, i, (t - s) mod T] * x[n, i, s]
 *
 * i.e. an ordinary linear layer whose dense weight is block-circulant over a cyclic group of
 * order T.  The library never forms that dense weight: it evaluates Algorithm 1 -- a real DFT
 * along the group axis, one complex channel-mixing product per retained frequency
 * k = 0..floor(T/2), and the inverse real DFT plus bias -- for the forward pass and for both
 * gradients.
 *
 * Conventions common to every entry point
 *   - Features are dense row-major [N, C*T] with the group index fastest: element (n, c, t) is at
 *     n*C*T + c*T + t.  The weight is [C_out, C_in, T] with the group offset r fastest; the bias
 *     is [C_out].
 *   - x, y, dy, dx, w and bias have the plan's dtype (EQL_FP32: float; EQL_FP16: IEEE half, EQL_BF16: bfloat16,
 *     both with float accumulation).  dw and db are always float.
 *   - Every tensor pointer is DEVICE memory owned by the caller, 16-byte aligned; outputs must not
 *     alias inputs.  The *_host entry points are the only ones that take host pointers.
 *   - The library allocates no device memory.  The plan keeps its derived weights in a
 *     caller-owned device workspace; eqlinear_bwd_weight uses a caller-owned device scratch buffer.
 *     Both must stay valid (and untouched by the caller) while in use.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls are
 *     asynchronous on that stream and never synchronise the device, except where stated.
 *   - Errors are return codes.  Argument errors are detected on the host before any launch.
 *     N == 0 is a successful no-op.  Nothing traps or aborts on the device.
 *   - A plan may be used from one stream at a time, and only while the device it was built on is the
 *     current device: every entry point that takes a plan returns EQL_ERR_INVALID_ARG, before any
 *     launch, when another device is current.  Different plans may be used from different host threads.
 */
#ifndef EQLINEAR_H_
#define EQLINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eqlinear_plan_s* eqlinear_plan_t;   /* opaque host object */

typedef enum {
    EQL_OK = 0,
    EQL_ERR_INVALID_ARG = 1,      /* NULL pointer, negative size, bad enum                    */
    EQL_ERR_UNSUPPORTED = 2,      /* group order or channel count outside the supported set   */
    EQL_ERR_ALIGNMENT = 3,        /* pointer not 16-byte aligned, or row bytes not multiple of 16 */
    EQL_ERR_WORKSPACE = 4,        /* workspace / scratch / staging buffer too small           */
    EQL_ERR_ARCH = 5,             /* current device is not compute capability 10.x            */
    EQL_ERR_CUDA = 6,             /* a CUDA runtime or driver call failed                      */
    EQL_ERR_DEVICE_TIMEOUT = 7    /* a bounded wait inside a kernel ran out                    */
} eql_status_t;

/* EQL_FP16 / EQL_BF16: 16-bit I/O (IEEE half / bfloat16) with float accumulation; the spectra of the activations and of
 * the weight are rounded to the same 16-bit type once, everything else is float. */
typedef enum { EQL_FP32 = 0, EQL_FP16 = 1, EQL_BF16 = 2 } eql_dtype_t;

/* Plan flags. */
enum {
    /* Use the index (s - t) mod T printed in Eq. 1-2 (circular correlation) instead of the
     * (t - s) mod T of Eq. 3-5 / Eq. 19-21.  Costs nothing at run time (the weight spectrum is
     * conjugated when the plan is built). */
    EQL_FLAG_CORRELATION = 1u,
    /* Force the CUDA-core (FFMA) kernels even where a tensor-core kernel exists. */
    EQL_FLAG_FORCE_SIMT = 2u,
    /* Among the tensor-core kernels, always take the streaming one (activations transformed per
     * output-channel tile) even where the kernel that keeps the transformed activations of a token
     * tile resident in shared memory applies.  For comparisons and tests. */
    EQL_FLAG_FORCE_STREAMING = 4u,
    /* The streaming kernel has a CTA-pair form (FP16 plans, T = 4 or 8): clusters of two CTAs on two SMs work on
     * neighbouring token tiles, one tcgen05.mma.cta_group::2 covers both, and each SM loads and holds only half of
     * every spectral-weight tile.  Same results bit for bit.  Plans take it by themselves for wide layers (512 or
     * more channels per group element on both sides), where it measures 2-10 % faster; below it measures 2-4 %
     * slower.  EQL_FLAG_CTA_PAIR takes it wherever it exists, EQL_FLAG_NO_CTA_PAIR never (comparisons, tests). */
    EQL_FLAG_CTA_PAIR = 8u,
    EQL_FLAG_NO_CTA_PAIR = 16u,
    /* Forward pass only: apply GELU (exact form, x * Phi(x)) to every output element in the epilogue, in FP32, before
     * the result is rounded and stored -- the fc1 -> GELU pair of a transformer MLP block as one kernel (a pointwise
     * map applied to each group element alike keeps the layer equivariant).  For inference: eqlinear_bwd_data and
     * eqlinear_bwd_weight remain the gradients of the LINEAR layer; a caller that trains multiplies dy by GELU'(pre-
     * activation) itself and therefore needs the unfused forward.  EQL_ERR_UNSUPPORTED for FP32 plans on the tensor
     * cores with more than 256 input channels (their forward sums segments in global memory). */
    EQL_FLAG_GELU = 32u,
    /* The group is the DIHEDRAL group D_T (the T rotations of the cyclic group and their T reflections, order 2T) --
     * the reflection extension the paper's Conclusion names as future work.  T is the number of rotations (2, 3, 4, 5,
     * 6 or 8); features are [N, C * 2T] and the weight [C_out, C_in, 2T] with the group index g = f*T + t fastest
     * (element r^t s^f: rotation t, reflection flag f; s r = r^-1 s), and the layer is the group convolution
     *     y[n, o, g] = bias[o] + sum_i sum_h w[o, i, h^-1 g] x[n, i, h],
     * whose restriction to the rotations is the cyclic layer.  Algorithm 1 carries over with the group's irreducible
     * representations in place of the DFT frequencies (one- and two-dimensional real blocks); the kernels run on the
     * CUDA cores.  Not combinable with EQL_FLAG_CORRELATION, EQL_FLAG_FORCE_STREAMING or EQL_FLAG_CTA_PAIR.
     * Size the workspace with eqlinear_workspace_bytes_flags. */
    EQL_FLAG_DIHEDRAL = 64u
};

typedef struct {
    int32_t T, C_in, C_out, dtype;
    uint32_t flags;
    int32_t fwd_kernel;           /* 0 = CUDA-core FFMA kernel, 1 = tcgen05 streaming kernel,
                                     2 = tcgen05 kernel with resident transformed activations,
                                     3 = tcgen05 streaming kernel run by CTA pairs (cta_group::2) */
    int32_t bwd_data_kernel;
    int32_t bwd_weight_kernel;
    int64_t macs_per_token;       /* Step-2 multiply-accumulates of Algorithm 1 per token, exact count */
    int64_t dense_macs_per_token; /* the naive dense layer's: (C_out*T)*(C_in*T)               */
    int64_t bytes_per_token_fwd;  /* algorithmic HBM bytes per token of fwd: (C_in + C_out)*T*elem */
    int64_t bytes_per_token_bwd_data;
    int64_t bytes_per_token_bwd_weight;
    size_t  workspace_bytes;
} eql_info_t;

/* ---- host-only helpers (no GPU needed) ------------------------------------------------------ */

/* Text for a status code; never NULL. */
const char* eqlinear_status_string(eql_status_t status);

/* Multiply-accumulate counts for N tokens.  Step 2 of Algorithm 1 costs one real product per real
 * frequency plane (k = 0 and, for even T, k = T/2) and four per complex one, so for even T
 *   spectral = (2T - 2) * N * C_in * C_out   (6/16 of dense at T = 4, Theorem 1),
 * for odd T (2T - 1) * N * C_in * C_out; dense = N * (C_out*T) * (C_in*T) (Eq. 1).
 * Either output pointer may be NULL. */
eql_status_t eqlinear_count_macs(int T, int C_in, int C_out, int64_t N,
                                 int64_t* spectral_macs, int64_t* dense_macs);

/* Size in bytes of the device workspace a plan of this shape needs. */
eql_status_t eqlinear_workspace_bytes(int T, int C_in, int C_out, eql_dtype_t dtype, size_t* bytes);

/* The same for a plan built with `flags` (EQL_FLAG_DIHEDRAL changes the tuple length and hence the size). */
eql_status_t eqlinear_workspace_bytes_flags(int T, int C_in, int C_out, eql_dtype_t dtype, unsigned flags, size_t* bytes);

/* ---- plan (Algorithm 1, step 1 for the weight: the spectral weight, computed once) ---------- */

/* Build a plan on the current device: validates the shape, takes the group DFT of w (Eq. 4),
 * and stores the frequency planes of w -- in the operand layouts of the forward and of the
 * conjugate-transposed data-gradient product, with the 1/T of the inverse DFT folded in -- and a
 * copy of the bias in `workspace`.
 *   T            group order: 1 to 8, 12, 16 or 32 (Algorithm 1 holds for every cyclic group; the paper's own kernels
 *                cover T = 4).  Powers of two from 4 run on the tensor cores (T = 2: forward and data gradient of
 *                16-bit plans), the other orders -- odd ones included -- on CUDA-core kernels with a table-driven real DFT
 *   C_in, C_out  channels per group element, >= 1; C_in*T*elem and C_out*T*elem must be
 *                multiples of 16 bytes
 *   w            device, [C_out, C_in, T], plan dtype
 *   bias         device, [C_out], plan dtype, or NULL for no bias
 *   workspace    device, 256-byte aligned, at least eqlinear_workspace_bytes() bytes; owned by the
 *                caller, used by the plan until eqlinear_plan_destroy
 * The weight transform is enqueued on `stream`; later calls on the same stream see it.
 * On error *plan is set to NULL. */
eql_status_t eqlinear_plan(eqlinear_plan_t* plan, int T, int C_in, int C_out, eql_dtype_t dtype,
                           const void* w, const void* bias,
                           void* workspace, size_t workspace_bytes,
                           unsigned flags, void* stream);

/* Recompute the spectral weight from new parameter values (after an optimiser step).
 * bias == NULL keeps "no bias" only if the plan was built without one (else INVALID_ARG). */
eql_status_t eqlinear_plan_set_weight(eqlinear_plan_t plan, const void* w, const void* bias, void* stream);

eql_status_t eqlinear_plan_info(eqlinear_plan_t plan, eql_info_t* info);

/* Kernel launches ONE call of each entry point makes for N tokens with this plan (launch accounting for
 * benchmarks; no GPU work): counts[0] eqlinear_fwd, counts[1] eqlinear_bwd_data, counts[2] eqlinear_bwd_weight
 * (or eqlinear_bwd_weight_from_spectrum), counts[3] the launches eqlinear_fwd_save_spectrum adds to eqlinear_fwd.
 * More than one launch per call occurs for FP32 plans only: reductions over more than 256 channels run as
 * segments, long token ranges of the weight gradient as blocks (the plan's FP32 semantics, see eqlinear_plan). */
eql_status_t eqlinear_plan_launch_counts(eqlinear_plan_t plan, int64_t N, int32_t counts[4]);

/* Reads the plan's device status word (synchronises `stream`): EQL_OK, or
 * EQL_ERR_DEVICE_TIMEOUT if a bounded wait inside one of the plan's kernels gave up. */
eql_status_t eqlinear_plan_device_status(eqlinear_plan_t plan, void* stream);

/* Sets the plan's device status word back to "ok" (asynchronous on `stream`), e.g. after a reported time-out. */
eql_status_t eqlinear_plan_clear_device_status(eqlinear_plan_t plan, void* stream);

/* Self-test of that error path: launches (asynchronously on `stream`) a one-warp kernel whose single bounded wait -
 * the helper every tensor-core kernel of the library waits with - is never satisfied.  The kernel ends by itself
 * after its poll budget (tens of milliseconds), nothing faults, and eqlinear_plan_device_status then reports
 * EQL_ERR_DEVICE_TIMEOUT until the status is cleared; the plan stays usable. */
eql_status_t eqlinear_plan_selftest_expired_wait(eqlinear_plan_t plan, void* stream);

/* Frees the host object only (the workspace is the caller's). NULL is accepted. */
eql_status_t eqlinear_plan_destroy(eqlinear_plan_t plan);

/* ---- the hot path ---------------------------------------------------------------------------- */

/* Forward (Algorithm 1, steps 1-4; Eq. 4-7): y = circular-convolution layer of x, plus bias.
 *   x  device [N, C_in*T]   y  device [N, C_out*T]   both plan dtype, N >= 0 tokens. */
eql_status_t eqlinear_fwd(eqlinear_plan_t plan, const void* x, void* y, int64_t N, void* stream);

/* Gradient with respect to the input: the same Fourier-domain decomposition with the conjugate
 * transposed spectral weight, dx^_k = dy^_k . conj(w^_k) (appendix, "Forward and backward passes").
 *   dy device [N, C_out*T]   dx device [N, C_in*T]. */
eql_status_t eqlinear_bwd_data(eqlinear_plan_t plan, const void* dy, void* dx, int64_t N, void* stream);

/* Bytes of device scratch eqlinear_bwd_weight needs for N tokens with this plan. */
eql_status_t eqlinear_bwd_weight_scratch_bytes(eqlinear_plan_t plan, int64_t N, size_t* bytes);

/* Gradients with respect to the original parameters (appendix, "Forward and backward passes"):
 *   dw^_k[o, i] = sum_n dy^_k[n, o] * conj(x^_k[n, i]),  dw = inverse group DFT of dw^ (with 1/T),
 *   db[o] = sum_n sum_t dy[n, o, t].
 *   x device [N, C_in*T], dy device [N, C_out*T] (plan dtype);
 *   dw device [C_out, C_in, T] float;  db device [C_out] float or NULL;
 *   scratch device, 256-byte aligned, >= eqlinear_bwd_weight_scratch_bytes(); holds the per-split
 *   partial spectra between the two kernels of this call; contents are undefined afterwards.
 * dw and db are overwritten (not accumulated into); with N == 0 they are set to zero.
 * The reduction order is fixed, so results are bit-reproducible run to run. */
eql_status_t eqlinear_bwd_weight(eqlinear_plan_t plan, const void* x, const void* dy,
                                 void* dw, void* db, int64_t N,
                                 void* scratch, size_t scratch_bytes, void* stream);

/* ---- training with a saved spectrum (FP16 / BF16 plans whose weight gradient runs on the tensor cores) --
 * Algorithm 1 transforms x once for the forward pass; the weight gradient needs the same spectrum
 * x^ again, and computing it there is the largest share of that kernel's instructions (every
 * output-channel tile repeats it).  These three calls let the forward pass save x^ -- rounded to
 * the plan's 16-bit type, in the operand layout of the weight-gradient kernel -- so that the weight gradient reads it
 * back instead of x.  (The paper's kernels keep no frequency-domain tensor in global memory; this
 * is an optional trade of N*C_in*T*2 bytes of device memory and one extra write of that size for a
 * shorter backward pass.)  The buffer's layout is private to the library; it is valid for the plan
 * and N it was written with. */

/* Bytes of the saved-spectrum buffer for N tokens.  EQL_ERR_UNSUPPORTED for plans without this path
 * (FP32 plans, EQL_FLAG_FORCE_SIMT). */
eql_status_t eqlinear_spectrum_bytes(eqlinear_plan_t plan, int64_t N, size_t* bytes);

/* eqlinear_fwd that also writes the spectrum of x.
 *   spectrum: device, 256-byte aligned, >= eqlinear_spectrum_bytes(plan, N). */
eql_status_t eqlinear_fwd_save_spectrum(eqlinear_plan_t plan, const void* x, void* y, int64_t N,
                                        void* spectrum, size_t spectrum_bytes, void* stream);

/* eqlinear_bwd_weight with the saved spectrum in place of x (same outputs, same scratch size, same
 * fixed reduction order).  N must be the N of the eqlinear_fwd_save_spectrum call that wrote it. */
eql_status_t eqlinear_bwd_weight_from_spectrum(eqlinear_plan_t plan, const void* spectrum, size_t spectrum_bytes,
                                               const void* dy, void* dw, void* db, int64_t N,
                                               void* scratch, size_t scratch_bytes, void* stream);

/* Size of the scratch array that is built into the library for eqlinear_bwd_weight_static. */
#define EQL_STATIC_SCRATCH_BYTES (32u << 20)

/* eqlinear_bwd_weight without a scratch argument.  (The paper has no counterpart: this entry point
 * exists for the library's users, not for the method.)
 *
 * Who it is for: code that must compute the weight gradient at a point where it cannot obtain
 * device memory -- a plug-in running inside a host application that owns the allocator and gives
 * the plug-in none, a service whose memory pool has already claimed the whole GPU so that a fresh
 * cudaMalloc would fail, or a latency-critical loop that may not risk the device-wide stall an
 * allocation can cause.  Such callers still pass their inputs and outputs (x, dy, dw, db, as for
 * eqlinear_bwd_weight); only the scratch for the per-split partial spectra comes from the library,
 * from a fixed device array of EQL_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library image.
 * This call allocates nothing and frees nothing.
 *
 *   - When the 32 MiB become resident: CUDA loads the parts of a library lazily, and the array's part
 *     is loaded on a GPU the first time the array's address is looked up there.  eqlinear_plan does
 *     that look-up for its device, so building the first plan on a GPU is what reserves the array
 *     (once per GPU, until the process exits) -- do it while device memory can still be had, i.e.
 *     before a pool claims the rest of the GPU.  After that no call of this entry point loads,
 *     reserves or looks up anything: free device memory is the same before and after it.
 *   - Returns EQL_ERR_WORKSPACE, and launches nothing, when eqlinear_bwd_weight_scratch_bytes(plan, N)
 *     is larger than EQL_STATIC_SCRATCH_BYTES; use eqlinear_bwd_weight with your own buffer then.
 *   - The array's device address is looked up once per device, by eqlinear_plan (with the plan's
 *     device current).  Should that look-up have failed, this call repeats it and returns
 *     EQL_ERR_CUDA if it fails again; build plans, and so do the look-up, before any stream capture
 *     begins.  The plan's device must be the current device (EQL_ERR_INVALID_ARG otherwise).
 *   - All calls, from every plan and stream, share the one array, and it keeps whatever the last
 *     call left in it.  Nothing in it has to start at zero: each call overwrites every partial it
 *     later reads.  Two calls that overlap in time on the GPU race on it; order them on one stream
 *     (or with events).
 *   - Results are identical to eqlinear_bwd_weight's for the same plan and N. */
eql_status_t eqlinear_bwd_weight_static(eqlinear_plan_t plan, const void* x, const void* dy,
                                        void* dw, void* db, int64_t N, void* stream);

/* ---- host-buffer variants (end-to-end measurement, small-batch convenience) ------------------ */
/* Same operations with HOST input/output buffers (pinned memory recommended).  Each call copies
 * its inputs into the caller's device staging buffers, runs the kernels above and copies the
 * results back, all asynchronously; the host buffers may be read once `stream` has been
 * synchronised.  Staging buffers are device memory with the sizes of the corresponding
 * device-variant tensors.
 * eqlinear_fwd_host and eqlinear_step_host move batches of 8192 tokens or more in up to sixteen token
 * chunks through a three-stream pipeline (host -> device copies, kernels on `stream`, device -> host
 * copies), so that both copy directions and the kernels overlap; `stream` waits for the last copy
 * before the call's remaining work.  The two extra streams and their events belong to the plan:
 * created at the first such call, destroyed by eqlinear_plan_destroy (no device memory). */
eql_status_t eqlinear_fwd_host(eqlinear_plan_t plan, const void* x_host, void* y_host, int64_t N,
                               void* x_staging, void* y_staging, void* stream);
eql_status_t eqlinear_bwd_data_host(eqlinear_plan_t plan, const void* dy_host, void* dx_host, int64_t N,
                                    void* dy_staging, void* dx_staging, void* stream);
eql_status_t eqlinear_bwd_weight_host(eqlinear_plan_t plan, const void* x_host, const void* dy_host,
                                      void* dw_host, void* db_host, int64_t N,
                                      void* x_staging, void* dy_staging, void* dw_staging, void* db_staging,
                                      void* scratch, size_t scratch_bytes, void* stream);

/* One whole training step of the layer from host buffers: copies x and dy to the device once, runs
 * eqlinear_fwd, eqlinear_bwd_data and eqlinear_bwd_weight, and copies y, dx, dw and db back, all
 * asynchronously on `stream` (N > 0).  db_host / db_staging may both be NULL. */
eql_status_t eqlinear_step_host(eqlinear_plan_t plan, const void* x_host, const void* dy_host,
                                void* y_host, void* dx_host, void* dw_host, void* db_host, int64_t N,
                                void* x_staging, void* dy_staging, void* y_staging, void* dx_staging,
                                void* dw_staging, void* db_staging,
                                void* scratch, size_t scratch_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* EQLINEAR_H_ */
