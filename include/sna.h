/*
 * sna.h — C ABI of the spherical neighborhood attention library for NVIDIA B200 (sm_100a).
 *
 * The operator (paper: "Attention on the Sphere", arXiv 2505.11157):
 *
 *   out[n,h,w,:] = sum_j alpha_j v_j / sum_j alpha_j ,   alpha_j = exp(q[n,h,w,:] . k_j / sqrt(C)) * omega_j
 *
 * where j runs over the input grid points inside the geodesic disc of radius theta_cutoff around the
 * output point (h, w) (Eq. s2_neighborhood_attention), omega_j is the quadrature weight of the input
 * point (Eq. quadrature), and the discrete form is Eq. s2_attention_discrete_detailed of App. B.3.
 * The backward pass returns the gradients of App. B.4 with respect to q, k and v.
 *
 * Conventions that hold for every call:
 *   - No exception crosses this boundary; every call returns an sna_status_t (0 = success).
 *   - "host" pointers are ordinary CPU memory owned by the caller; "device" pointers are CUDA global
 *     memory on the device that was current when the plan was created, owned by the caller.
 *   - Tensors are contiguous fp32, channels last, batch and heads leading:
 *         q, out, dout, dq : [B][H][nlat_out][nlon_out][C]
 *         k, v, dk, dv     : [B][H][nlat_in ][nlon_in ][C]
 *         lse, and each half of the workspace : [B][H][nlat_out][nlon_out]
 *     Device pointers must be 16-byte aligned.  B*H heads are independent problems.
 *   - C must be a multiple of 4 between 4 and 128 (SNA_ERR_UNSUPPORTED otherwise).
 *   - Compute calls must be made with the plan's device current; otherwise they return SNA_ERR_INVALID_ARG and
 *     launch nothing.
 *   - Compute calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*; NULL is the
 *     default stream) and return without synchronising.  They validate arguments on the host first and
 *     launch nothing if validation fails.  Outputs are overwritten, never accumulated into.
 *   - A plan is immutable after creation and may be used from several streams at once, as long as
 *     calls that run concurrently do not share a workspace (see sna_backward).
 *   - Accuracy: results are fp32; against an fp64 evaluation of the same formulas the normalised maximum
 *     error max|x - ref| / max|ref| per tensor is below 1e-5 for out and below 1e-4 for dq, dk, dv
 *     (measured 2e-6 and 2e-5).  No atomics are used: the same call on the same inputs gives the same bits.
 */
#ifndef SNA_H
#define SNA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sna_plan sna_plan_t; /* opaque; created and destroyed by the library */

typedef enum {
    SNA_OK = 0,
    SNA_ERR_INVALID_ARG = 1,        /* null pointer, non-positive size, NaN or non-positive cutoff, misaligned pointer */
    SNA_ERR_UNSUPPORTED = 2,        /* nlon_in not a multiple of nlon_out; unsupported C; unknown grid */
    SNA_ERR_EMPTY_NEIGHBORHOOD = 3, /* some output latitude has no input point inside its disc */
    SNA_ERR_ALLOC = 4,              /* host or device allocation failed */
    SNA_ERR_CUDA = 5,               /* a CUDA call or launch failed; see sna_last_error_message */
    SNA_ERR_AMBIGUOUS_TIE = 6,      /* a point lies within 1e-8 rad of the disc boundary without being on it */
    SNA_ERR_WORKSPACE = 7           /* caller-supplied workspace or static scratch too small */
} sna_status_t;

typedef enum {
    /* theta_h = pi*h/(nlat-1), h = 0..nlat-1: both poles are grid rings; Clenshaw-Curtis latitude weights.
     * (The equiangular grid of App. A.1, Eq. latlon_grid, with the pole-including variant of the rule.) */
    SNA_GRID_EQUIANGULAR = 0,
    /* "Gaussian grid" (Sec. 3.3): theta_h = arccos(x_h), x_h the roots of the Legendre polynomial P_nlat in
     * descending order (north to south), Gauss-Legendre weights. */
    SNA_GRID_LEGENDRE_GAUSS = 1,
    /* The equiangular grid exactly as App. A.1 prints it (Eq. latlon_grid, Eq. latlon_quad_weights):
     * theta_h = pi*h/nlat, h = 0..nlat-1 (north pole a ring, south pole not), point weights
     * 2 pi^2/(nlat nlon) sin(theta_h): the trapezoid rule in theta, summing to 4 pi only approximately.  The pole
     * ring has weight zero: its points are listed by the table queries but contribute to no output, and their
     * dk / dv are zero.  A theta_cutoff so small that the pole output point sees only the pole ring leaves that
     * output undefined (0/0) and is refused with SNA_ERR_EMPTY_NEIGHBORHOOD. */
    SNA_GRID_EQUIANGULAR_TRAPEZOID = 2
} sna_grid_t;

/*
 * Build a plan: colatitudes of both grids, fp64 quadrature weights omega[h'] = w_lat[h'] * 2*pi/nlon_in of the
 * input grid (Eq. quadrature; they sum to 4*pi over all points), and the neighborhood table of App. B.3: for
 * every output latitude h the set of (lat_in, lon_off) with geodesic distance between the output point
 * (h, longitude 0) and the input point (lat_in, lon_off) at most theta_cutoff.  Because the grids are invariant
 * under rotation about the pole the same row serves every output longitude w: the input column is
 * (lon_off + w*ps) mod nlon_in with ps = nlon_in / nlon_out.
 *
 * Points exactly on the disc boundary are members: the test is d <= theta_cutoff + 1e-10, and a point with
 * 1e-12 < |d - theta_cutoff| < 1e-8 makes creation fail with SNA_ERR_AMBIGUOUS_TIE rather than letting rounding
 * decide.  theta_cutoff >= pi selects every input point.
 *
 * The plan's tables are copied to the current CUDA device; the plan must be used and destroyed with that
 * device.  *plan_out is written only on success.  nlat_* >= 2, nlon_* >= 1, nlon_in % nlon_out == 0.
 */
sna_status_t sna_plan_create(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                             sna_grid_t grid_in, sna_grid_t grid_out, double theta_cutoff,
                             sna_plan_t** plan_out);

/*
 * Plan for GLOBAL spherical attention (Eq. s2_attention_discrete; App. B.1-B.2): every output point attends to every
 * input point, i.e. softmax attention over the whole input grid with the additive bias log omega_j.  Equivalent to
 * sna_plan_create with theta_cutoff >= pi, but no per-pair structure is built or stored: the plan holds only the grids,
 * the quadrature weights and the per-ring lists the dense tensor-core kernels walk.  All compute calls accept it; with
 * C = 32 they run entirely on the dense tcgen05 kernels (the forward pass then needs an lse buffer, and the backward
 * pass runs fastest with out and lse from sna_forward_ex); other shapes use the generic kernels.
 */
sna_status_t sna_plan_create_global(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                                    sna_grid_t grid_in, sna_grid_t grid_out, sna_plan_t** plan_out);

/* Same construction, but nothing is copied to a GPU and no CUDA call is made: the plan serves the
 * introspection calls below only (compute calls on it return SNA_ERR_INVALID_ARG).  For inspecting or
 * validating tables on a machine without a GPU. */
sna_status_t sna_plan_create_host_only(int nlat_in, int nlon_in, int nlat_out, int nlon_out,
                                       sna_grid_t grid_in, sna_grid_t grid_out, double theta_cutoff,
                                       sna_plan_t** plan_out);

/* Free the plan's host and device memory (including a workspace it may have grown).  NULL is accepted. */
sna_status_t sna_plan_destroy(sna_plan_t* plan);

/* Waits for the plan's device to finish and reports whether any kernel launched through this plan gave up on one of
 * its bounded waits (SNA_ERR_CUDA; its outputs would be incomplete).  Kernels never spin without limit; this is the
 * way to find out that a limit was hit.  Not expected to happen.  A failure is reported once: the call that returns
 * SNA_ERR_CUDA also clears the record, so outputs written since the previous check must be recomputed. */
sna_status_t sna_plan_check(const sna_plan_t* plan);

/* Test aid for that failure path.  Launches, on the given stream, one tiny kernel in which a single thread waits on a
 * barrier that nothing ever arrives on, using the same bounded wait routine as the tensor-core kernels but limited to
 * `polls` polls (1..100000; each poll suspends for at most about 2 microseconds).  The wait runs out, the kernel
 * records that in the plan's status word and returns normally: no trap, no fault, the context stays usable.  The next
 * sna_plan_check reports SNA_ERR_CUDA once and clears the word; compute calls on the plan work before and after. */
sna_status_t sna_debug_exercise_bounded_wait(const sna_plan_t* plan, int polls, void* cuda_stream);

/* ---- introspection into caller-owned HOST buffers ------------------------------------------------------ */

/* Number of (lat_in, lon_off) entries in the table. */
sna_status_t sna_plan_get_nnz(const sna_plan_t* plan, int64_t* nnz);
/* theta_in[nlat_in], theta_out[nlat_out] in radians; either pointer may be NULL. */
sna_status_t sna_plan_get_colatitudes(const sna_plan_t* plan, double* theta_in, double* theta_out);
/* omega_in[nlat_in]: per-point quadrature weight of each input ring. */
sna_status_t sna_plan_get_quad_weights(const sna_plan_t* plan, double* omega_in);
/* CSR table in canonical order: rows = output latitudes, entries sorted by lat_in, then lon_off in [0, nlon_in).
 * row_ptr[nlat_out+1], lat_in[nnz], lon_off[nnz]. */
sna_status_t sna_plan_get_table(const sna_plan_t* plan, int64_t* row_ptr, int32_t* lat_in, int32_t* lon_off);
/* Transposed table used by the backward pass: row (lat_in*ps + r) lists, for input columns congruent to r
 * modulo ps, the pairs (lat_out, lon_off) of the forward table with lat_in in them and lon_off % ps == r,
 * sorted by lat_out, then lon_off.  The output longitude is w = ((column - lon_off) mod nlon_in) / ps.
 * row_ptr[nlat_in*ps+1], lat_out[nnz], lon_off[nnz]. */
sna_status_t sna_plan_get_table_transposed(const sna_plan_t* plan, int64_t* row_ptr, int32_t* lat_out,
                                           int32_t* lon_off);

/* ---- compute -------------------------------------------------------------------------------------------- */

/* Bytes of device workspace sna_backward_ex needs for this problem size (two fp32 values per output point,
 * rounded up to 256 bytes).  Returns 0 for invalid arguments. */
size_t sna_workspace_bytes(const sna_plan_t* plan, int B, int H, int C);

/* Forward pass (Eq. s2_attention_discrete_detailed).  q, k, v, out: device. */
sna_status_t sna_forward(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                         int B, int H, int C, void* cuda_stream);

/* Number of GPU kernels sna_forward_ex launches for this plan and channel count (with_lse != 0: an lse buffer is
 * passed).  1, or 2 when whole-ring and wide windows take the dense tensor-core kernel first.  0 for invalid arguments. */
int sna_forward_kernel_count(const sna_plan_t* plan, int C, int with_lse);

/* Forward pass that also stores lse[n,h,w] = log(sum_j exp(s_j) omega_j) (device, may be NULL), which the
 * backward pass can reuse. */
sna_status_t sna_forward_ex(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                            float* lse, int B, int H, int C, void* cuda_stream);

/*
 * Backward pass (App. B.4): given dout = dL/dout, writes dq, dk, dv (device, all three required).
 * With p_j = alpha_j / sum_l alpha_l, t_j = dout_i . v_j, D_i = sum_j p_j t_j:
 *     dq_i = (1/sqrt(C)) sum_j p_j (t_j - D_i) k_j
 *     dk_j = (1/sqrt(C)) sum_{i: j in disc(i)} p_ij (t_ij - D_i) q_i        dv_j = sum_{i: j in disc(i)} p_ij dout_i
 * dk and dv are gathered per input point over the transposed table; no atomics are used, so results are
 * reproducible bit for bit.  This form recomputes the softmax statistics and keeps them in a workspace owned
 * by the plan, which is (re)allocated with cudaMalloc when a call needs a larger one than any call before —
 * such a call synchronises the device.  Two sna_backward calls on the same plan must not overlap on the GPU.
 */
sna_status_t sna_backward(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                          const float* dout, float* dq, float* dk, float* dv,
                          int B, int H, int C, void* cuda_stream);

/*
 * Backward pass with caller-supplied state.  out and lse (device) are the results of sna_forward_ex on the same
 * q, k, v; either may be NULL, in which case the statistics it would provide are recomputed.  workspace is
 * device memory of at least sna_workspace_bytes(plan, B, H, C) bytes, 256-byte aligned, private to this call
 * until the call's work on the stream has finished.  Never allocates.
 */
sna_status_t sna_backward_ex(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                             const float* dout, const float* out, const float* lse,
                             float* dq, float* dk, float* dv,
                             void* workspace, size_t workspace_bytes,
                             int B, int H, int C, void* cuda_stream);

/*
 * The two stages of sna_backward_ex as separate calls, for callers that want to overlap or time them.
 *
 * sna_backward_dq: dq of App. B.4 (quotient-rule form) for every output point, plus D[n,h,w] = sum_j p_j t_j,
 * which the second stage needs.  lse (device, required) is the forward pass's lse; out (device) may be NULL.
 * D is device memory of B*H*nlat_out*nlon_out floats, written by this call.
 *
 * sna_backward_dkdv: dk and dv gathered per input point over the transposed table, from lse and D.
 */
sna_status_t sna_backward_dq(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                             const float* dout, const float* out, const float* lse, float* dq, float* D,
                             int B, int H, int C, void* cuda_stream);
sna_status_t sna_backward_dkdv(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                               const float* dout, const float* lse, const float* D, float* dk, float* dv,
                               int B, int H, int C, void* cuda_stream);

/*
 * Channels-first entry points.  The paper states its tensors as B x C x H x W (App. B.3); with heads, tensor x_cf
 * has the layout [B][H*C][nlat][nlon], i.e. channel c of head h of batch b is the plane (b*H + h)*C + c, while every
 * other call of this header takes channels-last arrays [B][H][nlat][nlon][C].  These two calls change the layout on the
 * GPU (tiled transposes, HBM-bound: each element read once and written once) around sna_forward_ex / sna_backward_ex:
 *
 *   sna_forward_cf   q_cf, k_cf, v_cf -> out_cf; leaves the channels-last q, k, v, out and lse in `state` (device,
 *                    sna_cf_state_bytes, 256-byte aligned, caller-owned) for the backward pass;
 *   sna_backward_cf  dout_cf and that state -> dq_cf, dk_cf, dv_cf; `scratch` (device, sna_cf_scratch_bytes, 256-byte
 *                    aligned) is private to the call until its work on the stream has finished.
 *
 * B*H must not exceed 65535.  Neither call allocates.  Errors as for sna_forward_ex / sna_backward_ex, plus
 * SNA_ERR_WORKSPACE for a state or scratch buffer that is too small.  The size queries return 0 for invalid arguments.
 */
size_t sna_cf_state_bytes(const sna_plan_t* plan, int B, int H, int C);
size_t sna_cf_scratch_bytes(const sna_plan_t* plan, int B, int H, int C);
sna_status_t sna_forward_cf(const sna_plan_t* plan, const float* q_cf, const float* k_cf, const float* v_cf, float* out_cf,
                            void* state, size_t state_bytes, int B, int H, int C, void* cuda_stream);
sna_status_t sna_backward_cf(const sna_plan_t* plan, const float* dout_cf, const void* state, size_t state_bytes,
                             void* scratch, size_t scratch_bytes, float* dq_cf, float* dk_cf, float* dv_cf,
                             int B, int H, int C, void* cuda_stream);

/*
 * Reduced-precision variant of the forward and backward pass.  The paper lists "neither reduced precision nor tensor
 * core" support as a limitation of its kernels (Sec. 5, Limitations); here every contraction of
 * Eq. s2_attention_discrete_detailed and App. B.4 is taken as ONE TF32 tensor-core product (operands rounded to 11
 * significand bits, fp32 accumulation, fp32 softmax) instead of the error-compensated products of the default path.
 * Same arguments, layouts and semantics as sna_forward_ex / sna_backward_ex.  Accuracy: normalised maximum error
 * max|x - ref| / max|ref| per tensor below 5e-3 against an fp64 evaluation (measured ~1e-3); about 1.5x faster.
 * Needs C in {16, 32, 64} and nlon_out >= 32 (SNA_ERR_UNSUPPORTED otherwise).
 */
sna_status_t sna_forward_tf32(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                              float* lse, int B, int H, int C, void* cuda_stream);
sna_status_t sna_backward_tf32(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                               const float* dout, const float* out, const float* lse,
                               float* dq, float* dk, float* dv,
                               void* workspace, size_t workspace_bytes,
                               int B, int H, int C, void* cuda_stream);

/*
 * Backward pass for callers that must not allocate device memory.  (The paper has no counterpart; this is a
 * packaging variant of sna_backward.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they need gradients: code running
 * inside a memory-pool or arena that owns the whole device, real-time loops where an allocation (and the
 * device synchronisation it implies) is not acceptable, or plug-ins that are only handed input and output
 * buffers.  sna_backward needs scratch memory for the per-output-point softmax statistics (lse and D);
 * here that scratch is a fixed array that is part of the library image itself, so neither this call nor
 * anything it uses calls cudaMalloc, cudaFree or any allocating routine.
 *
 * Limit: the array holds the statistics of at most SNA_STATIC_SCRATCH_MAX_POINTS output points
 * (B*H*nlat_out*nlon_out); it occupies 8 MiB on every GPU that loads the library, until the process exits.
 * A larger problem is rejected with SNA_ERR_WORKSPACE and nothing is launched.
 *
 * Arguments, layouts and results are those of sna_backward.  Things to know:
 *   - The first call on each device looks up the array's device address (once per device, with that device
 *     current).  Make that first call outside any CUDA stream capture.
 *   - Every call on a device uses the same array.  Nothing in it has to start at zero (both halves are fully
 *     rewritten before they are read), and it keeps the last call's values afterwards.  Two calls whose GPU
 *     work overlaps (different streams, or several host threads) race on it: serialise them.
 */
#define SNA_STATIC_SCRATCH_MAX_POINTS (1 << 20)
sna_status_t sna_backward_static(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                                 const float* dout, float* dq, float* dk, float* dv,
                                 int B, int H, int C, void* cuda_stream);

/*
 * Measurement aid (the paper has no counterpart): runs a pure FP32 fused-multiply-add loop on every SM of the
 * current device and returns the sustained rate in TFLOP/s (2 flops per FMA) in *tflops (host).  It is the
 * denominator check for the roofline, which is stated against the FP32 FMA peak (SMs x 128 lanes x 2 x clock).
 * Blocks until the probe has finished (about a millisecond); allocates a few KB of device memory for its result.
 */
sna_status_t sna_measure_fp32_fma_peak(double* tflops);

/* Human-readable name of a status code (static string). */
const char* sna_status_string(sna_status_t status);
/* Detail of the most recent failure on the calling thread (static thread-local buffer; "" if none). */
const char* sna_last_error_message(void);

#ifdef __cplusplus
}
#endif
#endif /* SNA_H */
