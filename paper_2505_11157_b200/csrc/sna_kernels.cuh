// Device-side view of a plan and the launchers of the CUDA kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace sna {

// All pointers are device memory owned by the plan.
struct DevPlan {
    int nlat_in, nlon_in, nlat_out, nlon_out, ps;
    // forward table, run-length form: windows [row_ptr[h], row_ptr[h+1]) of output latitude h
    const int32_t* row_ptr;
    const int32_t* win_lat;     // input ring
    const int32_t* win_m;       // half width in input columns, -1 = whole ring
    const int32_t* row_order;   // output latitudes, most table entries first
    // transposed table: windows [t_row_ptr[h'], t_row_ptr[h'+1]) of input latitude h'
    const int32_t* t_row_ptr;
    const int32_t* t_win_lat;   // output ring
    const int32_t* t_win_m;
    const int32_t* t_row_order; // input latitudes, most work first
    const float* log2_omega;    // [nlat_in] log2 of the per-point quadrature weight
    // column streams of the tensor-core kernels (see sna_plan.hpp); null if not built
    const int4* fwd_stream;         // 16 entries per chunk: {base|abs flag, e | mask<<16, bias, aux}
    const int32_t* fwd_chunk_ptr;   // [groups of output latitudes + 1]
    const int32_t* grp_order;       // groups of output latitudes, longest stream first
    // band-only forward stream (whole-ring and wide windows left to the dense kernel) and the dense kernel's lists
    const int4* fwdb_stream;
    const int32_t* fwdb_chunk_ptr;
    const int32_t* grpb_order;
    const int32_t* dense_ptr;       // [nlat_out+1] the dense kernels' windows per output latitude
    const int32_t* dense_lat;       // their input rings
    const int32_t* dense_m;         // their half widths in input columns, -1 = whole ring
    const int32_t* dense_rows;      // output latitudes with at least one such window
    int n_dense_rows;
    // the same for the transposed side (dk/dv): band-only transposed stream and, per input latitude, the output rings
    // that attend to it as a whole
    const int4* tb_stream;
    const int32_t* tb_chunk_ptr;
    const int32_t* tb_grp_order;
    const int32_t* t_dense_ptr;     // [nlat_in+1]
    const int32_t* t_dense_lat;     // output rings
    const int32_t* t_dense_m;       // half widths in input columns, -1 = whole ring
    const int32_t* t_dense_rows;    // input latitudes with at least one such output ring
    int n_t_dense_rows;
    float dense_fraction;           // share of the table's entries that the dense kernels' windows cover
    int* dev_status;                // set to non-zero by a kernel whose bounded wait ran out
    const int4* t_stream;
    const int32_t* t_chunk_ptr;     // [groups of input latitudes * ps + 1]
    const int32_t* t_grp_order;     // groups of input latitudes, longest stream first
    int t_consecutive;              // 1: transposed tiles are 8 consecutive input columns; 0: split by residue mod ps
    int is_global;                  // 1: every window is a whole ring and no column stream exists (dense kernels or generic kernels only)
};

// Tensor-core kernels (C = 16, 32 or 64, nlon_out >= 32); same contracts as the generic launchers.
cudaError_t mma_prepare_device();   // once per device: opt in to the kernels' shared-memory sizes
bool mma_path_supported(const DevPlan& p, int C);
// Reduced-precision variant of the three kernels: every product is one TF32 MMA (relative product error ~2^-11).
cudaError_t launch_forward_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                  int N, int C, cudaStream_t stream);
cudaError_t launch_backward_dq_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                      const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream);
cudaError_t launch_backward_dkdv_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                        const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream);
cudaError_t launch_forward_mma(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                               int N, int C, cudaStream_t stream);
// Dense (tcgen05) kernels (sna_kernels_dense2.cu: TMA loads, warp-specialised, operands and accumulators in TMEM) for
// the windows in the plan's dense lists: whole input rings, and wide banded windows as masked blocks.  The forward kernel
// writes the partial result (normalised out, lse) of the output latitudes in p.dense_rows and launch_forward_mma_band
// continues from it with the narrower windows; both need lse != null.  dense2_path_supported tells whether the pair may
// be used for this problem.
cudaError_t dense2_prepare_device();   // once per device: opt in to the kernels' shared-memory sizes
bool dense2_path_supported(const DevPlan& p, int C);
cudaError_t launch_bounded_wait_probe(const DevPlan& p, int polls, cudaStream_t stream);
bool dense2_global_supported(const DevPlan& p, int C);   // every window is a whole ring and the dense kernels can do all the work
cudaError_t launch_forward_dense2(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                  int N, int C, cudaStream_t stream);
// The same split for the dq stage: the dense kernel writes its part of dq (out and dq must be different buffers) and,
// if Dws != null, D; the band kernel adds the narrower windows' part.
cudaError_t launch_backward_dq_dense2(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                      const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream);
// And for dk/dv: the dense kernel writes its part for the input latitudes in p.t_dense_rows, the band kernel adds the rest.
cudaError_t launch_backward_dkdv_dense2(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                        const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream);
cudaError_t launch_backward_dq_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                        const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream);
cudaError_t launch_backward_dkdv_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                          const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream);
cudaError_t launch_forward_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                    int N, int C, cudaStream_t stream);
// out is required (D_i = dout_i . out_i); out and dq may be the same buffer.
cudaError_t launch_backward_dq_mma(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                   const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream);
cudaError_t launch_backward_dkdv_mma(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                     const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream);

// Layout changes (sna_kernels_layout.cu): [slices][C][P] channels first <-> [slices][P][C] channels last, slices <= 65535.
cudaError_t launch_cf_to_cl(const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream);
cudaError_t launch_cl_to_cf(const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream);

// Generic kernels (any supported C): C/4 lanes cooperate on one grid point.
// forward: out and/or lse may be null (lse-only pass = softmax statistics).
cudaError_t launch_forward_generic(const DevPlan& p, const float* q, const float* k, const float* v, float* out,
                                   float* lse, int N, int C, cudaStream_t stream);
// dq pass.  lse is required.  If out != null, D_i = dout_i . out_i is used; otherwise D_i is accumulated.
// Writes dq and Dws[i] = D_i.
cudaError_t launch_backward_dq_generic(const DevPlan& p, const float* q, const float* k, const float* v,
                                       const float* dout, const float* out, const float* lse, float* dq, float* Dws,
                                       int N, int C, cudaStream_t stream);
// dk, dv gather pass over the transposed table; needs lse and D of every output point.
cudaError_t launch_backward_dkdv_generic(const DevPlan& p, const float* q, const float* k, const float* v,
                                         const float* dout, const float* lse, const float* Dws, float* dk, float* dv,
                                         int N, int C, cudaStream_t stream);

}  // namespace sna
