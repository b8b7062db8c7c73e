// C ABI of the library (declared in include/sna.h): plan life cycle, introspection and the compute entry
// points.  Host-side validation happens here; kernels live in the other translation units.
#include "../../include/sna.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <numeric>
#include <string>
#include <vector>

#include "sna_kernels.cuh"
#include "sna_plan.hpp"

namespace {

thread_local char g_last_error[512] = "";

void set_error(const char* fmt, ...) __attribute__((format(printf, 1, 2)));
void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
}

sna_status_t cuda_fail(cudaError_t e, const char* what) {
    set_error("%s: %s", what, cudaGetErrorString(e));
    return SNA_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

struct sna_plan {
    sna::HostPlan host;
    sna::DevPlan dev{};
    int device = 0;
    std::vector<int> zero_rings;       // input rings of quadrature weight zero (no kernel of a global plan visits them)
    bool is_global = false;            // created by sna_plan_create_global: no column streams, dense kernels only
    void* dev_blob = nullptr;          // one allocation holding every device table
    mutable std::mutex ws_mutex;
    mutable void* ws = nullptr;        // workspace grown on demand by sna_backward
    mutable size_t ws_bytes = 0;
};

namespace {

bool supported_C(int C) { return C >= 4 && C <= 128 && C % 4 == 0; }

sna_status_t check_problem(const sna_plan_t* plan, int B, int H, int C) {
    if (plan == nullptr) { set_error("plan is NULL"); return SNA_ERR_INVALID_ARG; }
    if (plan->dev_blob == nullptr) { set_error("plan was created host-only; it cannot compute"); return SNA_ERR_INVALID_ARG; }
    if (B <= 0 || H <= 0 || C <= 0) { set_error("B, H and C must be positive"); return SNA_ERR_INVALID_ARG; }
    if (!supported_C(C)) { set_error("C=%d unsupported (a multiple of 4 between 4 and 128)", C); return SNA_ERR_UNSUPPORTED; }
    // The plan's tables, and by contract the caller's tensors, live on the device the plan was created on; launching
    // with another device current would hand that device foreign addresses.
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != plan->device) {
        set_error("the current CUDA device (%d) is not the plan's device (%d)", current, plan->device);
        return SNA_ERR_INVALID_ARG;
    }
    const long long N = (long long)B * H;
    const long long big = std::max((long long)plan->host.nlat_in * plan->host.nlon_in,
                                   (long long)plan->host.nlat_out * plan->host.nlon_out);
    if (N > 0x7fffffffLL || N * big > 0x7fffffffLL) { set_error("problem too large: B*H*nlat*nlon must fit in 31 bits"); return SNA_ERR_UNSUPPORTED; }
    return SNA_OK;
}

template <typename... P>
bool all_aligned(P... ptrs) { return (aligned16(ptrs) && ...); }

size_t stats_elems(const sna_plan_t* plan, int B, int H) {
    return (size_t)B * H * plan->host.nlat_out * plan->host.nlon_out;
}
size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" {

const char* sna_status_string(sna_status_t s) {
    switch (s) {
        case SNA_OK: return "SNA_OK";
        case SNA_ERR_INVALID_ARG: return "SNA_ERR_INVALID_ARG";
        case SNA_ERR_UNSUPPORTED: return "SNA_ERR_UNSUPPORTED";
        case SNA_ERR_EMPTY_NEIGHBORHOOD: return "SNA_ERR_EMPTY_NEIGHBORHOOD";
        case SNA_ERR_ALLOC: return "SNA_ERR_ALLOC";
        case SNA_ERR_CUDA: return "SNA_ERR_CUDA";
        case SNA_ERR_AMBIGUOUS_TIE: return "SNA_ERR_AMBIGUOUS_TIE";
        case SNA_ERR_WORKSPACE: return "SNA_ERR_WORKSPACE";
    }
    return "SNA_ERR_UNKNOWN";
}

const char* sna_last_error_message(void) { return g_last_error; }

// Measured on the benchmark configurations (fwd+bwd, against whole rings only): 128 gives -4 % at 361x720, -1.5 % at
// 128x256 and -0.7 % on the 2:1 down-sampling case; 96 and below lose, because a masked 128-row block uses at most
// W / (ps * 127 + W) of its entries.
constexpr int DENSE_MIN_WIDTH = 128;

static sna_status_t plan_create(int nlat_in, int nlon_in, int nlat_out, int nlon_out, sna_grid_t grid_in,
                                sna_grid_t grid_out, double theta_cutoff, bool upload, sna_plan_t** plan_out,
                                bool global = false) {
    if (plan_out == nullptr) { set_error("plan_out is NULL"); return SNA_ERR_INVALID_ARG; }
    sna_plan* plan = new (std::nothrow) sna_plan();
    if (plan == nullptr) { set_error("out of host memory"); return SNA_ERR_ALLOC; }
    std::string why;
    sna::PlanStatus ps;
    try {
        ps = sna::build_plan(nlat_in, nlon_in, nlat_out, nlon_out, (int)grid_in, (int)grid_out, theta_cutoff, plan->host, why);
    } catch (const std::bad_alloc&) {
        delete plan;
        set_error("out of host memory while building the table");
        return SNA_ERR_ALLOC;
    }
    if (ps != sna::PLAN_OK) {
        delete plan;
        set_error("%s", why.c_str());
        return ps == sna::PLAN_INVALID ? SNA_ERR_INVALID_ARG : ps == sna::PLAN_UNSUPPORTED ? SNA_ERR_UNSUPPORTED
             : ps == sna::PLAN_EMPTY ? SNA_ERR_EMPTY_NEIGHBORHOOD : SNA_ERR_AMBIGUOUS_TIE;
    }
    if (!upload) { *plan_out = plan; return SNA_OK; }
    // the kernels walk the table without rings of weight zero; plan->host keeps every member for the table queries
    sna::HostPlan weighted;
    const bool dropped = sna::drop_zero_weight_rings(plan->host, weighted);
    const sna::HostPlan& hp = dropped ? weighted : plan->host;
    for (int h = 0; h < hp.nlat_in; ++h) if (!(hp.omega[h] > 0.0)) plan->zero_rings.push_back(h);
    // heavy-first orders
    std::vector<int32_t> row_order(hp.nlat_out), t_row_order(hp.nlat_in);
    std::iota(row_order.begin(), row_order.end(), 0);
    std::iota(t_row_order.begin(), t_row_order.end(), 0);
    std::stable_sort(row_order.begin(), row_order.end(), [&](int a, int b) { return hp.row_nnz[a] > hp.row_nnz[b]; });
    std::stable_sort(t_row_order.begin(), t_row_order.end(), [&](int a, int b) { return hp.t_row_nnz[a] > hp.t_row_nnz[b]; });
    std::vector<int32_t> win_lat(hp.windows.size()), win_m(hp.windows.size()), t_lat(hp.t_windows.size()), t_m(hp.t_windows.size());
    for (size_t i = 0; i < hp.windows.size(); ++i) { win_lat[i] = hp.windows[i].lat; win_m[i] = hp.windows[i].m; }
    for (size_t i = 0; i < hp.t_windows.size(); ++i) { t_lat[i] = hp.t_windows[i].lat; t_m[i] = hp.t_windows[i].m; }
    std::vector<float> log2_omega(hp.nlat_in);
    for (int h = 0; h < hp.nlat_in; ++h) log2_omega[h] = (float)std::log2(hp.omega[h]);

    sna::Stream fwd_stream, t_stream, fwdb_stream, tb_stream;
    sna::DenseLists dense, t_dense;
    std::vector<int32_t> grp_order, t_grp_order, grpb_order, tb_grp_order;
#ifdef SNA_PROF
    const int32_t zero_status[512] = {};   // room for the per-role profile of a -DSNA_PROF build
#else
    const int32_t zero_status[64] = {};
#endif
    bool t_consecutive = false;
    plan->is_global = global;
    // Windows at least this many input columns wide (and whole rings) run on the dense tcgen05 kernels, as masked blocks;
    // narrower ones stay on the band kernels, whose 8-column tiles waste less on a slanted band.
    const int dense_min_width = DENSE_MIN_WIDTH;
    try {
        sna::build_dense_lists(hp, dense, dense_min_width);
        sna::build_transposed_dense_lists(hp, t_dense, dense_min_width);
        // rows with the longest lists first: the dense kernels run one block per SM, so the long tiles must not start last
        std::stable_sort(dense.rows.begin(), dense.rows.end(), [&](int a, int b) { return dense.ptr[a + 1] - dense.ptr[a] > dense.ptr[b + 1] - dense.ptr[b]; });
        std::stable_sort(t_dense.rows.begin(), t_dense.rows.end(), [&](int a, int b) { return t_dense.ptr[a + 1] - t_dense.ptr[a] > t_dense.ptr[b + 1] - t_dense.ptr[b]; });
        if (global) {
            // every window is a whole ring: the dense kernels do all the work, so the column streams (which would list
            // every pair of the dense problem) are not built; they stay empty and the band kernels are never launched
            const size_t g_out = (hp.nlat_out + sna::TILE_LAT - 1) / sna::TILE_LAT, g_in = (hp.nlat_in + sna::TILE_LAT - 1) / sna::TILE_LAT;
            fwd_stream.chunk_ptr.assign(g_out + 1, 0);
            fwdb_stream.chunk_ptr.assign(g_out + 1, 0);
            t_stream.chunk_ptr.assign(g_in + 1, 0);
            tb_stream.chunk_ptr.assign(g_in + 1, 0);
            t_consecutive = true;
            grp_order.resize(g_out);
            std::iota(grp_order.begin(), grp_order.end(), 0);
            grpb_order = grp_order;
        } else {
        sna::build_forward_stream(hp, fwd_stream);
        t_consecutive = sna::build_transposed_stream(hp, t_stream);
        sna::build_forward_stream(hp, fwdb_stream, dense_min_width);
        grpb_order.resize(fwdb_stream.chunk_ptr.size() - 1);
        std::iota(grpb_order.begin(), grpb_order.end(), 0);
        std::stable_sort(grpb_order.begin(), grpb_order.end(), [&](int a, int b) {
            return fwdb_stream.chunk_ptr[a + 1] - fwdb_stream.chunk_ptr[a] > fwdb_stream.chunk_ptr[b + 1] - fwdb_stream.chunk_ptr[b];
        });
        // heavy-first orders of the ring groups (by stream length; for the transposed stream summed over residues)
        grp_order.resize(fwd_stream.chunk_ptr.size() - 1);
        std::iota(grp_order.begin(), grp_order.end(), 0);
        std::stable_sort(grp_order.begin(), grp_order.end(), [&](int a, int b) {
            return fwd_stream.chunk_ptr[a + 1] - fwd_stream.chunk_ptr[a] > fwd_stream.chunk_ptr[b + 1] - fwd_stream.chunk_ptr[b];
        });
        sna::build_transposed_stream(hp, tb_stream, dense_min_width);
        }
        const int rows_per_group = t_consecutive ? 1 : hp.ps;
        tb_grp_order.resize((tb_stream.chunk_ptr.size() - 1) / rows_per_group);
        std::iota(tb_grp_order.begin(), tb_grp_order.end(), 0);
        std::stable_sort(tb_grp_order.begin(), tb_grp_order.end(), [&](int a, int b) {
            return tb_stream.chunk_ptr[(a + 1) * rows_per_group] - tb_stream.chunk_ptr[a * rows_per_group] >
                   tb_stream.chunk_ptr[(b + 1) * rows_per_group] - tb_stream.chunk_ptr[b * rows_per_group];
        });
        t_grp_order.resize((t_stream.chunk_ptr.size() - 1) / rows_per_group);
        std::iota(t_grp_order.begin(), t_grp_order.end(), 0);
        std::stable_sort(t_grp_order.begin(), t_grp_order.end(), [&](int a, int b) {
            return t_stream.chunk_ptr[(a + 1) * rows_per_group] - t_stream.chunk_ptr[a * rows_per_group] >
                   t_stream.chunk_ptr[(b + 1) * rows_per_group] - t_stream.chunk_ptr[b * rows_per_group];
        });
    } catch (const std::bad_alloc&) {
        delete plan;
        set_error("out of host memory while building the column streams");
        return SNA_ERR_ALLOC;
    }
    static_assert(sizeof(sna::StreamEntry) == 16, "stream entries are read as int4");

    // pack everything into one device allocation (each array 256-byte aligned)
    struct Piece { const void* src; size_t bytes; size_t offset; };
    std::vector<Piece> pieces = {
        {hp.row_ptr.data(), hp.row_ptr.size() * 4, 0}, {win_lat.data(), win_lat.size() * 4, 0}, {win_m.data(), win_m.size() * 4, 0},
        {row_order.data(), row_order.size() * 4, 0}, {hp.t_row_ptr.data(), hp.t_row_ptr.size() * 4, 0}, {t_lat.data(), t_lat.size() * 4, 0},
        {t_m.data(), t_m.size() * 4, 0}, {t_row_order.data(), t_row_order.size() * 4, 0}, {log2_omega.data(), log2_omega.size() * 4, 0},
        {fwd_stream.entries.data(), fwd_stream.entries.size() * 16, 0}, {fwd_stream.chunk_ptr.data(), fwd_stream.chunk_ptr.size() * 4, 0},
        {t_stream.entries.data(), t_stream.entries.size() * 16, 0}, {t_stream.chunk_ptr.data(), t_stream.chunk_ptr.size() * 4, 0},
        {grp_order.data(), grp_order.size() * 4, 0}, {t_grp_order.data(), t_grp_order.size() * 4, 0},
        {fwdb_stream.entries.data(), fwdb_stream.entries.size() * 16, 0}, {fwdb_stream.chunk_ptr.data(), fwdb_stream.chunk_ptr.size() * 4, 0},
        {grpb_order.data(), grpb_order.size() * 4, 0}, {dense.ptr.data(), dense.ptr.size() * 4, 0},
        {dense.lat.data(), dense.lat.size() * 4, 0}, {dense.rows.data(), dense.rows.size() * 4, 0}, {zero_status, sizeof(zero_status), 0},
        {tb_stream.entries.data(), tb_stream.entries.size() * 16, 0}, {tb_stream.chunk_ptr.data(), tb_stream.chunk_ptr.size() * 4, 0},
        {tb_grp_order.data(), tb_grp_order.size() * 4, 0}, {t_dense.ptr.data(), t_dense.ptr.size() * 4, 0},
        {t_dense.lat.data(), t_dense.lat.size() * 4, 0}, {t_dense.rows.data(), t_dense.rows.size() * 4, 0},
        {dense.m.data(), dense.m.size() * 4, 0}, {t_dense.m.data(), t_dense.m.size() * 4, 0}};
    size_t total = 0;
    for (Piece& p : pieces) { p.offset = total; total += round256(p.bytes); }
    cudaError_t e = cudaGetDevice(&plan->device);
    if (e != cudaSuccess) { delete plan; return cuda_fail(e, "cudaGetDevice"); }
    e = cudaMalloc(&plan->dev_blob, total);
    if (e != cudaSuccess) { delete plan; set_error("cudaMalloc of %zu bytes: %s", total, cudaGetErrorString(e)); return SNA_ERR_ALLOC; }
    for (const Piece& p : pieces) {
        if (p.bytes == 0) continue;
        e = cudaMemcpy((char*)plan->dev_blob + p.offset, p.src, p.bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { cudaFree(plan->dev_blob); delete plan; return cuda_fail(e, "cudaMemcpy of plan tables"); }
    }
    auto at = [&](int i) { return (const int32_t*)((char*)plan->dev_blob + pieces[i].offset); };
    sna::DevPlan& d = plan->dev;
    d.nlat_in = hp.nlat_in; d.nlon_in = hp.nlon_in; d.nlat_out = hp.nlat_out; d.nlon_out = hp.nlon_out; d.ps = hp.ps;
    d.row_ptr = at(0); d.win_lat = at(1); d.win_m = at(2); d.row_order = at(3);
    d.t_row_ptr = at(4); d.t_win_lat = at(5); d.t_win_m = at(6); d.t_row_order = at(7);
    d.log2_omega = (const float*)at(8);
    d.fwd_stream = (const int4*)at(9); d.fwd_chunk_ptr = at(10);
    d.t_stream = (const int4*)at(11); d.t_chunk_ptr = at(12);
    d.grp_order = at(13); d.t_grp_order = at(14);
    d.t_consecutive = t_consecutive ? 1 : 0;
    d.fwdb_stream = (const int4*)at(15); d.fwdb_chunk_ptr = at(16); d.grpb_order = at(17);
    d.dense_ptr = at(18); d.dense_lat = at(19); d.dense_rows = at(20);
    d.n_dense_rows = (int)dense.rows.size();
    d.dense_fraction = hp.nnz > 0 ? (float)((double)dense.pairs / (double)hp.nnz) : 0.f;
    d.is_global = global ? 1 : 0;
    d.dev_status = (int*)((char*)plan->dev_blob + pieces[21].offset);
    d.tb_stream = (const int4*)at(22); d.tb_chunk_ptr = at(23); d.tb_grp_order = at(24);
    d.t_dense_ptr = at(25); d.t_dense_lat = at(26); d.t_dense_rows = at(27);
    d.n_t_dense_rows = (int)t_dense.rows.size();
    d.dense_m = at(28); d.t_dense_m = at(29);
    // opt in to the kernels' dynamic shared-memory sizes on this device (once here instead of on every launch)
    e = sna::dense2_prepare_device();
    if (e == cudaSuccess) e = sna::mma_prepare_device();
    if (e != cudaSuccess) { sna_plan_destroy(plan); return cuda_fail(e, "cudaFuncSetAttribute"); }
    *plan_out = plan;
    return SNA_OK;
}

sna_status_t sna_plan_create(int nlat_in, int nlon_in, int nlat_out, int nlon_out, sna_grid_t grid_in,
                             sna_grid_t grid_out, double theta_cutoff, sna_plan_t** plan_out) {
    return plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, true, plan_out);
}

sna_status_t sna_plan_create_global(int nlat_in, int nlon_in, int nlat_out, int nlon_out, sna_grid_t grid_in,
                                    sna_grid_t grid_out, sna_plan_t** plan_out) {
    // theta_cutoff = pi selects every input point for every output point; no distance is evaluated
    return plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, 3.14159265358979323846, true, plan_out, true);
}

sna_status_t sna_plan_create_host_only(int nlat_in, int nlon_in, int nlat_out, int nlon_out, sna_grid_t grid_in,
                                       sna_grid_t grid_out, double theta_cutoff, sna_plan_t** plan_out) {
    return plan_create(nlat_in, nlon_in, nlat_out, nlon_out, grid_in, grid_out, theta_cutoff, false, plan_out);
}

sna_status_t sna_plan_destroy(sna_plan_t* plan) {
    if (plan == nullptr) return SNA_OK;
    cudaError_t e1 = plan->dev_blob ? cudaFree(plan->dev_blob) : cudaSuccess;
    cudaError_t e2 = plan->ws ? cudaFree(plan->ws) : cudaSuccess;
    delete plan;
    if (e1 != cudaSuccess) return cuda_fail(e1, "cudaFree");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaFree");
    return SNA_OK;
}

sna_status_t sna_plan_check(const sna_plan_t* plan) {
    if (!plan) { set_error("plan is NULL"); return SNA_ERR_INVALID_ARG; }
    if (plan->dev_blob == nullptr) return SNA_OK;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    int status = 0;
    e = cudaMemcpy(&status, plan->dev.dev_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy of the device status word");
    if (status != 0) {
        // reported once: the word is cleared so that the plan can be used (and checked) again
        e = cudaMemset(plan->dev.dev_status, 0, sizeof(int));
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemset of the device status word");
        set_error("a kernel gave up on a bounded wait; its outputs are incomplete");
        return SNA_ERR_CUDA;
    }
    return SNA_OK;
}

sna_status_t sna_debug_exercise_bounded_wait(const sna_plan_t* plan, int polls, void* cuda_stream) {
    if (!plan || plan->dev_blob == nullptr) { set_error("needs a plan that lives on a GPU"); return SNA_ERR_INVALID_ARG; }
    if (polls < 1 || polls > 100000) { set_error("polls must be between 1 and 100000"); return SNA_ERR_INVALID_ARG; }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != plan->device) { set_error("the plan's device is not current"); return SNA_ERR_INVALID_ARG; }
    cudaError_t e = sna::launch_bounded_wait_probe(plan->dev, polls, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "probe launch");
    return SNA_OK;
}

sna_status_t sna_plan_get_nnz(const sna_plan_t* plan, int64_t* nnz) {
    if (!plan || !nnz) { set_error("NULL argument"); return SNA_ERR_INVALID_ARG; }
    *nnz = plan->host.nnz;
    return SNA_OK;
}

sna_status_t sna_plan_get_colatitudes(const sna_plan_t* plan, double* theta_in, double* theta_out) {
    if (!plan) { set_error("plan is NULL"); return SNA_ERR_INVALID_ARG; }
    if (theta_in) std::memcpy(theta_in, plan->host.theta_in.data(), sizeof(double) * plan->host.nlat_in);
    if (theta_out) std::memcpy(theta_out, plan->host.theta_out.data(), sizeof(double) * plan->host.nlat_out);
    return SNA_OK;
}

sna_status_t sna_plan_get_quad_weights(const sna_plan_t* plan, double* omega_in) {
    if (!plan || !omega_in) { set_error("NULL argument"); return SNA_ERR_INVALID_ARG; }
    std::memcpy(omega_in, plan->host.omega.data(), sizeof(double) * plan->host.nlat_in);
    return SNA_OK;
}

sna_status_t sna_plan_get_table(const sna_plan_t* plan, int64_t* row_ptr, int32_t* lat_in, int32_t* lon_off) {
    if (!plan || !row_ptr || !lat_in || !lon_off) { set_error("NULL argument"); return SNA_ERR_INVALID_ARG; }
    const sna::HostPlan& hp = plan->host;
    int64_t n = 0;
    for (int h = 0; h < hp.nlat_out; ++h) {
        row_ptr[h] = n;
        for (int e = hp.row_ptr[h]; e < hp.row_ptr[h + 1]; ++e) {
            const sna::RingWindow& w = hp.windows[e];
            // canonical order: offsets ascending in [0, nlon_in): 0..m first, then nlon_in-m..nlon_in-1
            if (w.m < 0) {
                for (int o = 0; o < hp.nlon_in; ++o) { lat_in[n] = w.lat; lon_off[n++] = o; }
            } else {
                for (int o = 0; o <= w.m; ++o) { lat_in[n] = w.lat; lon_off[n++] = o; }
                for (int o = hp.nlon_in - w.m; o < hp.nlon_in; ++o) { lat_in[n] = w.lat; lon_off[n++] = o; }
            }
        }
    }
    row_ptr[hp.nlat_out] = n;
    return SNA_OK;
}

sna_status_t sna_plan_get_table_transposed(const sna_plan_t* plan, int64_t* row_ptr, int32_t* lat_out, int32_t* lon_off) {
    if (!plan || !row_ptr || !lat_out || !lon_off) { set_error("NULL argument"); return SNA_ERR_INVALID_ARG; }
    const sna::HostPlan& hp = plan->host;
    int64_t n = 0;
    for (int hin = 0; hin < hp.nlat_in; ++hin) {
        for (int r = 0; r < hp.ps; ++r) {
            row_ptr[(int64_t)hin * hp.ps + r] = n;
            for (int e = hp.t_row_ptr[hin]; e < hp.t_row_ptr[hin + 1]; ++e) {
                const sna::RingWindow& w = hp.t_windows[e];
                auto emit = [&](int lo, int hi) {
                    for (int o = lo; o <= hi; ++o)
                        if (o % hp.ps == r) { lat_out[n] = w.lat; lon_off[n++] = o; }
                };
                if (w.m < 0) emit(0, hp.nlon_in - 1);
                else { emit(0, w.m); emit(hp.nlon_in - w.m, hp.nlon_in - 1); }
            }
        }
    }
    row_ptr[(int64_t)hp.nlat_in * hp.ps] = n;
    return SNA_OK;
}

size_t sna_workspace_bytes(const sna_plan_t* plan, int B, int H, int C) {
    if (plan == nullptr || B <= 0 || H <= 0 || C <= 0) return 0;
    return round256(2 * stats_elems(plan, B, H) * sizeof(float));
}

int sna_forward_kernel_count(const sna_plan_t* plan, int C, int with_lse) {
    if (plan == nullptr || plan->dev_blob == nullptr || !supported_C(C)) return 0;
    if (plan->is_global || sna::dense2_global_supported(plan->dev, C)) return 1;
    return (with_lse && sna::dense2_path_supported(plan->dev, C)) ? 2 : 1;
}

sna_status_t sna_forward_ex(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                            float* lse, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !out) { set_error("q, k, v and out must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, out) || (reinterpret_cast<uintptr_t>(lse) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    cudaError_t e;
    if (lse != nullptr && sna::dense2_global_supported(plan->dev, C)) {
        // every window is a whole ring (a global plan, or a cutoff that reaches every point): the dense kernel alone
        // produces the final out and lse
        e = sna::launch_forward_dense2(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    } else if (plan->is_global) {
        e = sna::launch_forward_generic(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    } else if (lse != nullptr && sna::dense2_path_supported(plan->dev, C)) {
        // whole-ring and wide windows on the tcgen05 kernel (its partial result travels in out / lse), the rest on the band kernel
        e = sna::launch_forward_dense2(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
        if (e == cudaSuccess) e = sna::launch_forward_mma_band(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    } else if (sna::mma_path_supported(plan->dev, C)) {
        e = sna::launch_forward_mma(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    } else {
        e = sna::launch_forward_generic(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "forward launch");
    return SNA_OK;
}

sna_status_t sna_forward(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                         int B, int H, int C, void* cuda_stream) {
    return sna_forward_ex(plan, q, k, v, out, nullptr, B, H, C, cuda_stream);
}

sna_status_t sna_backward_dq(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                             const float* dout, const float* out, const float* lse, float* dq, float* D,
                             int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !dout || !lse || !dq || !D) { set_error("q, k, v, dout, lse, dq and D must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, dout, dq, out) || ((reinterpret_cast<uintptr_t>(lse) | reinterpret_cast<uintptr_t>(D)) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    cudaError_t e;
    // The dense dq kernel takes the whole-ring and wide windows when they are at least a tenth of the work (measured on the
    // benchmark configurations: -8 % on the dq stage at a 22 % share, -6 % at 13 %).
    if (out != nullptr && out != dq && sna::dense2_global_supported(plan->dev, C)) {
        e = sna::launch_backward_dq_dense2(plan->dev, q, k, v, dout, out, lse, dq, D, B * H, C, (cudaStream_t)cuda_stream);
    } else if (plan->is_global) {
        e = sna::launch_backward_dq_generic(plan->dev, q, k, v, dout, out, lse, dq, D, B * H, C, (cudaStream_t)cuda_stream);
    } else if (out != nullptr && out != dq && plan->dev.dense_fraction >= 0.10f && sna::dense2_path_supported(plan->dev, C)) {
        // whole-ring and wide windows on the tcgen05 kernel (its part of dq is written first), the rest is added by the band kernel
        e = sna::launch_backward_dq_dense2(plan->dev, q, k, v, dout, out, lse, dq, nullptr, B * H, C, (cudaStream_t)cuda_stream);
        if (e == cudaSuccess) e = sna::launch_backward_dq_mma_band(plan->dev, q, k, v, dout, out, lse, dq, D, B * H, C, (cudaStream_t)cuda_stream);
    } else if (out != nullptr && sna::mma_path_supported(plan->dev, C)) {
        e = sna::launch_backward_dq_mma(plan->dev, q, k, v, dout, out, lse, dq, D, B * H, C, (cudaStream_t)cuda_stream);
    } else {
        e = sna::launch_backward_dq_generic(plan->dev, q, k, v, dout, out, lse, dq, D, B * H, C, (cudaStream_t)cuda_stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "backward dq launch");
    return SNA_OK;
}

sna_status_t sna_backward_dkdv(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                               const float* dout, const float* lse, const float* D, float* dk, float* dv,
                               int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !dout || !lse || !D || !dk || !dv) { set_error("q, k, v, dout, lse, D, dk and dv must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, dout, dk, dv) || ((reinterpret_cast<uintptr_t>(lse) | reinterpret_cast<uintptr_t>(D)) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    cudaError_t e;
    if (plan->is_global || sna::dense2_global_supported(plan->dev, C)) {
        // the dense kernel writes only the rings some window refers to; rings of weight zero get their (zero) gradient here
        const bool dense = sna::dense2_global_supported(plan->dev, C);
        const size_t ring_bytes = (size_t)plan->host.nlon_in * C * sizeof(float), pitch = ring_bytes * plan->host.nlat_in;
        for (size_t i = 0; dense && i < plan->zero_rings.size(); ++i) {
            const size_t off = ring_bytes * plan->zero_rings[i];
            e = cudaMemset2DAsync((char*)dk + off, pitch, 0, ring_bytes, (size_t)B * H, (cudaStream_t)cuda_stream);
            if (e == cudaSuccess) e = cudaMemset2DAsync((char*)dv + off, pitch, 0, ring_bytes, (size_t)B * H, (cudaStream_t)cuda_stream);
            if (e != cudaSuccess) return cuda_fail(e, "clearing the gradients of zero-weight rings");
        }
        e = dense
                ? sna::launch_backward_dkdv_dense2(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream)
                : sna::launch_backward_dkdv_generic(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream);
    } else if (plan->dev.dense_fraction >= 0.10f && plan->dev.n_t_dense_rows > 0 && sna::dense2_path_supported(plan->dev, C)) {
        // whole-ring and wide windows on the tcgen05 kernel (its part of dk, dv is written first), the band kernel adds the rest
        e = sna::launch_backward_dkdv_dense2(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream);
        if (e == cudaSuccess) e = sna::launch_backward_dkdv_mma_band(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream);
    } else if (sna::mma_path_supported(plan->dev, C)) {
        e = sna::launch_backward_dkdv_mma(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream);
    } else {
        e = sna::launch_backward_dkdv_generic(plan->dev, q, k, v, dout, lse, D, dk, dv, B * H, C, (cudaStream_t)cuda_stream);
    }
    if (e != cudaSuccess) return cuda_fail(e, "backward dk/dv launch");
    return SNA_OK;
}

sna_status_t sna_backward_ex(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                             const float* dout, const float* out, const float* lse, float* dq, float* dk, float* dv,
                             void* workspace, size_t workspace_bytes, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !dout || !dq || !dk || !dv) { set_error("q, k, v, dout, dq, dk and dv must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, dout, dq, dk, dv, out) || (reinterpret_cast<uintptr_t>(lse) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) { set_error("workspace must be non-NULL and 256-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (workspace_bytes < sna_workspace_bytes(plan, B, H, C)) { set_error("workspace too small: %zu < %zu bytes", workspace_bytes, sna_workspace_bytes(plan, B, H, C)); return SNA_ERR_WORKSPACE; }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int N = B * H;
    float* ws_lse = (float*)workspace;
    float* ws_D = ws_lse + stats_elems(plan, B, H);
    cudaError_t e;
    if (plan->is_global) {
        if (lse == nullptr || out == nullptr) {
            // recompute the forward pass.  The dense dq kernel may not read out from the dq buffer, so out goes into
            // the dk buffer (written only after the dq stage) when that is large enough; otherwise only the
            // statistics are recomputed and the generic dq kernel runs.
            const bool fits = (long long)plan->host.nlat_in * plan->host.nlon_in >= (long long)plan->host.nlat_out * plan->host.nlon_out;
            if (fits && sna::dense2_global_supported(plan->dev, C)) {
                e = sna::launch_forward_dense2(plan->dev, q, k, v, dk, ws_lse, N, C, stream);
                out = dk;
            } else {
                e = sna::launch_forward_generic(plan->dev, q, k, v, nullptr, ws_lse, N, C, stream);
                out = nullptr;
            }
            if (e != cudaSuccess) return cuda_fail(e, "statistics launch");
            lse = ws_lse;
        }
    } else if (sna::mma_path_supported(plan->dev, C)) {
        if (lse == nullptr || out == nullptr) {
            // recompute the forward pass: lse into the workspace, out into the dq buffer, which the dq stage
            // reads row by row before it overwrites the same rows with dq
            e = sna::launch_forward_mma(plan->dev, q, k, v, dq, ws_lse, N, C, stream);
            if (e != cudaSuccess) return cuda_fail(e, "statistics launch");
            lse = ws_lse;
            out = dq;
        }
    } else if (lse == nullptr) {   // recompute the softmax statistics
        e = sna::launch_forward_generic(plan->dev, q, k, v, nullptr, ws_lse, N, C, stream);
        if (e != cudaSuccess) return cuda_fail(e, "statistics launch");
        lse = ws_lse;
    }
    st = sna_backward_dq(plan, q, k, v, dout, out, lse, dq, ws_D, B, H, C, cuda_stream);
    if (st != SNA_OK) return st;
    return sna_backward_dkdv(plan, q, k, v, dout, lse, ws_D, dk, dv, B, H, C, cuda_stream);
}

sna_status_t sna_backward(const sna_plan_t* plan, const float* q, const float* k, const float* v, const float* dout,
                          float* dq, float* dk, float* dv, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    const size_t need = sna_workspace_bytes(plan, B, H, C);
    void* ws;
    {
        std::lock_guard<std::mutex> lock(plan->ws_mutex);
        if (plan->ws_bytes < need) {
            // a larger workspace than ever before: wait for work that may still use the old one, then replace it
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
            if (plan->ws) cudaFree(plan->ws);
            plan->ws = nullptr;
            plan->ws_bytes = 0;
            e = cudaMalloc(&plan->ws, need);
            if (e != cudaSuccess) { set_error("cudaMalloc of %zu workspace bytes: %s", need, cudaGetErrorString(e)); return SNA_ERR_ALLOC; }
            plan->ws_bytes = need;
        }
        ws = plan->ws;
    }
    return sna_backward_ex(plan, q, k, v, dout, nullptr, nullptr, dq, dk, dv, ws, need, B, H, C, cuda_stream);
}

// ---- channels-first entry points --------------------------------------------------------------------------
namespace {
struct CfState { float *q, *k, *v, *out, *lse; };
size_t in_elems(const sna_plan_t* plan, int B, int H, int C) { return (size_t)B * H * plan->host.nlat_in * plan->host.nlon_in * C; }
size_t out_elems(const sna_plan_t* plan, int B, int H, int C) { return stats_elems(plan, B, H) * C; }
CfState carve_state(const sna_plan_t* plan, void* state, int B, int H, int C) {
    char* p = (char*)state;
    CfState s;
    s.q = (float*)p;   p += round256(out_elems(plan, B, H, C) * sizeof(float));
    s.k = (float*)p;   p += round256(in_elems(plan, B, H, C) * sizeof(float));
    s.v = (float*)p;   p += round256(in_elems(plan, B, H, C) * sizeof(float));
    s.out = (float*)p; p += round256(out_elems(plan, B, H, C) * sizeof(float));
    s.lse = (float*)p;
    return s;
}
}  // namespace

size_t sna_cf_state_bytes(const sna_plan_t* plan, int B, int H, int C) {
    if (!plan || B <= 0 || H <= 0 || !supported_C(C)) return 0;
    return 2 * round256(out_elems(plan, B, H, C) * sizeof(float)) + 2 * round256(in_elems(plan, B, H, C) * sizeof(float)) +
           round256(stats_elems(plan, B, H) * sizeof(float));
}

size_t sna_cf_scratch_bytes(const sna_plan_t* plan, int B, int H, int C) {
    if (!plan || B <= 0 || H <= 0 || !supported_C(C)) return 0;
    return 2 * round256(out_elems(plan, B, H, C) * sizeof(float)) + 2 * round256(in_elems(plan, B, H, C) * sizeof(float)) +
           sna_workspace_bytes(plan, B, H, C);
}

sna_status_t sna_forward_cf(const sna_plan_t* plan, const float* q_cf, const float* k_cf, const float* v_cf, float* out_cf,
                            void* state, size_t state_bytes, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q_cf || !k_cf || !v_cf || !out_cf) { set_error("q, k, v and out must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q_cf, k_cf, v_cf, out_cf)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (state == nullptr || (reinterpret_cast<uintptr_t>(state) & 255u)) { set_error("state must be non-NULL and 256-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (state_bytes < sna_cf_state_bytes(plan, B, H, C)) { set_error("state too small: %zu < %zu bytes", state_bytes, sna_cf_state_bytes(plan, B, H, C)); return SNA_ERR_WORKSPACE; }
    if ((long long)B * H > 65535) { set_error("the channels-first entry points take at most 65535 batch*head slices"); return SNA_ERR_UNSUPPORTED; }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const CfState s = carve_state(plan, state, B, H, C);
    const long long p_in = (long long)plan->host.nlat_in * plan->host.nlon_in, p_out = (long long)plan->host.nlat_out * plan->host.nlon_out;
    cudaError_t e = sna::launch_cf_to_cl(q_cf, s.q, B * H, C, p_out, stream);
    if (e == cudaSuccess) e = sna::launch_cf_to_cl(k_cf, s.k, B * H, C, p_in, stream);
    if (e == cudaSuccess) e = sna::launch_cf_to_cl(v_cf, s.v, B * H, C, p_in, stream);
    if (e != cudaSuccess) return cuda_fail(e, "layout launch");
    st = sna_forward_ex(plan, s.q, s.k, s.v, s.out, s.lse, B, H, C, cuda_stream);
    if (st != SNA_OK) return st;
    e = sna::launch_cl_to_cf(s.out, out_cf, B * H, C, p_out, stream);
    if (e != cudaSuccess) return cuda_fail(e, "layout launch");
    return SNA_OK;
}

sna_status_t sna_backward_cf(const sna_plan_t* plan, const float* dout_cf, const void* state, size_t state_bytes,
                             void* scratch, size_t scratch_bytes, float* dq_cf, float* dk_cf, float* dv_cf,
                             int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!dout_cf || !dq_cf || !dk_cf || !dv_cf) { set_error("dout, dq, dk and dv must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(dout_cf, dq_cf, dk_cf, dv_cf)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (state == nullptr || (reinterpret_cast<uintptr_t>(state) & 255u) || scratch == nullptr || (reinterpret_cast<uintptr_t>(scratch) & 255u)) {
        set_error("state and scratch must be non-NULL and 256-byte aligned");
        return SNA_ERR_INVALID_ARG;
    }
    if (state_bytes < sna_cf_state_bytes(plan, B, H, C) || scratch_bytes < sna_cf_scratch_bytes(plan, B, H, C)) {
        set_error("state or scratch too small: %zu / %zu bytes given, %zu / %zu needed", state_bytes, scratch_bytes,
                  sna_cf_state_bytes(plan, B, H, C), sna_cf_scratch_bytes(plan, B, H, C));
        return SNA_ERR_WORKSPACE;
    }
    if ((long long)B * H > 65535) { set_error("the channels-first entry points take at most 65535 batch*head slices"); return SNA_ERR_UNSUPPORTED; }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const CfState s = carve_state(plan, const_cast<void*>(state), B, H, C);
    char* p = (char*)scratch;
    float* dout = (float*)p; p += round256(out_elems(plan, B, H, C) * sizeof(float));
    float* dq = (float*)p;   p += round256(out_elems(plan, B, H, C) * sizeof(float));
    float* dk = (float*)p;   p += round256(in_elems(plan, B, H, C) * sizeof(float));
    float* dv = (float*)p;   p += round256(in_elems(plan, B, H, C) * sizeof(float));
    void* ws = p;
    const long long p_in = (long long)plan->host.nlat_in * plan->host.nlon_in, p_out = (long long)plan->host.nlat_out * plan->host.nlon_out;
    cudaError_t e = sna::launch_cf_to_cl(dout_cf, dout, B * H, C, p_out, stream);
    if (e != cudaSuccess) return cuda_fail(e, "layout launch");
    st = sna_backward_ex(plan, s.q, s.k, s.v, dout, s.out, s.lse, dq, dk, dv, ws, sna_workspace_bytes(plan, B, H, C), B, H, C, cuda_stream);
    if (st != SNA_OK) return st;
    e = sna::launch_cl_to_cf(dq, dq_cf, B * H, C, p_out, stream);
    if (e == cudaSuccess) e = sna::launch_cl_to_cf(dk, dk_cf, B * H, C, p_in, stream);
    if (e == cudaSuccess) e = sna::launch_cl_to_cf(dv, dv_cf, B * H, C, p_in, stream);
    if (e != cudaSuccess) return cuda_fail(e, "layout launch");
    return SNA_OK;
}

sna_status_t sna_forward_tf32(const sna_plan_t* plan, const float* q, const float* k, const float* v, float* out,
                              float* lse, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !out) { set_error("q, k, v and out must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, out) || (reinterpret_cast<uintptr_t>(lse) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (!sna::mma_path_supported(plan->dev, C)) { set_error("the reduced-precision variant needs C in {16, 32, 64} and nlon_out >= 32"); return SNA_ERR_UNSUPPORTED; }
    cudaError_t e = sna::launch_forward_mma_lp(plan->dev, q, k, v, out, lse, B * H, C, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "forward launch");
    return SNA_OK;
}

sna_status_t sna_backward_tf32(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                               const float* dout, const float* out, const float* lse, float* dq, float* dk, float* dv,
                               void* workspace, size_t workspace_bytes, int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    if (!q || !k || !v || !dout || !dq || !dk || !dv) { set_error("q, k, v, dout, dq, dk and dv must not be NULL"); return SNA_ERR_INVALID_ARG; }
    if (!all_aligned(q, k, v, dout, dq, dk, dv, out) || (reinterpret_cast<uintptr_t>(lse) & 3u)) { set_error("device pointers must be 16-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) { set_error("workspace must be non-NULL and 256-byte aligned"); return SNA_ERR_INVALID_ARG; }
    if (workspace_bytes < sna_workspace_bytes(plan, B, H, C)) { set_error("workspace too small: %zu < %zu bytes", workspace_bytes, sna_workspace_bytes(plan, B, H, C)); return SNA_ERR_WORKSPACE; }
    if (!sna::mma_path_supported(plan->dev, C)) { set_error("the reduced-precision variant needs C in {16, 32, 64} and nlon_out >= 32"); return SNA_ERR_UNSUPPORTED; }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int N = B * H;
    float* ws_lse = (float*)workspace;
    float* ws_D = ws_lse + stats_elems(plan, B, H);
    cudaError_t e;
    if (lse == nullptr || out == nullptr) {   // recompute the forward pass: lse into the workspace, out into the dq buffer
        e = sna::launch_forward_mma_lp(plan->dev, q, k, v, dq, ws_lse, N, C, stream);
        if (e != cudaSuccess) return cuda_fail(e, "statistics launch");
        lse = ws_lse;
        out = dq;
    }
    e = sna::launch_backward_dq_mma_lp(plan->dev, q, k, v, dout, out, lse, dq, ws_D, N, C, stream);
    if (e == cudaSuccess) e = sna::launch_backward_dkdv_mma_lp(plan->dev, q, k, v, dout, lse, ws_D, dk, dv, N, C, stream);
    if (e != cudaSuccess) return cuda_fail(e, "backward launch");
    return SNA_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------
// Allocation-free backward pass: the scratch for the softmax statistics lives in the library image.
// ---------------------------------------------------------------------------------------------------------

// lse and D of up to SNA_STATIC_SCRATCH_MAX_POINTS output points.  In host code this name is only a handle for
// the runtime, not a device address: the address is looked up per device below and passed to the kernels.
static __device__ __align__(256) float g_static_scratch[2 * SNA_STATIC_SCRATCH_MAX_POINTS];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_static_scratch_mutex;
float* g_static_scratch_ptr[MAX_DEVICES] = {};

// Device address of g_static_scratch on the current device; resolved on the first call per device.
sna_status_t static_scratch_for_current_device(float** ptr_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= MAX_DEVICES) { set_error("device ordinal %d out of range", dev); return SNA_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (p == nullptr) { set_error("cudaGetSymbolAddress returned a null address"); return SNA_ERR_CUDA; }
        g_static_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *ptr_out = g_static_scratch_ptr[dev];
    return SNA_OK;
}
}  // namespace

extern "C" sna_status_t sna_backward_static(const sna_plan_t* plan, const float* q, const float* k, const float* v,
                                            const float* dout, float* dq, float* dk, float* dv,
                                            int B, int H, int C, void* cuda_stream) {
    sna_status_t st = check_problem(plan, B, H, C);
    if (st != SNA_OK) return st;
    const size_t points = stats_elems(plan, B, H);
    if (points > (size_t)SNA_STATIC_SCRATCH_MAX_POINTS) {
        set_error("problem has %zu output points; the static scratch of sna_backward_static holds at most %d "
                  "(use sna_backward or sna_backward_ex)", points, SNA_STATIC_SCRATCH_MAX_POINTS);
        return SNA_ERR_WORKSPACE;
    }
    float* scratch = nullptr;
    st = static_scratch_for_current_device(&scratch);
    if (st != SNA_OK) return st;
    // statistics are recomputed into the scratch (lse half, then D half); nothing needs clearing
    return sna_backward_ex(plan, q, k, v, dout, nullptr, nullptr, dq, dk, dv, scratch,
                           sizeof(float) * 2 * (size_t)SNA_STATIC_SCRATCH_MAX_POINTS, B, H, C, cuda_stream);
}


#ifdef SNA_PROF
// Profiling builds only: copies the per-role cycle counters that a -DSNA_PROF kernel left in the plan's status area.
extern "C" int sna_debug_read(const sna_plan_t* plan, long long* out, int count) {
    cudaDeviceSynchronize();
    return (int)cudaMemcpy(out, plan->dev.dev_status + 2, (size_t)count * 8, cudaMemcpyDeviceToHost);
}
#endif
