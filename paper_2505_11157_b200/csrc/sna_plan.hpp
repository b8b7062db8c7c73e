// Host-side planner: grids, quadrature weights and the neighborhood table in run-length form.
// Pure C++ (no CUDA); everything is computed in double (long double inside the node/weight routines).
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace sna {

enum PlanStatus { PLAN_OK = 0, PLAN_INVALID = 1, PLAN_UNSUPPORTED = 2, PLAN_EMPTY = 3, PLAN_AMBIGUOUS = 6 };

// One input ring seen from one output latitude.  Because the disc is symmetric about the meridian of the
// output point, the member columns of a ring are always lon_off in {-m..m} (mod nlon_in) or the whole ring.
struct RingWindow {
    int32_t lat;   // input ring h' (forward table) or output ring h (transposed table)
    int32_t m;     // half width in input columns; -1 means the whole ring
};

struct HostPlan {
    int nlat_in = 0, nlon_in = 0, nlat_out = 0, nlon_out = 0, ps = 1;
    int grid_in = 0, grid_out = 0;
    double theta_cutoff = 0.0;
    std::vector<double> theta_in, theta_out;   // colatitudes
    std::vector<double> omega;                 // per-point quadrature weight of each input ring
    std::vector<int32_t> row_ptr;              // [nlat_out+1] into windows
    std::vector<RingWindow> windows;           // forward: per output latitude, input rings ascending
    std::vector<int32_t> t_row_ptr;            // [nlat_in+1] into t_windows
    std::vector<RingWindow> t_windows;         // transposed: per input latitude, output rings ascending
    std::vector<int64_t> row_nnz;              // [nlat_out] table entries per output latitude
    std::vector<int64_t> t_row_nnz;            // [nlat_in] (output ring, offset) pairs per input latitude (all columns)
    int64_t nnz = 0;

    int window_count(const RingWindow& w) const { return w.m < 0 ? nlon_in : 2 * w.m + 1; }
};

// Builds the plan.  On failure returns a status and fills `why`.
PlanStatus build_plan(int nlat_in, int nlon_in, int nlat_out, int nlon_out, int grid_in, int grid_out,
                      double theta_cutoff, HostPlan& plan, std::string& why);

}  // namespace sna
