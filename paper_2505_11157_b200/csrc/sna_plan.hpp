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

// The table the kernels walk: `full` without the input rings of quadrature weight zero (the pole ring of the
// trapezoid grid).  Such points are members of discs but add nothing to any sum, and their own gradients are zero,
// which the kernels produce for any input ring no window refers to.  Returns false (out untouched) if no ring has
// weight zero.
bool drop_zero_weight_rings(const HostPlan& full, HostPlan& out);

// Column streams for the tensor-core kernels.  A warp owns a tile of 16 points: TILE_LON = 8 consecutive
// longitudes on each of TILE_LAT = 2 adjacent rings (a "ring group"); tile row i is ring i / 8 of the group,
// longitude first + i % 8.  Two adjacent rings see almost the same partner points, and 8-wide rows waste fewer
// columns on the slanted band than 16-wide rows would.  The warp walks a stream of partner points ("columns"),
// 16 per step.  For a window with offsets e in [e_lo, e_hi] (in units of ps input columns for the forward
// table, of output columns for the transposed one) a row at longitude first + i uses partner first + e_rel iff
// e_lo <= e_rel - i <= e_hi: that is the row's bit in the column's 16-bit mask.  The stream of a ring group is
// the concatenation, over partner rings and residues, of the columns at least one row uses, padded to a
// multiple of 16 with mask-0 columns; it is the same for every tile of the group, so it is built once on the host.
constexpr int TILE_LON = 8;
constexpr int TILE_LAT = 2;

struct StreamEntry {
    int32_t base;      // flat row index of the partner ring plus the residue r; bit 31 set = e is absolute
    int32_t e_mask;    // low 16 bits: e_rel (signed) or the absolute partner index; high 16 bits: row mask
    float bias;        // forward: log2 of the partner ring's quadrature weight; transposed: unused (0)
    int32_t aux;       // unused
};

struct Stream {
    std::vector<int32_t> chunk_ptr;     // [rows+1] first 16-column chunk of each stream row
    std::vector<StreamEntry> entries;   // 16 * chunk_ptr.back()
};

// Forward stream: one row per group of output latitudes (ceil(nlat_out / TILE_LAT) rows); partners are input
// points, flat index base + u*ps.
// With dense_min_width > 0 the columns of the windows that served_by_dense() accepts are left out: those are served
// by the dense kernels (see DenseLists), and the stream only carries the narrower windows.
void build_forward_stream(const HostPlan& plan, Stream& out, int dense_min_width = 0);

// Which windows the dense (tcgen05) kernels take: whole rings, and banded windows of at least dense_min_width input
// columns (they run as masked blocks there).  dense_min_width = nlon_in + 1 selects the whole rings only.
inline bool served_by_dense(const RingWindow& w, int dense_min_width) {
    return dense_min_width > 0 && (w.m < 0 || 2 * w.m + 1 >= dense_min_width);
}

// The dense kernels' windows per output latitude: ring h attends to the input rings lat[ptr[h]] .. lat[ptr[h+1]-1],
// to all of ring lat[e] if m[e] < 0, else to the columns within m[e] of its own.
struct DenseLists {
    std::vector<int32_t> ptr;    // [nlat_out+1]
    std::vector<int32_t> lat;    // input rings
    std::vector<int32_t> m;      // window half widths in input columns, -1 = whole ring
    std::vector<int32_t> rows;   // output latitudes that have at least one such window
    int64_t pairs = 0;           // table entries covered, per output longitude / input column
};
void build_dense_lists(const HostPlan& plan, DenseLists& out, int dense_min_width);
// The transposed lists for the dense dk/dv kernel: input ring h' is attended to through such a window by the output
// rings lat[ptr[h']] .. lat[ptr[h'+1]-1]; rows = input latitudes with at least one such output ring.
void build_transposed_dense_lists(const HostPlan& plan, DenseLists& out, int dense_min_width);
// Transposed stream for dk/dv; partners are output points (h, w).  Two layouts:
//  - consecutive (when ps divides 8): one stream row per group of input latitudes; tile rows are 8 consecutive
//    input columns c = c0 + i%8 (c0 a multiple of 8) and the partner index is c0/ps + e_rel.  Neighbouring
//    input columns share most of their partners, so this needs ~ps times fewer stream columns per input column
//    than splitting by residue.
//  - by residue (any other ps): one stream row per (group, residue r); tile rows are c = ps*(u0+i%8) + r and
//    the partner index is u0 + e_rel.
// Returns true for the consecutive layout.
bool build_transposed_stream(const HostPlan& plan, Stream& out, int dense_min_width = 0);

// Builds the plan.  On failure returns a status and fills `why`.
PlanStatus build_plan(int nlat_in, int nlon_in, int nlat_out, int nlon_out, int grid_in, int grid_out,
                      double theta_cutoff, HostPlan& plan, std::string& why);

}  // namespace sna
