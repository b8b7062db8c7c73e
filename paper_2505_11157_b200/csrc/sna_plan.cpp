// Host planner.  Grids and quadrature: App. A.1 and Eq. (quadrature); neighborhood indicator: App. B.3,
// disc of Eq. (s2_neighborhood_attention).
//
// Construction (deliberately not a brute-force scan): on a fixed input ring the geodesic distance to the
// output point grows monotonically with the longitude difference, so each ring contributes one window
// symmetric about offset 0.  The half width follows from the spherical law of cosines,
//     cos(dphi_max) = (cos(theta_c) - cos(t_o) cos(t_i)) / (sin(t_o) sin(t_i)),
// and the columns around that estimate are then tested exactly with a cross/dot (atan2) distance, which is
// accurate for small and large angles alike.  Boundary ties are members (d <= theta_c + 1e-10); a candidate in
// the band 1e-12 < |d - theta_c| < 1e-8 aborts the build as ambiguous.
#include "sna_plan.hpp"

#include <algorithm>
#include <climits>
#include <cmath>
#include <cstdint>

namespace sna {
namespace {

const long double PI_L = 3.14159265358979323846264338327950288L;
const double TIE_SLACK = 1e-10, BAND_LO = 1e-12, BAND_HI = 1e-8;

// Gauss-Legendre nodes (descending) and weights by Newton iteration in extended precision, started from
// Tricomi's asymptotic estimate of the roots.
void legendre_gauss(int n, std::vector<double>& x, std::vector<double>& w) {
    x.resize(n);
    w.resize(n);
    for (int i = 1; i <= (n + 1) / 2; ++i) {
        long double z = (1.0L - (n - 1.0L) / (8.0L * n * n * n)) * cosl(PI_L * (4.0L * i - 1.0L) / (4.0L * n + 2.0L));
        long double pn = 0, pn1 = 0;
        for (int it = 0; it < 64; ++it) {
            long double a = 1.0L, b = z;   // P_0, P_1
            for (int l = 1; l < n; ++l) {
                long double c = ((2 * l + 1) * z * b - l * a) / (l + 1);
                a = b;
                b = c;
            }
            pn = b;
            pn1 = a;
            long double deriv = n * (pn1 - z * pn) / (1.0L - z * z);
            long double step = pn / deriv;
            z -= step;
            if (fabsl(step) < 1e-19L) break;
        }
        // re-evaluate at the converged node for the weight
        long double a = 1.0L, b = z;
        for (int l = 1; l < n; ++l) {
            long double c = ((2 * l + 1) * z * b - l * a) / (l + 1);
            a = b;
            b = c;
        }
        long double deriv = n * (a - z * b) / (1.0L - z * z);
        long double wt = 2.0L / ((1.0L - z * z) * deriv * deriv);
        x[i - 1] = (double)z;
        w[i - 1] = (double)wt;
        x[n - i] = (double)(-z);
        w[n - i] = (double)wt;
    }
    if (n % 2 == 1) x[n / 2] = 0.0;
}

// Clenshaw-Curtis weights on nlat equally spaced colatitudes including both poles.
void clenshaw_curtis(int nlat, std::vector<double>& w) {
    const int n = nlat - 1;
    w.resize(nlat);
    for (int h = 0; h <= n; ++h) {
        long double acc = 1.0L;
        for (int k = 1; k <= n / 2; ++k) {
            long long arg = (2LL * k * h) % (2LL * n);           // cos(2 k pi h / n) with an exactly reduced argument
            long double bk = (2 * k == n) ? 1.0L : 2.0L;
            acc -= bk * cosl(PI_L * (long double)arg / (long double)n) / (4.0L * k * k - 1.0L);
        }
        long double ch = (h == 0 || h == n) ? 1.0L : 2.0L;
        w[h] = (double)(ch * acc / n);
    }
}

bool make_grid(int grid, int nlat, std::vector<double>& theta, std::vector<double>& wlat) {
    if (grid == 0) {
        theta.resize(nlat);
        for (int h = 0; h < nlat; ++h) theta[h] = (double)(PI_L * h / (nlat - 1));
        clenshaw_curtis(nlat, wlat);
        return true;
    }
    if (grid == 1) {
        std::vector<double> x;
        legendre_gauss(nlat, x, wlat);
        theta.resize(nlat);
        for (int h = 0; h < nlat; ++h) theta[h] = std::acos(x[h]);
        return true;
    }
    if (grid == 2) {
        // the grid as App. A.1 prints it (Eq. latlon_grid, Eq. latlon_quad_weights): north pole in, south pole out,
        // trapezoid weights (pi/nlat) sin(theta) in latitude; the pole ring's weight is exactly zero
        theta.resize(nlat);
        wlat.resize(nlat);
        for (int h = 0; h < nlat; ++h) {
            theta[h] = (double)(PI_L * h / nlat);
            wlat[h] = h == 0 ? 0.0 : (double)(PI_L / nlat * sinl(PI_L * h / nlat));
        }
        return true;
    }
    return false;
}

// Geodesic distance between (t_o, 0) and (t_i, phi) from cross and dot products of the unit vectors.
double geodesic(double so, double co, double si, double ci, double phi) {
    const double cp = std::cos(phi), sp = std::sin(phi);
    const double ox = so, oz = co;
    const double ix = si * cp, iy = si * sp, iz = ci;
    const double cx = -oz * iy, cy = oz * ix - ox * iz, cz = ox * iy;
    return std::atan2(std::sqrt(cx * cx + cy * cy + cz * cz), ox * ix + oz * iz);
}

}  // namespace

PlanStatus build_plan(int nlat_in, int nlon_in, int nlat_out, int nlon_out, int grid_in, int grid_out,
                      double theta_cutoff, HostPlan& P, std::string& why) {
    if (nlat_in < 2 || nlat_out < 2 || nlon_in < 1 || nlon_out < 1) { why = "nlat must be >= 2 and nlon >= 1"; return PLAN_INVALID; }
    if (!(theta_cutoff > 0.0) || std::isnan(theta_cutoff)) { why = "theta_cutoff must be positive"; return PLAN_INVALID; }
    if (nlon_in % nlon_out != 0) { why = "nlon_in must be a multiple of nlon_out"; return PLAN_UNSUPPORTED; }
    P = HostPlan();
    P.nlat_in = nlat_in; P.nlon_in = nlon_in; P.nlat_out = nlat_out; P.nlon_out = nlon_out;
    P.ps = nlon_in / nlon_out; P.grid_in = grid_in; P.grid_out = grid_out; P.theta_cutoff = theta_cutoff;
    std::vector<double> wlat_in, wlat_out;
    if (!make_grid(grid_in, nlat_in, P.theta_in, wlat_in) || !make_grid(grid_out, nlat_out, P.theta_out, wlat_out)) {
        why = "unknown grid type";
        return PLAN_UNSUPPORTED;
    }
    P.omega.resize(nlat_in);
    for (int h = 0; h < nlat_in; ++h) P.omega[h] = wlat_in[h] * (double)(2.0L * PI_L / nlon_in);

    const bool everything = theta_cutoff >= (double)PI_L;
    const int half = nlon_in / 2;                        // largest |column offset| on a ring
    const double dphi = (double)(2.0L * PI_L / nlon_in);
    const double cos_tc = std::cos(theta_cutoff);
    bool ambiguous = false;
    auto member = [&](double d) {
        const double gap = std::fabs(d - theta_cutoff);
        if (gap > BAND_LO && gap < BAND_HI) ambiguous = true;
        return d <= theta_cutoff + TIE_SLACK;
    };

    P.row_ptr.assign(nlat_out + 1, 0);
    P.row_nnz.assign(nlat_out, 0);
    std::vector<std::vector<RingWindow>> by_input(nlat_in);
    for (int h = 0; h < nlat_out; ++h) {
        const double so = std::sin(P.theta_out[h]), co = std::cos(P.theta_out[h]);
        for (int hp = 0; hp < nlat_in; ++hp) {
            int m = -2;   // -2: ring not in the disc, -1: whole ring, >= 0: half width
            if (everything) {
                m = -1;
            } else {
                const double si = std::sin(P.theta_in[hp]), ci = std::cos(P.theta_in[hp]);
                if (!member(geodesic(so, co, si, ci, 0.0))) continue;   // nearest point of the ring is outside
                const double denom = so * si;
                int guess;
                if (denom < 1e-300) {
                    guess = half;   // a pole is involved: every column is equally far
                } else {
                    const double r = (cos_tc - co * ci) / denom;
                    guess = r <= -1.0 ? half : (r >= 1.0 ? 0 : (int)std::floor(std::acos(r) / dphi));
                }
                // exact test around the estimate; membership is monotone in the offset
                int lo = std::max(0, guess - 2), hi = std::min(half, guess + 2);
                while (lo > 0 && !member(geodesic(so, co, si, ci, lo * dphi))) lo = std::max(0, lo - 4);
                m = lo;
                for (int j = lo + 1; j <= hi; ++j) {
                    if (member(geodesic(so, co, si, ci, j * dphi))) m = j; else break;
                }
                if (m == hi && hi < half) {   // estimate was too small (never seen, but stay correct)
                    int j = hi + 1;
                    while (j <= half && member(geodesic(so, co, si, ci, j * dphi))) m = j++;
                }
                if (2 * m + 1 >= nlon_in) m = -1;
            }
            RingWindow w{hp, m};
            P.windows.push_back(w);
            P.row_nnz[h] += P.window_count(w);
            by_input[hp].push_back(RingWindow{h, m});
        }
        P.row_ptr[h + 1] = (int32_t)P.windows.size();
        if (P.row_ptr[h + 1] == P.row_ptr[h] && !ambiguous) { why = "an output latitude has no input point within theta_cutoff"; return PLAN_EMPTY; }
        bool weighted = false;
        for (int i = P.row_ptr[h]; i < P.row_ptr[h + 1]; ++i) weighted = weighted || P.omega[P.windows[i].lat] > 0.0;
        if (!weighted && !ambiguous) { why = "every input point within theta_cutoff of an output latitude has quadrature weight zero"; return PLAN_EMPTY; }
        P.nnz += P.row_nnz[h];
    }
    if (ambiguous) { why = "a grid point lies within 1e-8 rad of the disc boundary without being on it"; return PLAN_AMBIGUOUS; }

    P.t_row_ptr.assign(nlat_in + 1, 0);
    P.t_row_nnz.assign(nlat_in, 0);
    for (int hp = 0; hp < nlat_in; ++hp) {
        for (const RingWindow& w : by_input[hp]) {
            P.t_windows.push_back(w);
            P.t_row_nnz[hp] += P.window_count(w);
        }
        P.t_row_ptr[hp + 1] = (int32_t)P.t_windows.size();
    }
    return PLAN_OK;
}

bool drop_zero_weight_rings(const HostPlan& full, HostPlan& out) {
    bool any = false;
    for (double w : full.omega) any = any || !(w > 0.0);
    if (!any) return false;
    out = full;
    out.windows.clear();
    out.t_windows.clear();
    out.nnz = 0;
    for (int h = 0; h < full.nlat_out; ++h) {
        out.row_ptr[h] = (int32_t)out.windows.size();
        out.row_nnz[h] = 0;
        for (int i = full.row_ptr[h]; i < full.row_ptr[h + 1]; ++i) {
            const RingWindow& w = full.windows[i];
            if (!(full.omega[w.lat] > 0.0)) continue;
            out.windows.push_back(w);
            out.row_nnz[h] += full.window_count(w);
        }
        out.nnz += out.row_nnz[h];
    }
    out.row_ptr[full.nlat_out] = (int32_t)out.windows.size();
    for (int hp = 0; hp < full.nlat_in; ++hp) {
        out.t_row_ptr[hp] = (int32_t)out.t_windows.size();
        out.t_row_nnz[hp] = 0;
        if (!(full.omega[hp] > 0.0)) continue;
        for (int i = full.t_row_ptr[hp]; i < full.t_row_ptr[hp + 1]; ++i) {
            out.t_windows.push_back(full.t_windows[i]);
            out.t_row_nnz[hp] += full.window_count(full.t_windows[i]);
        }
    }
    out.t_row_ptr[full.nlat_in] = (int32_t)out.t_windows.size();
    return true;
}

namespace {

inline int floor_div(int a, int b) { int q = a / b; return ((a % b != 0) && ((a < 0) != (b < 0))) ? q - 1 : q; }
inline int ceil_div(int a, int b) { return -floor_div(-a, b); }

// One partner ring as seen from the rings of a group: per group ring either absent, a band of offsets, or whole.
struct GroupRange {
    bool present = false, whole = false;
    int lo = 0, hi = -1;
};

// Appends the columns of one partner ring / residue for a ring group.
void append_group_columns(std::vector<StreamEntry>& v, int32_t base, float bias, const GroupRange (&rg)[TILE_LAT], int whole_count) {
    uint32_t whole_rows = 0, band_rows_any = 0;
    for (int k = 0; k < TILE_LAT; ++k) {
        if (rg[k].present && rg[k].whole) whole_rows |= ((1u << TILE_LON) - 1u) << (k * TILE_LON);
        if (rg[k].present && !rg[k].whole && rg[k].hi >= rg[k].lo) band_rows_any |= 1u << k;
    }
    if (whole_rows) {   // absolute partner index: every partner of the ring, for the rings that take it whole
        for (int u = 0; u < whole_count; ++u)
            v.push_back(StreamEntry{(int32_t)(base | (int32_t)0x80000000), (int32_t)((u & 0xffff) | (whole_rows << 16)), bias, 0});
    }
    if (!band_rows_any) return;
    int lo = INT32_MAX, hi = INT32_MIN;
    for (int k = 0; k < TILE_LAT; ++k)
        if (band_rows_any & (1u << k)) { lo = std::min(lo, rg[k].lo); hi = std::max(hi, rg[k].hi); }
    for (int x = 0; x < TILE_LON - 1 + (hi - lo + 1); ++x) {
        const int e_rel = lo + x;
        uint32_t mask = 0;
        for (int k = 0; k < TILE_LAT; ++k) {
            if (!(band_rows_any & (1u << k))) continue;
            for (int i = 0; i < TILE_LON; ++i)
                if (e_rel - i >= rg[k].lo && e_rel - i <= rg[k].hi) mask |= 1u << (k * TILE_LON + i);
        }
        if (mask) v.push_back(StreamEntry{base, (int32_t)(((uint32_t)e_rel & 0xffffu) | (mask << 16)), bias, 0});
    }
}

void pad_row(std::vector<StreamEntry>& v, size_t row_start) {
    while ((v.size() - row_start) % 16 != 0) {
        StreamEntry pad = v.size() > row_start ? v.back() : StreamEntry{0, 0, 0.f, 0};
        pad.e_mask &= 0xffff;   // row mask 0: the column is ignored
        v.push_back(pad);
    }
}

// Merges the window lists of the rings of a group (each sorted by partner ring) and calls
// emit(partner_ring, m[TILE_LAT]) with m = -2 for "not in this ring's list".
template <typename Emit>
void merge_group(const std::vector<int32_t>& ptr, const std::vector<RingWindow>& win, int first_ring, int nrings, Emit&& emit) {
    int pos[TILE_LAT], end[TILE_LAT];
    for (int k = 0; k < TILE_LAT; ++k) {
        const int ring = first_ring + k;
        pos[k] = ring < nrings ? ptr[ring] : 0;
        end[k] = ring < nrings ? ptr[ring + 1] : 0;
    }
    for (;;) {
        int lat = INT32_MAX;
        for (int k = 0; k < TILE_LAT; ++k)
            if (pos[k] < end[k]) lat = std::min(lat, win[pos[k]].lat);
        if (lat == INT32_MAX) break;
        int m[TILE_LAT];
        for (int k = 0; k < TILE_LAT; ++k) m[k] = (pos[k] < end[k] && win[pos[k]].lat == lat) ? win[pos[k]++].m : -2;
        emit(lat, m);
    }
}

}  // namespace

void build_dense_lists(const HostPlan& P, DenseLists& D, int dense_min_width) {
    D = DenseLists();
    D.ptr.assign(P.nlat_out + 1, 0);
    for (int h = 0; h < P.nlat_out; ++h) {
        for (int e = P.row_ptr[h]; e < P.row_ptr[h + 1]; ++e) {
            if (!served_by_dense(P.windows[e], dense_min_width)) continue;
            D.lat.push_back(P.windows[e].lat);
            D.m.push_back(P.windows[e].m);
            D.pairs += P.window_count(P.windows[e]);
        }
        D.ptr[h + 1] = (int32_t)D.lat.size();
        if (D.ptr[h + 1] > D.ptr[h]) D.rows.push_back(h);
    }
}

void build_transposed_dense_lists(const HostPlan& P, DenseLists& D, int dense_min_width) {
    D = DenseLists();
    D.ptr.assign(P.nlat_in + 1, 0);
    for (int hp = 0; hp < P.nlat_in; ++hp) {
        for (int e = P.t_row_ptr[hp]; e < P.t_row_ptr[hp + 1]; ++e) {
            if (!served_by_dense(P.t_windows[e], dense_min_width)) continue;
            D.lat.push_back(P.t_windows[e].lat);
            D.m.push_back(P.t_windows[e].m);
            D.pairs += P.window_count(P.t_windows[e]);
        }
        D.ptr[hp + 1] = (int32_t)D.lat.size();
        if (D.ptr[hp + 1] > D.ptr[hp]) D.rows.push_back(hp);
    }
}

void build_forward_stream(const HostPlan& P, Stream& S, int dense_min_width) {
    const int groups = (P.nlat_out + TILE_LAT - 1) / TILE_LAT;
    S.chunk_ptr.assign(groups + 1, 0);
    S.entries.clear();
    for (int gi = 0; gi < groups; ++gi) {
        const size_t start = S.entries.size();
        merge_group(P.row_ptr, P.windows, gi * TILE_LAT, P.nlat_out, [&](int lat, const int (&m)[TILE_LAT]) {
            const float bias = (float)std::log2(P.omega[lat]);
            for (int r = 0; r < P.ps; ++r) {
                GroupRange rg[TILE_LAT];
                for (int k = 0; k < TILE_LAT; ++k) {
                    if (m[k] == -2) continue;
                    if (served_by_dense(RingWindow{lat, m[k]}, dense_min_width)) continue;
                    rg[k].present = true;
                    if (m[k] < 0) rg[k].whole = true;
                    else { rg[k].lo = ceil_div(-m[k] - r, P.ps); rg[k].hi = floor_div(m[k] - r, P.ps); }
                }
                append_group_columns(S.entries, lat * P.nlon_in + r, bias, rg, P.nlon_out);
            }
        });
        pad_row(S.entries, start);
        S.chunk_ptr[gi + 1] = (int32_t)(S.entries.size() / 16);
    }
}

bool build_transposed_stream(const HostPlan& P, Stream& S, int dense_min_width) {
    const int groups = (P.nlat_in + TILE_LAT - 1) / TILE_LAT;
    S.entries.clear();
    if (TILE_LON % P.ps == 0) {
        // Consecutive layout.  Tile row i of ring k is input column c0 + i; output point (h, w) is its partner iff
        // (c0 + i) - w*ps in [-m, m]  <=>  w - c0/ps in [ceil((i - m)/ps), floor((i + m)/ps)].
        S.chunk_ptr.assign((size_t)groups + 1, 0);
        for (int gi = 0; gi < groups; ++gi) {
            const size_t start = S.entries.size();
            merge_group(P.t_row_ptr, P.t_windows, gi * TILE_LAT, P.nlat_in, [&](int lat, const int (&m)[TILE_LAT]) {
                const int32_t base = lat * P.nlon_out;
                uint32_t whole_rows = 0;
                int lo = INT32_MAX, hi = INT32_MIN;
                for (int k = 0; k < TILE_LAT; ++k) {
                    if (m[k] == -2) continue;
                    if (served_by_dense(RingWindow{lat, m[k]}, dense_min_width)) continue;
                    if (m[k] < 0) { whole_rows |= ((1u << TILE_LON) - 1u) << (k * TILE_LON); continue; }
                    lo = std::min(lo, ceil_div(-m[k], P.ps));
                    hi = std::max(hi, floor_div(TILE_LON - 1 + m[k], P.ps));
                }
                if (whole_rows)
                    for (int u = 0; u < P.nlon_out; ++u)
                        S.entries.push_back(StreamEntry{(int32_t)(base | (int32_t)0x80000000), (int32_t)((u & 0xffff) | (whole_rows << 16)), 0.f, 0});
                for (int e_rel = lo; e_rel <= hi; ++e_rel) {
                    uint32_t mask = 0;
                    for (int k = 0; k < TILE_LAT; ++k) {
                        if (m[k] < 0 || served_by_dense(RingWindow{lat, m[k]}, dense_min_width)) continue;   // absent, whole (above) or dense
                        for (int i = 0; i < TILE_LON; ++i)
                            if (e_rel >= ceil_div(i - m[k], P.ps) && e_rel <= floor_div(i + m[k], P.ps)) mask |= 1u << (k * TILE_LON + i);
                    }
                    if (mask) S.entries.push_back(StreamEntry{base, (int32_t)(((uint32_t)e_rel & 0xffffu) | (mask << 16)), 0.f, 0});
                }
            });
            pad_row(S.entries, start);
            S.chunk_ptr[(size_t)gi + 1] = (int32_t)(S.entries.size() / 16);
        }
        return true;
    }
    // By residue.  Row (group, r): tile rows are input columns c = ps*u + r.  Output point (h, w) is a partner of
    // column u of input ring h' iff c - w*ps in [-m, m]  <=>  w - u in [ceil((r - m)/ps), floor((r + m)/ps)].
    S.chunk_ptr.assign((size_t)groups * P.ps + 1, 0);
    for (int gi = 0; gi < groups; ++gi) {
        for (int r = 0; r < P.ps; ++r) {
            const size_t start = S.entries.size();
            merge_group(P.t_row_ptr, P.t_windows, gi * TILE_LAT, P.nlat_in, [&](int lat, const int (&m)[TILE_LAT]) {
                GroupRange rg[TILE_LAT];
                for (int k = 0; k < TILE_LAT; ++k) {
                    if (m[k] == -2) continue;
                    if (served_by_dense(RingWindow{lat, m[k]}, dense_min_width)) continue;
                    rg[k].present = true;
                    if (m[k] < 0) rg[k].whole = true;
                    else { rg[k].lo = ceil_div(r - m[k], P.ps); rg[k].hi = floor_div(r + m[k], P.ps); }
                }
                append_group_columns(S.entries, lat * P.nlon_out, 0.f, rg, P.nlon_out);
            });
            pad_row(S.entries, start);
            S.chunk_ptr[(size_t)gi * P.ps + r + 1] = (int32_t)(S.entries.size() / 16);
        }
    }
    return false;
}

}  // namespace sna
