// Generic kernels: correct for every supported channel count (any multiple of 4 up to 128).  A group of LP lanes
// holds one grid point, each lane a float4 of channels; LP is C/4 rounded up to a power of two, and the surplus
// lanes of a group carry zeros and store nothing.  Dot products are reduced with warp shuffles, the softmax is kept
// online in registers.
// Forward: Eq. (s2_attention_discrete_detailed); backward: App. B.4.
#include "sna_kernels.cuh"

#include <type_traits>

namespace sna {
namespace {

constexpr int THREADS = 256;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

__device__ __forceinline__ float dot4(const float4& a, const float4& b) {
    return fmaf(a.x, b.x, fmaf(a.y, b.y, fmaf(a.z, b.z, a.w * b.w)));
}
template <int LP>
__device__ __forceinline__ float group_sum(float x) {
#pragma unroll
    for (int s = LP / 2; s > 0; s >>= 1) x += __shfl_xor_sync(0xffffffffu, x, s);
    return x;
}
__device__ __forceinline__ void axpy4(float4& acc, float a, const float4& x) {
    acc.x = fmaf(a, x.x, acc.x); acc.y = fmaf(a, x.y, acc.y); acc.z = fmaf(a, x.z, acc.z); acc.w = fmaf(a, x.w, acc.w);
}
__device__ __forceinline__ void scale4(float4& acc, float a) { acc.x *= a; acc.y *= a; acc.z *= a; acc.w *= a; }
__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
// the float4 of a lane that holds channels, zeros for a padding lane
__device__ __forceinline__ float4 ldg4(const float* p, bool lane_ok) { return lane_ok ? ldg4(p) : make_float4(0.f, 0.f, 0.f, 0.f); }

// Decode a block index into (slice n, output/input latitude, first longitude of the block's tile); the
// latitudes with the most work come first so the long polar rows do not form the tail of the grid.
__device__ __forceinline__ void decode_block(int b, int N, int tiles, const int32_t* order, int& n, int& lat, int& tile) {
    tile = b % tiles;
    int r = b / tiles;
    n = r % N;
    lat = order[r / N];
}

template <int LP>
__global__ void __launch_bounds__(THREADS)
forward_generic_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                       float* __restrict__ out, float* __restrict__ lse, int N, int C, float scale_log2) {
    constexpr int PPB = THREADS / LP;
    const int tiles = (p.nlon_out + PPB - 1) / PPB;
    int n, h, tile;
    decode_block(blockIdx.x, N, tiles, p.row_order, n, h, tile);
    const int lane = threadIdx.x % LP;
    const bool lane_ok = lane * 4 < C;
    const int w = tile * PPB + threadIdx.x / LP;
    const bool active = w < p.nlon_out;
    const int wc = active ? w : p.nlon_out - 1;      // inactive groups shadow a valid point (shuffles stay converged)
    const size_t oi = ((size_t)(n * p.nlat_out + h) * p.nlon_out + wc);
    const float4 qv = ldg4(q + oi * C + lane * 4, lane_ok);
    float m = -INFINITY, Z = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int c0 = wc * p.ps;
    for (int e = p.row_ptr[h]; e < p.row_ptr[h + 1]; ++e) {
        const int hp = p.win_lat[e], hm = p.win_m[e];
        const int cnt = hm < 0 ? p.nlon_in : 2 * hm + 1;
        int col = hm < 0 ? c0 : c0 - hm;
        if (col < 0) col += p.nlon_in;
        const float bias = p.log2_omega[hp];
        const float* kr = k + (size_t)(n * p.nlat_in + hp) * p.nlon_in * C + lane * 4;
        const float* vr = v + (size_t)(n * p.nlat_in + hp) * p.nlon_in * C + lane * 4;
        for (int j = 0; j < cnt; j += 2) {
            const bool two = j + 1 < cnt;
            int col1 = col + 1; if (col1 >= p.nlon_in) col1 -= p.nlon_in;
            const float4 k0 = ldg4(kr + (size_t)col * C, lane_ok);
            const float4 k1 = ldg4(kr + (size_t)(two ? col1 : col) * C, lane_ok);
            float s0 = group_sum<LP>(dot4(qv, k0)) * scale_log2 + bias;
            float s1 = two ? group_sum<LP>(dot4(qv, k1)) * scale_log2 + bias : -INFINITY;
            const float mn = fmaxf(m, fmaxf(s0, s1));
            const float corr = exp2f(m - mn);
            const float p0 = exp2f(s0 - mn), p1 = exp2f(s1 - mn);
            Z = fmaf(Z, corr, p0 + p1);
            m = mn;
            if (out != nullptr) {
                const float4 v0 = ldg4(vr + (size_t)col * C, lane_ok);
                const float4 v1 = ldg4(vr + (size_t)(two ? col1 : col) * C, lane_ok);
                scale4(acc, corr);
                axpy4(acc, p0, v0);
                axpy4(acc, p1, v1);
            }
            col = col1 + 1; if (col >= p.nlon_in) col -= p.nlon_in;
        }
    }
    if (!active) return;
    if (out != nullptr && lane_ok) {
        const float inv = 1.f / Z;
        scale4(acc, inv);
        *reinterpret_cast<float4*>(out + oi * C + lane * 4) = acc;
    }
    if (lse != nullptr && lane == 0) lse[oi] = (m + log2f(Z)) * LN2;
}

template <int LP, bool HAVE_OUT>
__global__ void __launch_bounds__(THREADS)
backward_dq_generic_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                           const float* __restrict__ dout, const float* __restrict__ out, const float* __restrict__ lse,
                           float* __restrict__ dq, float* __restrict__ Dws, int N, int C, float scale, float scale_log2) {
    constexpr int PPB = THREADS / LP;
    const int tiles = (p.nlon_out + PPB - 1) / PPB;
    int n, h, tile;
    decode_block(blockIdx.x, N, tiles, p.row_order, n, h, tile);
    const int lane = threadIdx.x % LP;
    const bool lane_ok = lane * 4 < C;
    const int w = tile * PPB + threadIdx.x / LP;
    const bool active = w < p.nlon_out;
    const int wc = active ? w : p.nlon_out - 1;
    const size_t oi = ((size_t)(n * p.nlat_out + h) * p.nlon_out + wc);
    const float4 qv = ldg4(q + oi * C + lane * 4, lane_ok);
    const float4 dy = ldg4(dout + oi * C + lane * 4, lane_ok);
    const float lse2 = lse[oi] * LOG2E;
    float D = 0.f;
    if (HAVE_OUT) D = group_sum<LP>(dot4(dy, ldg4(out + oi * C + lane * 4, lane_ok)));
    float4 a1 = make_float4(0.f, 0.f, 0.f, 0.f), a2 = make_float4(0.f, 0.f, 0.f, 0.f);
    float Dacc = 0.f;
    const int c0 = wc * p.ps;
    for (int e = p.row_ptr[h]; e < p.row_ptr[h + 1]; ++e) {
        const int hp = p.win_lat[e], hm = p.win_m[e];
        const int cnt = hm < 0 ? p.nlon_in : 2 * hm + 1;
        int col = hm < 0 ? c0 : c0 - hm;
        if (col < 0) col += p.nlon_in;
        const float bias = p.log2_omega[hp] - lse2;
        const float* kr = k + (size_t)(n * p.nlat_in + hp) * p.nlon_in * C + lane * 4;
        const float* vr = v + (size_t)(n * p.nlat_in + hp) * p.nlon_in * C + lane * 4;
        for (int j = 0; j < cnt; ++j) {
            const float4 kj = ldg4(kr + (size_t)col * C, lane_ok);
            const float4 vj = ldg4(vr + (size_t)col * C, lane_ok);
            float s = dot4(qv, kj), t = dot4(dy, vj);
#pragma unroll
            for (int sh = LP / 2; sh > 0; sh >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, sh);
                t += __shfl_xor_sync(0xffffffffu, t, sh);
            }
            const float pj = exp2f(fmaf(s, scale_log2, bias));
            if (HAVE_OUT) {
                axpy4(a1, pj * (t - D), kj);
            } else {
                Dacc = fmaf(pj, t, Dacc);
                axpy4(a1, pj * t, kj);
                axpy4(a2, pj, kj);
            }
            if (++col >= p.nlon_in) col = 0;
        }
    }
    if (!active) return;
    if (!HAVE_OUT) {
        D = Dacc;
        a1.x -= D * a2.x; a1.y -= D * a2.y; a1.z -= D * a2.z; a1.w -= D * a2.w;
    }
    scale4(a1, scale);
    if (lane_ok) *reinterpret_cast<float4*>(dq + oi * C + lane * 4) = a1;
    if (lane == 0) Dws[oi] = D;
}

__device__ __forceinline__ int floor_div(int a, int b) { int q = a / b; return (a % b != 0 && (a < 0)) ? q - 1 : q; }

template <int LP>
__global__ void __launch_bounds__(THREADS)
backward_dkdv_generic_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                             const float* __restrict__ dout, const float* __restrict__ lse, const float* __restrict__ Dws,
                             float* __restrict__ dk, float* __restrict__ dv, int N, int C, float scale, float scale_log2) {
    constexpr int PPB = THREADS / LP;
    const int tiles = (p.nlon_in + PPB - 1) / PPB;
    int n, hp, tile;
    decode_block(blockIdx.x, N, tiles, p.t_row_order, n, hp, tile);
    const int lane = threadIdx.x % LP;
    const bool lane_ok = lane * 4 < C;
    const int c = tile * PPB + threadIdx.x / LP;
    const bool active = c < p.nlon_in;
    const int cc = active ? c : p.nlon_in - 1;
    const size_t ji = ((size_t)(n * p.nlat_in + hp) * p.nlon_in + cc);
    const float4 kj = ldg4(k + ji * C + lane * 4, lane_ok);
    const float4 vj = ldg4(v + ji * C + lane * 4, lane_ok);
    const float bias = p.log2_omega[hp];
    float4 gk = make_float4(0.f, 0.f, 0.f, 0.f), gv = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int e = p.t_row_ptr[hp]; e < p.t_row_ptr[hp + 1]; ++e) {
        const int h = p.t_win_lat[e], hm = p.t_win_m[e];
        // output longitudes w with (cc - w*ps) mod nlon_in inside the window
        // (the trip count must not differ between the groups of a warp because of the shuffles below, so the
        // loop runs to the largest possible count and masks the surplus iterations)
        int wlo, cnt, cnt_uniform;
        if (hm < 0) { wlo = 0; cnt = p.nlon_out; cnt_uniform = cnt; }
        else {
            wlo = -floor_div(-(cc - hm), p.ps);                 // ceil((cc - hm)/ps)
            cnt = floor_div(cc + hm, p.ps) - wlo + 1;
            cnt_uniform = (2 * hm) / p.ps + 1;
        }
        int w = wlo % p.nlon_out; if (w < 0) w += p.nlon_out;
        const size_t rowbase = (size_t)(n * p.nlat_out + h) * p.nlon_out;
        for (int j = 0; j < cnt_uniform; ++j) {
            const bool valid = j < cnt;
            const size_t oi = rowbase + w;
            const float4 qi = ldg4(q + oi * C + lane * 4, lane_ok);
            const float4 dy = ldg4(dout + oi * C + lane * 4, lane_ok);
            float s = dot4(qi, kj), t = dot4(dy, vj);
#pragma unroll
            for (int sh = LP / 2; sh > 0; sh >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, sh);
                t += __shfl_xor_sync(0xffffffffu, t, sh);
            }
            const float pij = valid ? exp2f(fmaf(s, scale_log2, bias - lse[oi] * LOG2E)) : 0.f;
            axpy4(gk, pij * (t - Dws[oi]), qi);
            axpy4(gv, pij, dy);
            if (++w >= p.nlon_out) w = 0;
        }
    }
    if (!active) return;
    scale4(gk, scale);
    if (lane_ok) {
        *reinterpret_cast<float4*>(dk + ji * C + lane * 4) = gk;
        *reinterpret_cast<float4*>(dv + ji * C + lane * 4) = gv;
    }
}

template <typename F>
cudaError_t dispatch_lp(int C, F&& f) {
    if (C < 4 || C > 128 || C % 4 != 0) return cudaErrorInvalidValue;
    const int lanes = C / 4;   // rounded up to a power of two
    if (lanes <= 1) return f(std::integral_constant<int, 1>());
    if (lanes <= 2) return f(std::integral_constant<int, 2>());
    if (lanes <= 4) return f(std::integral_constant<int, 4>());
    if (lanes <= 8) return f(std::integral_constant<int, 8>());
    if (lanes <= 16) return f(std::integral_constant<int, 16>());
    return f(std::integral_constant<int, 32>());
}

}  // namespace

cudaError_t launch_forward_generic(const DevPlan& p, const float* q, const float* k, const float* v, float* out,
                                   float* lse, int N, int C, cudaStream_t stream) {
    const float scale_log2 = LOG2E / sqrtf((float)C);
    return dispatch_lp(C, [&](auto lp) {
        constexpr int LP = decltype(lp)::value;
        const int tiles = (p.nlon_out + THREADS / LP - 1) / (THREADS / LP);
        const long long blocks = (long long)tiles * p.nlat_out * N;
        if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
        forward_generic_kernel<LP><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, out, lse, N, C, scale_log2);
        return cudaGetLastError();
    });
}

cudaError_t launch_backward_dq_generic(const DevPlan& p, const float* q, const float* k, const float* v,
                                       const float* dout, const float* out, const float* lse, float* dq, float* Dws,
                                       int N, int C, cudaStream_t stream) {
    const float scale = 1.0f / sqrtf((float)C), scale_log2 = LOG2E * scale;
    return dispatch_lp(C, [&](auto lp) {
        constexpr int LP = decltype(lp)::value;
        const int tiles = (p.nlon_out + THREADS / LP - 1) / (THREADS / LP);
        const long long blocks = (long long)tiles * p.nlat_out * N;
        if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
        if (out != nullptr)
            backward_dq_generic_kernel<LP, true><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, dout, out, lse, dq, Dws, N, C, scale, scale_log2);
        else
            backward_dq_generic_kernel<LP, false><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, dout, out, lse, dq, Dws, N, C, scale, scale_log2);
        return cudaGetLastError();
    });
}

cudaError_t launch_backward_dkdv_generic(const DevPlan& p, const float* q, const float* k, const float* v,
                                         const float* dout, const float* lse, const float* Dws, float* dk, float* dv,
                                         int N, int C, cudaStream_t stream) {
    const float scale = 1.0f / sqrtf((float)C), scale_log2 = LOG2E * scale;
    return dispatch_lp(C, [&](auto lp) {
        constexpr int LP = decltype(lp)::value;
        const int tiles = (p.nlon_in + THREADS / LP - 1) / (THREADS / LP);
        const long long blocks = (long long)tiles * p.nlat_in * N;
        if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
        backward_dkdv_generic_kernel<LP><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, dout, lse, Dws, dk, dv, N, C, scale, scale_log2);
        return cudaGetLastError();
    });
}

}  // namespace sna
