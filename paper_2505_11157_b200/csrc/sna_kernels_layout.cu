// Layout changes for the channels-first entry points: the paper's tensors are B x C x H x W (App. B.3), the kernels
// work on channels-last arrays [slice][point][C] so that one point's channels are one 16-byte-aligned run.  Both
// directions are tiled transposes through shared memory, coalesced on both sides; they are bound by HBM bandwidth
// (each element is read once and written once).
#include "sna_kernels.cuh"

#include <cstdint>

namespace sna {
namespace {

constexpr int LT_THREADS = 256;
constexpr int LT_MAXC = 128;
constexpr int LT_WORDS = 64 * 129;      // shared tile: 64 channels x 128 points, or 128 channels x 32 points (pitch + 1)

// Tiles of PTS points x C channels; PTS = 128 (each lane moves 16 bytes along the points) when C <= 64 and the planes are
// 16-byte aligned (P % 4 == 0), else PTS = 32 with 4-byte accesses on the channels-first side.
// src: [slices][C][P] (channels first), dst: [slices][P][C] (channels last)
template <int PTS>
__global__ void __launch_bounds__(LT_THREADS) cf_to_cl_kernel(const float* __restrict__ src, float* __restrict__ dst, int C, long long P) {
    __shared__ float tile[LT_WORDS];
    constexpr int PITCH = PTS + 1;
    const long long p0 = (long long)blockIdx.x * PTS;
    const size_t n = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if constexpr (PTS == 128) {
        const bool in = p0 + 4 * lane < P;      // P % 4 == 0: a float4 is inside or outside as a whole
        for (int c = warp; c < C; c += LT_THREADS / 32) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (in) x = __ldg(reinterpret_cast<const float4*>(src + (n * C + c) * (size_t)P + p0) + lane);
            float* t = tile + c * PITCH + 4 * lane;
            t[0] = x.x; t[1] = x.y; t[2] = x.z; t[3] = x.w;
        }
    } else {
        const bool in = p0 + lane < P;
        for (int c = warp; c < C; c += LT_THREADS / 32) tile[c * PITCH + lane] = in ? __ldg(src + (n * C + c) * (size_t)P + p0 + lane) : 0.f;
    }
    __syncthreads();
    const int c4n = C / 4;
    for (int idx = threadIdx.x; idx < PTS * c4n; idx += LT_THREADS) {
        const int pt = idx / c4n, c4 = idx - pt * c4n;
        if (p0 + pt < P) {
            const float* t = tile + 4 * c4 * PITCH + pt;
            *reinterpret_cast<float4*>(dst + (n * (size_t)P + p0 + pt) * C + 4 * c4) = make_float4(t[0], t[PITCH], t[2 * PITCH], t[3 * PITCH]);
        }
    }
}

// src: [slices][P][C] (channels last), dst: [slices][C][P] (channels first)
template <int PTS>
__global__ void __launch_bounds__(LT_THREADS) cl_to_cf_kernel(const float* __restrict__ src, float* __restrict__ dst, int C, long long P) {
    __shared__ float tile[LT_WORDS];
    constexpr int PITCH = PTS + 1;
    const long long p0 = (long long)blockIdx.x * PTS;
    const size_t n = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c4n = C / 4;
    for (int idx = threadIdx.x; idx < PTS * c4n; idx += LT_THREADS) {
        const int pt = idx / c4n, c4 = idx - pt * c4n;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p0 + pt < P) x = __ldg(reinterpret_cast<const float4*>(src + (n * (size_t)P + p0 + pt) * C + 4 * c4));
        float* t = tile + 4 * c4 * PITCH + pt;
        t[0] = x.x; t[PITCH] = x.y; t[2 * PITCH] = x.z; t[3 * PITCH] = x.w;
    }
    __syncthreads();
    if constexpr (PTS == 128) {
        if (p0 + 4 * lane < P)
            for (int c = warp; c < C; c += LT_THREADS / 32) {
                const float* t = tile + c * PITCH + 4 * lane;
                reinterpret_cast<float4*>(dst + (n * C + c) * (size_t)P + p0)[lane] = make_float4(t[0], t[1], t[2], t[3]);
            }
    } else {
        if (p0 + lane < P)
            for (int c = warp; c < C; c += LT_THREADS / 32) dst[(n * C + c) * (size_t)P + p0 + lane] = tile[c * PITCH + lane];
    }
}

cudaError_t launch(bool to_cl, const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream) {
    if (C <= 0 || C > LT_MAXC || C % 4 != 0 || slices <= 0 || slices > 65535 || P <= 0) return cudaErrorInvalidValue;
    const bool wide = C <= 64 && P % 4 == 0;
    const int pts = wide ? 128 : 32;
    const long long tiles = (P + pts - 1) / pts;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)tiles, (unsigned)slices);
    if (to_cl) {
        if (wide) cf_to_cl_kernel<128><<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
        else cf_to_cl_kernel<32><<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
    } else {
        if (wide) cl_to_cf_kernel<128><<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
        else cl_to_cf_kernel<32><<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_cf_to_cl(const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream) {
    return launch(true, src, dst, slices, C, P, stream);
}
cudaError_t launch_cl_to_cf(const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream) {
    return launch(false, src, dst, slices, C, P, stream);
}

}  // namespace sna
