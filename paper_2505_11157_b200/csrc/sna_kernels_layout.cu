// Layout changes for the channels-first entry points: the paper's tensors are B x C x H x W (App. B.3), the kernels
// work on channels-last arrays [slice][point][C] so that one point's channels are one 16-byte-aligned run.  Both
// directions are tiled transposes through shared memory, coalesced on both sides; they are bound by HBM bandwidth
// (each element is read once and written once).
#include "sna_kernels.cuh"

#include <cstdint>

namespace sna {
namespace {

constexpr int LT_PTS = 32;        // points per tile
constexpr int LT_THREADS = 256;
constexpr int LT_MAXC = 128;

// src: [slices][C][P] (channels first), dst: [slices][P][C] (channels last)
__global__ void __launch_bounds__(LT_THREADS) cf_to_cl_kernel(const float* __restrict__ src, float* __restrict__ dst, int C, long long P) {
    __shared__ float tile[LT_MAXC][LT_PTS + 1];
    const long long p0 = (long long)blockIdx.x * LT_PTS;
    const size_t n = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool in = p0 + lane < P;
    for (int c = warp; c < C; c += LT_THREADS / 32) tile[c][lane] = in ? __ldg(src + (n * C + c) * (size_t)P + p0 + lane) : 0.f;
    __syncthreads();
    const int c4n = C / 4;
    for (int idx = threadIdx.x; idx < LT_PTS * c4n; idx += LT_THREADS) {
        const int pt = idx / c4n, c4 = idx - pt * c4n;
        if (p0 + pt < P)
            *reinterpret_cast<float4*>(dst + (n * (size_t)P + p0 + pt) * C + 4 * c4) =
                make_float4(tile[4 * c4][pt], tile[4 * c4 + 1][pt], tile[4 * c4 + 2][pt], tile[4 * c4 + 3][pt]);
    }
}

// src: [slices][P][C] (channels last), dst: [slices][C][P] (channels first)
__global__ void __launch_bounds__(LT_THREADS) cl_to_cf_kernel(const float* __restrict__ src, float* __restrict__ dst, int C, long long P) {
    __shared__ float tile[LT_MAXC][LT_PTS + 1];
    const long long p0 = (long long)blockIdx.x * LT_PTS;
    const size_t n = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c4n = C / 4;
    for (int idx = threadIdx.x; idx < LT_PTS * c4n; idx += LT_THREADS) {
        const int pt = idx / c4n, c4 = idx - pt * c4n;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p0 + pt < P) x = __ldg(reinterpret_cast<const float4*>(src + (n * (size_t)P + p0 + pt) * C + 4 * c4));
        tile[4 * c4][pt] = x.x; tile[4 * c4 + 1][pt] = x.y; tile[4 * c4 + 2][pt] = x.z; tile[4 * c4 + 3][pt] = x.w;
    }
    __syncthreads();
    if (p0 + lane < P)
        for (int c = warp; c < C; c += LT_THREADS / 32) dst[(n * C + c) * (size_t)P + p0 + lane] = tile[c][lane];
}

cudaError_t launch(bool to_cl, const float* src, float* dst, int slices, int C, long long P, cudaStream_t stream) {
    if (C <= 0 || C > LT_MAXC || C % 4 != 0 || slices <= 0 || slices > 65535 || P <= 0) return cudaErrorInvalidValue;
    const long long tiles = (P + LT_PTS - 1) / LT_PTS;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)tiles, (unsigned)slices);
    if (to_cl) cf_to_cl_kernel<<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
    else cl_to_cf_kernel<<<grid, LT_THREADS, 0, stream>>>(src, dst, C, P);
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
