// Tensor-core kernels (sm_100a): every contraction of the path runs on mma.sync m16n8k8 TF32 with a three-term
// split (x = hi + lo; hi*hi + lo*hi + hi*lo, fp32 accumulate), which keeps fp32-level accuracy
// (measured ~1e-6 normalised error) at four times the FP32 FMA rate for dense tiles.
//
// Work decomposition: one warp owns 16 consecutive points of one ring (the M dimension of the MMA) and walks
// the host-built column stream of that ring row, 16 partner points per step.  Band structure and ragged edges
// are expressed by the 16-bit row mask carried by every stream column; masked scores become -inf.
// Operands are loaded straight from global memory (L1/L2) in fragment order; warps never synchronise with
// each other, and there is no shared memory.
//
// Forward: Eq. (s2_attention_discrete_detailed).  Backward: App. B.4.
#include "sna_kernels.cuh"

#include <cstdint>

namespace sna {
namespace {

constexpr int WARPS = 8;
constexpr int THREADS = WARPS * 32;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// x ~ hi + lo, both rounded to nearest to 11 significand bits by integer add (a truncated lo would bias long sums).
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
    const uint32_t h = (__float_as_uint(x) + 0x1000u) & 0xffffe000u;
    hi = h;
    lo = (__float_as_uint(x - __uint_as_float(h)) + 0x1000u) & 0xffffe000u;
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The tensor core adds into its fp32 accumulator with truncation, so a long chain of MMAs into one fragment
// drifts towards zero (measured: 3e-5 relative after ~1000 steps).  Every chain here is therefore short: the
// small correction terms lo*hi + hi*lo go first, the main terms hi*hi last, into a fragment that starts at
// zero, and long sums are carried in fp32 FMAs outside the tensor core.
__device__ __forceinline__ void mma_corr(float (&d)[4], const uint32_t (&ah)[4], const uint32_t (&al)[4],
                                         uint32_t bh0, uint32_t bh1, uint32_t bl0, uint32_t bl1) {
    mma_tf32(d, al[0], al[1], al[2], al[3], bh0, bh1);
    mma_tf32(d, ah[0], ah[1], ah[2], ah[3], bl0, bl1);
}
__device__ __forceinline__ void mma_main(float (&d)[4], const uint32_t (&ah)[4], uint32_t bh0, uint32_t bh1) {
    mma_tf32(d, ah[0], ah[1], ah[2], ah[3], bh0, bh1);
}

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// Flat index (within one batch*head slice) of the partner point of a stream column for a tile starting at w0.
__device__ __forceinline__ int partner_index(const int4& e, int w0, int nlon_tile, int stride) {
    int u = (int)(short)(e.y & 0xffff);
    if (e.x >= 0) {            // relative to the tile
        u += w0;
        if (u < 0) u += nlon_tile;
        if (u >= nlon_tile) u -= nlon_tile;
        if (u >= nlon_tile) u -= nlon_tile;
    }
    return (e.x & 0x7fffffff) + u * stride;
}

// ---------------------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------------------
template <int C>
__global__ void __launch_bounds__(THREADS)
forward_mma_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                   float* __restrict__ out, float* __restrict__ lse, int N, float scale_log2, int tiles_per_row, long long total_tasks) {
    constexpr int CPT = C / 4;    // channels per thread in A/C fragments (thread t owns [t*CPT, (t+1)*CPT))
    constexpr int KS = C / 8;     // k-steps of q.k, and n-tiles of p.v
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const long long task = (long long)blockIdx.x * WARPS + (threadIdx.x >> 5);
    if (task >= total_tasks) return;
    const int tile = (int)(task % tiles_per_row);
    const long long rest = task / tiles_per_row;
    const int n = (int)(rest % N);
    const int h = p.row_order[rest / N];
    const int w0 = tile * 16;
    const int r0 = min(w0 + g, p.nlon_out - 1), r1 = min(w0 + g + 8, p.nlon_out - 1);   // clamped tile rows
    const size_t orow = (size_t)(n * p.nlat_out + h) * p.nlon_out;

    // A fragments of q (pre-scaled into the log2 domain), split once
    uint32_t qh[KS][4], ql[KS][4];
    {
        const float* q0 = q + (orow + r0) * C + t * CPT;
        const float* q1 = q + (orow + r1) * C + t * CPT;
#pragma unroll
        for (int j = 0; j < CPT / 4; ++j) {
            const float4 a = ldg4(q0 + 4 * j), b = ldg4(q1 + 4 * j);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; i += 2) {
                const int ks = (4 * j + i) / 2;
                split_tf32(av[i] * scale_log2, qh[ks][0], ql[ks][0]);       // (row g,   k = t)
                split_tf32(bv[i] * scale_log2, qh[ks][1], ql[ks][1]);       // (row g+8, k = t)
                split_tf32(av[i + 1] * scale_log2, qh[ks][2], ql[ks][2]);   // (row g,   k = t+4)
                split_tf32(bv[i + 1] * scale_log2, qh[ks][3], ql[ks][3]);   // (row g+8, k = t+4)
            }
        }
    }
    float o[KS][4];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    const float* kb = k + (size_t)n * p.nlat_in * p.nlon_in * C;
    const float* vb = v + (size_t)n * p.nlat_in * p.nlon_in * C;
    const int4* stream = p.fwd_stream + (size_t)p.fwd_chunk_ptr[h] * 16;
    const int nchunks = p.fwd_chunk_ptr[h + 1] - p.fwd_chunk_ptr[h];

    for (int c = 0; c < nchunks; ++c) {
        const int4* ce = stream + c * 16;
        // two 8-column tiles: columns g (K operand) and 2t, 2t+1 (scores / V operand) of each
        float s[2][4];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            const int4 ek = __ldg(ce + tl * 8 + g);
            const float* kp = kb + (size_t)partner_index(ek, w0, p.nlon_out, p.ps) * C + t * CPT;
            float kr[CPT];
#pragma unroll
            for (int j = 0; j < CPT / 4; ++j) {
                const float4 a = ldg4(kp + 4 * j);
                kr[4 * j] = a.x; kr[4 * j + 1] = a.y; kr[4 * j + 2] = a.z; kr[4 * j + 3] = a.w;
            }
            s[tl][0] = s[tl][1] = s[tl][2] = s[tl][3] = 0.f;
            uint32_t kh[CPT], kl[CPT];
#pragma unroll
            for (int j = 0; j < CPT; ++j) split_tf32(kr[j], kh[j], kl[j]);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) mma_corr(s[tl], qh[ks], ql[ks], kh[2 * ks], kh[2 * ks + 1], kl[2 * ks], kl[2 * ks + 1]);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) mma_main(s[tl], qh[ks], kh[2 * ks], kh[2 * ks + 1]);
        }
        // bias (log2 omega), mask, online softmax
        int4 ev[2][2];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            ev[tl][0] = __ldg(ce + tl * 8 + 2 * t);
            ev[tl][1] = __ldg(ce + tl * 8 + 2 * t + 1);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float bias = __int_as_float(ev[tl][j].z);
                const uint32_t mask = (uint32_t)ev[tl][j].y >> 16;
                s[tl][j] = (mask >> g) & 1u ? s[tl][j] + bias : -INFINITY;
                s[tl][2 + j] = (mask >> (g + 8)) & 1u ? s[tl][2 + j] + bias : -INFINITY;
            }
        }
        float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0, ms1 = mn1 == -INFINITY ? 0.f : mn1;
        const float corr0 = ex2(m0 - ms0), corr1 = ex2(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            s[tl][0] = ex2(s[tl][0] - ms0); s[tl][1] = ex2(s[tl][1] - ms0);
            s[tl][2] = ex2(s[tl][2] - ms1); s[tl][3] = ex2(s[tl][3] - ms1);
            ps0 += s[tl][0] + s[tl][1];
            ps1 += s[tl][2] + s[tl][3];
        }
        l0 = fmaf(l0, corr0, ps0);
        l1 = fmaf(l1, corr1, ps1);
        // this chunk's P V goes into a zeroed fragment; P (A operand) comes from the score fragments with
        // k index t <-> tile column 2t and t+4 <-> 2t+1
        float pv[KS][4];
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) pv[nt][0] = pv[nt][1] = pv[nt][2] = pv[nt][3] = 0.f;
        uint32_t ph[2][4], pl[2][4], vh[2][2][KS], vl[2][2][KS];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            split_tf32(s[tl][0], ph[tl][0], pl[tl][0]);
            split_tf32(s[tl][2], ph[tl][1], pl[tl][1]);
            split_tf32(s[tl][1], ph[tl][2], pl[tl][2]);
            split_tf32(s[tl][3], ph[tl][3], pl[tl][3]);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float* vp = vb + (size_t)partner_index(ev[tl][j], w0, p.nlon_out, p.ps) * C + g * KS;
                float vr[KS];
                if constexpr (KS % 4 == 0) {
#pragma unroll
                    for (int i = 0; i < KS / 4; ++i) {
                        const float4 a = ldg4(vp + 4 * i);
                        vr[4 * i] = a.x; vr[4 * i + 1] = a.y; vr[4 * i + 2] = a.z; vr[4 * i + 3] = a.w;
                    }
                } else {
                    const float2 a = __ldg(reinterpret_cast<const float2*>(vp));
                    vr[0] = a.x; vr[1] = a.y;
                }
#pragma unroll
                for (int nt = 0; nt < KS; ++nt) split_tf32(vr[nt], vh[tl][j][nt], vl[tl][j][nt]);
            }
        }
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) {
#pragma unroll
            for (int tl = 0; tl < 2; ++tl) mma_corr(pv[nt], ph[tl], pl[tl], vh[tl][0][nt], vh[tl][1][nt], vl[tl][0][nt], vl[tl][1][nt]);
#pragma unroll
            for (int tl = 0; tl < 2; ++tl) mma_main(pv[nt], ph[tl], vh[tl][0][nt], vh[tl][1][nt]);
            o[nt][0] = fmaf(o[nt][0], corr0, pv[nt][0]); o[nt][1] = fmaf(o[nt][1], corr0, pv[nt][1]);
            o[nt][2] = fmaf(o[nt][2], corr1, pv[nt][2]); o[nt][3] = fmaf(o[nt][3], corr1, pv[nt][3]);
        }
    }
    // row sums across the four threads of a group, normalise, store
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;
    // thread owns channels t*CPT + {2t'-style interleave}: o[nt][0] -> channel 2t*KS + nt, o[nt][1] -> (2t+1)*KS + nt
    if (out != nullptr) {
        float* o0 = out + (orow + w0 + g) * C + t * CPT;
        float* o1 = out + (orow + w0 + g + 8) * C + t * CPT;
        float r0v[CPT], r1v[CPT];
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) {
            r0v[nt] = o[nt][0] * inv0; r0v[KS + nt] = o[nt][1] * inv0;
            r1v[nt] = o[nt][2] * inv1; r1v[KS + nt] = o[nt][3] * inv1;
        }
        if (w0 + g < p.nlon_out) {
#pragma unroll
            for (int j = 0; j < CPT / 4; ++j) *reinterpret_cast<float4*>(o0 + 4 * j) = make_float4(r0v[4 * j], r0v[4 * j + 1], r0v[4 * j + 2], r0v[4 * j + 3]);
        }
        if (w0 + g + 8 < p.nlon_out) {
#pragma unroll
            for (int j = 0; j < CPT / 4; ++j) *reinterpret_cast<float4*>(o1 + 4 * j) = make_float4(r1v[4 * j], r1v[4 * j + 1], r1v[4 * j + 2], r1v[4 * j + 3]);
        }
    }
    if (lse != nullptr && t == 0) {
        if (w0 + g < p.nlon_out) lse[orow + w0 + g] = (m0 + log2f(l0)) * LN2;
        if (w0 + g + 8 < p.nlon_out) lse[orow + w0 + g + 8] = (m1 + log2f(l1)) * LN2;
    }
}

}  // namespace

bool mma_path_supported(const DevPlan& p, int C) {
    return p.fwd_stream != nullptr && (C == 16 || C == 32 || C == 64) && p.nlon_out >= 32 && p.nlon_out < 32768;
}

cudaError_t launch_forward_mma(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                               int N, int C, cudaStream_t stream) {
    const float scale_log2 = LOG2E / sqrtf((float)C);
    const int tiles = (p.nlon_out + 15) / 16;
    const long long tasks = (long long)tiles * p.nlat_out * N;
    const long long blocks = (tasks + WARPS - 1) / WARPS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    switch (C) {
        case 16: forward_mma_kernel<16><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, out, lse, N, scale_log2, tiles, tasks); break;
        case 32: forward_mma_kernel<32><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, out, lse, N, scale_log2, tiles, tasks); break;
        case 64: forward_mma_kernel<64><<<(unsigned)blocks, THREADS, 0, stream>>>(p, q, k, v, out, lse, N, scale_log2, tiles, tasks); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace sna
