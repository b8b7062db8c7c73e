// Fragment-level building blocks shared by the tensor-core (mma.sync) kernels: operand splits, the two- and
// three-MMA products with fp32-level accuracy, and row loads / stores.  See sna_kernels_mma.cu for the fragment
// conventions.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace sna {
namespace mmac {

constexpr int TILE_LON = 8;   // a tile is 8 consecutive longitudes on each of 2 adjacent rings (must match the planner)
constexpr int TILE_LAT = 2;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The MMA reads only the top 19 bits of a TF32 operand (verified on B200), so for operands that are used once
// the raw fp32 word serves as hi and lo = x - trunc19(x) is exact; see split_b2 below.
// Split for operands that are reused over the whole stream (the A operand of a tile): both parts rounded to nearest.
__device__ __forceinline__ void split_rn(float x, uint32_t& hi, uint32_t& lo) {
    const uint32_t h = (__float_as_uint(x) + 0x1000u) & 0xffffe000u;
    hi = h;
    lo = (__float_as_uint(x - __uint_as_float(h)) + 0x1000u) & 0xffffe000u;
}

// The tensor core adds into its fp32 accumulator with truncation (verified: 1 + 1.75*2^-24 -> 1), so a long chain
// of MMAs into one fragment drifts towards zero (measured: 3e-5 relative after ~1000 steps).  Every chain here is
// therefore short: the correction MMAs go first, the main terms last, into a fragment that starts at zero, and long
// sums are carried in fp32 FMAs outside the tensor core.
__device__ __forceinline__ void mma_acc(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// Row fragment (CPT contiguous channels) of the point at `p`, raw.
template <int CPT>
__device__ __forceinline__ void load_row(const float* p, float (&x)[CPT]) {
#pragma unroll
    for (int j = 0; j < CPT / 4; ++j) {
        const float4 a = ldg4(p + 4 * j);
        x[4 * j] = a.x; x[4 * j + 1] = a.y; x[4 * j + 2] = a.z; x[4 * j + 3] = a.w;
    }
}
// ---------------------------------------------------------------------------------------------------------
// Three-MMA product, all TF32: a*b = a_lo*b_hi + a_hi*b_lo + a_hi*b_hi with ~2^-21 relative precision.  Used for
// the scores of the forward pass: softmax turns an absolute score error e into a relative weight error e*ln 2, so
// peaked softmaxes (|s| of tens) need the scores at full fp32-level precision.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
// Persistent A operand (tile rows g and g+8) from the row fragments of the two points, pre-multiplied by `mul`:
// TF32 hi and lo quads per k-step, both rounded to nearest.
template <int CPT>
__device__ __forceinline__ void make_a_operand3(const float* p0, const float* p1, float mul, uint32_t (&hi)[CPT / 2][4], uint32_t (&lo)[CPT / 2][4]) {
    float a[CPT], b[CPT];
    load_row<CPT>(p0, a);
    load_row<CPT>(p1, b);
#pragma unroll
    for (int ks = 0; ks < CPT / 2; ++ks) {
        split_rn(a[2 * ks] * mul, hi[ks][0], lo[ks][0]);       // (row g,   k = t)
        split_rn(b[2 * ks] * mul, hi[ks][1], lo[ks][1]);       // (row g+8, k = t)
        split_rn(a[2 * ks + 1] * mul, hi[ks][2], lo[ks][2]);   // (row g,   k = t+4)
        split_rn(b[2 * ks + 1] * mul, hi[ks][3], lo[ks][3]);   // (row g+8, k = t+4)
    }
}
// d[tl] = A . B^T for the two 8-column tiles of a chunk; B = row fragment x[tl] of the point in column g of tile
// tl, used raw as hi (the MMA truncates it) with lo = x - trunc19(x).  Corrections first, main terms last.
template <int CPT>
__device__ __forceinline__ void rows_dot_points3(float (&d)[2][4], const uint32_t (&ah)[CPT / 2][4], const uint32_t (&al)[CPT / 2][4], const float (&x)[2][CPT]) {
    uint32_t bh[2][CPT], bl[2][CPT];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl)
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            bh[tl][j] = __float_as_uint(x[tl][j]);
            bl[tl][j] = __float_as_uint(x[tl][j] - __uint_as_float(bh[tl][j] & 0xffffe000u));
        }
    mma_zero(d[0], al[0], bh[0][0], bh[0][1]);
    mma_zero(d[1], al[0], bh[1][0], bh[1][1]);
    mma_acc(d[0], ah[0], bl[0][0], bl[0][1]);
    mma_acc(d[1], ah[0], bl[1][0], bl[1][1]);
#pragma unroll
    for (int ks = 1; ks < CPT / 2; ++ks) {
        mma_acc(d[0], al[ks], bh[0][2 * ks], bh[0][2 * ks + 1]);
        mma_acc(d[1], al[ks], bh[1][2 * ks], bh[1][2 * ks + 1]);
        mma_acc(d[0], ah[ks], bl[0][2 * ks], bl[0][2 * ks + 1]);
        mma_acc(d[1], ah[ks], bl[1][2 * ks], bl[1][2 * ks + 1]);
    }
#pragma unroll
    for (int ks = 0; ks < CPT / 2; ++ks) {
        mma_acc(d[0], ah[ks], bh[0][2 * ks], bh[0][2 * ks + 1]);
        mma_acc(d[1], ah[ks], bh[1][2 * ks], bh[1][2 * ks + 1]);
    }
}

// ---------------------------------------------------------------------------------------------------------
// Two-MMA products: the main term a_hi*b_hi is one TF32 MMA and BOTH correction terms a_lo*b_hi + a_hi*b_lo are
// one BF16 m16n8k16 MMA whose 16 k-slots hold [a_lo | a_hi] against [b_hi ; b_lo] for the same 8 channels.  The
// corrections are ~2^-11 of the product, so BF16's 8 bits leave a relative error of 2^-17 (lo parts truncated;
// used by the backward pass, gate 1e-4) or below 2^-19 (lo parts rounded to nearest; forward pass, gate 1e-5), at
// two thirds of the tensor time of three TF32 MMAs.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_acc(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
// {lower half = bf16(x0), upper half = bf16(x1)} by truncation (the upper 16 bits of each fp32 word)
__device__ __forceinline__ uint32_t pack_bf16_trunc(uint32_t x0, uint32_t x1) { return __byte_perm(x0, x1, 0x7632); }
__device__ __forceinline__ uint32_t pack_bf16_rn(float x0, float x1) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
    return r;
}

// Persistent A operand of the two-MMA product: hi[ks] = TF32-rounded values (main term), c16[ks] = BF16 quads
// {lo(row g), lo(row g+8), hi(row g), hi(row g+8)} of the thread's channel pair of k-step ks.
template <int CPT>
__device__ __forceinline__ void make_a_operand2(const float* p0, const float* p1, float mul, uint32_t (&hi)[CPT / 2][4], uint32_t (&c16)[CPT / 2][4]) {
    float a[CPT], b[CPT];
    load_row<CPT>(p0, a);
    load_row<CPT>(p1, b);
#pragma unroll
    for (int ks = 0; ks < CPT / 2; ++ks) {
        uint32_t l[4];
        split_rn(a[2 * ks] * mul, hi[ks][0], l[0]);
        split_rn(b[2 * ks] * mul, hi[ks][1], l[1]);
        split_rn(a[2 * ks + 1] * mul, hi[ks][2], l[2]);
        split_rn(b[2 * ks + 1] * mul, hi[ks][3], l[3]);
        c16[ks][0] = pack_bf16_rn(__uint_as_float(l[0]), __uint_as_float(l[2]));      // row g:   lo of the channel pair
        c16[ks][1] = pack_bf16_rn(__uint_as_float(l[1]), __uint_as_float(l[3]));      // row g+8
        c16[ks][2] = pack_bf16_rn(__uint_as_float(hi[ks][0]), __uint_as_float(hi[ks][2]));   // row g:   hi of the pair
        c16[ks][3] = pack_bf16_rn(__uint_as_float(hi[ks][1]), __uint_as_float(hi[ks][3]));   // row g+8
    }
}

// B operand of one k-step from the raw channel pair (x0, x1): main registers are the raw words; the BF16 pair is
// {hi pair, lo pair} with lo = x - trunc19(x).
template <bool RN = false>
__device__ __forceinline__ void split_b2(float x0, float x1, uint32_t& m0, uint32_t& m1, uint32_t& h16, uint32_t& l16) {
    m0 = __float_as_uint(x0);
    m1 = __float_as_uint(x1);
    const float l0 = x0 - __uint_as_float(m0 & 0xffffe000u), l1 = x1 - __uint_as_float(m1 & 0xffffe000u);
    h16 = pack_bf16_trunc(m0, m1);
    // the lo parts carry the larger correction (2^-10 of the value): rounding them to nearest instead of truncating
    // brings the product's relative error from 2^-17 to below 2^-19, which the forward pass needs
    l16 = RN ? pack_bf16_rn(l0, l1) : pack_bf16_trunc(__float_as_uint(l0), __float_as_uint(l1));
}

// d[tl] = A . B^T for the two 8-column tiles with the two-MMA product (corrections first, then the main terms).
template <int CPT, bool RN = false>
__device__ __forceinline__ void rows_dot_points2(float (&d)[2][4], const uint32_t (&ah)[CPT / 2][4], const uint32_t (&a16)[CPT / 2][4], const float (&x)[2][CPT]) {
    uint32_t bm[2][CPT], bh16[2][CPT / 2], bl16[2][CPT / 2];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl)
#pragma unroll
        for (int ks = 0; ks < CPT / 2; ++ks) split_b2<RN>(x[tl][2 * ks], x[tl][2 * ks + 1], bm[tl][2 * ks], bm[tl][2 * ks + 1], bh16[tl][ks], bl16[tl][ks]);
    mma_bf16_zero(d[0], a16[0], bh16[0][0], bl16[0][0]);
    mma_bf16_zero(d[1], a16[0], bh16[1][0], bl16[1][0]);
#pragma unroll
    for (int ks = 1; ks < CPT / 2; ++ks) {
        mma_bf16_acc(d[0], a16[ks], bh16[0][ks], bl16[0][ks]);
        mma_bf16_acc(d[1], a16[ks], bh16[1][ks], bl16[1][ks]);
    }
#pragma unroll
    for (int ks = 0; ks < CPT / 2; ++ks) {
        mma_acc(d[0], ah[ks], bm[0][2 * ks], bm[0][2 * ks + 1]);
        mma_acc(d[1], ah[ks], bm[1][2 * ks], bm[1][2 * ks + 1]);
    }
}

// Second contraction with the two-MMA product: W (scores layout, 16 x 16 columns) times the column fragments.
// k-slots of the BF16 MMA of tile tl: [W_lo(8 columns) | W_hi(8 columns)] against [X_hi ; X_lo].
template <int KS, bool RN = false>
__device__ __forceinline__ void scores_times_points2(float (&d)[KS][4], const float (&w)[2][4], const float (&x)[2][2][KS]) {
    uint32_t wm[2][4], w16[2][4];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl) {
        uint32_t h[4], l[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            h[i] = __float_as_uint(w[tl][i]);
            l[i] = __float_as_uint(w[tl][i] - __uint_as_float(h[i] & 0xffffe000u));
        }
        wm[tl][0] = h[0]; wm[tl][1] = h[2]; wm[tl][2] = h[1]; wm[tl][3] = h[3];   // TF32 A quad: (g,2t) (g+8,2t) (g,2t+1) (g+8,2t+1)
        w16[tl][0] = RN ? pack_bf16_rn(__uint_as_float(l[0]), __uint_as_float(l[1])) : pack_bf16_trunc(l[0], l[1]);   // row g: lo of columns 2t, 2t+1
        w16[tl][1] = RN ? pack_bf16_rn(__uint_as_float(l[2]), __uint_as_float(l[3])) : pack_bf16_trunc(l[2], l[3]);   // row g+8
        w16[tl][2] = pack_bf16_trunc(h[0], h[1]);   // row g:   hi
        w16[tl][3] = pack_bf16_trunc(h[2], h[3]);   // row g+8
    }
    uint32_t xm[2][2][KS], xh16[2][KS], xl16[2][KS];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl)
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) split_b2<RN>(x[tl][0][nt], x[tl][1][nt], xm[tl][0][nt], xm[tl][1][nt], xh16[tl][nt], xl16[tl][nt]);
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_bf16_zero(d[nt], w16[0], xh16[0][nt], xl16[0][nt]);
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_bf16_acc(d[nt], w16[1], xh16[1][nt], xl16[1][nt]);
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_acc(d[nt], wm[0], xm[0][0][nt], xm[0][1][nt]);
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_acc(d[nt], wm[1], xm[1][0][nt], xm[1][1][nt]);
}

// ---------------------------------------------------------------------------------------------------------
// One-MMA products for the reduced-precision variant: both operands are used as plain TF32 (the tensor core reads the
// top 19 bits of the fp32 words), fp32 accumulation.  Relative error of a product ~2^-11.
// ---------------------------------------------------------------------------------------------------------
template <int CPT>
__device__ __forceinline__ void rows_dot_points1(float (&d)[2][4], const uint32_t (&ah)[CPT / 2][4], const float (&x)[2][CPT]) {
    mma_zero(d[0], ah[0], __float_as_uint(x[0][0]), __float_as_uint(x[0][1]));
    mma_zero(d[1], ah[0], __float_as_uint(x[1][0]), __float_as_uint(x[1][1]));
#pragma unroll
    for (int ks = 1; ks < CPT / 2; ++ks) {
        mma_acc(d[0], ah[ks], __float_as_uint(x[0][2 * ks]), __float_as_uint(x[0][2 * ks + 1]));
        mma_acc(d[1], ah[ks], __float_as_uint(x[1][2 * ks]), __float_as_uint(x[1][2 * ks + 1]));
    }
}
template <int KS>
__device__ __forceinline__ void scores_times_points1(float (&d)[KS][4], const float (&w)[2][4], const float (&x)[2][2][KS]) {
    uint32_t wm[2][4];
#pragma unroll
    for (int tl = 0; tl < 2; ++tl) {
        wm[tl][0] = __float_as_uint(w[tl][0]); wm[tl][1] = __float_as_uint(w[tl][2]);   // TF32 A quad: (g,2t) (g+8,2t) (g,2t+1) (g+8,2t+1)
        wm[tl][2] = __float_as_uint(w[tl][1]); wm[tl][3] = __float_as_uint(w[tl][3]);
    }
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_zero(d[nt], wm[0], __float_as_uint(x[0][0][nt]), __float_as_uint(x[0][1][nt]));
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) mma_acc(d[nt], wm[1], __float_as_uint(x[1][0][nt]), __float_as_uint(x[1][1][nt]));
}

template <int CPT>
__device__ __forceinline__ void store_row(float* p, const float (&x)[CPT]) {
#pragma unroll
    for (int j = 0; j < CPT / 4; ++j) *reinterpret_cast<float4*>(p + 4 * j) = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
}

}  // namespace mmac
}  // namespace sna
