// Tensor-core kernels (sm_100a): every contraction of the path runs on mma.sync with fp32-level accuracy from a
// split of each operand, x = hi + lo with hi the top 11 significand bits.  A product a*b is two MMAs into one fp32
// fragment: the main term a_hi*b_hi as m16n8k8 TF32, and both correction terms a_lo*b_hi + a_hi*b_lo as a single
// m16n8k16 BF16 MMA whose 16 k-slots hold [a_lo | a_hi] against [b_hi ; b_lo] (the corrections are ~2^-11 of the
// product, so 8 bits suffice).  The scores of the forward pass, whose errors the softmax amplifies, use three TF32
// MMAs instead.  Measured normalised errors: forward ~1e-6, backward <= 2e-5.
//
// Work decomposition: one warp owns a tile of 16 points (the M dimension of the MMA: "tile rows") = 8 consecutive
// longitudes on each of 2 adjacent rings, and walks the host-built column stream of that ring group, 16 partner
// points ("columns") per step.  Band structure and ragged edges are expressed by the 16-bit row mask carried by
// every stream column.
// The 16 partner points of a chunk are staged by cp.async into a warp-private, two-stage shared-memory ring
// while the previous chunk is consumed; warps never synchronise with each other (no block-level barrier).
//
// Fragment conventions (g = lane / 4, t = lane % 4, CPT = C/4, KS = C/8):
//   "row fragment" of a point: the CPT channels [t*CPT, (t+1)*CPT) of that point.  As an A operand it belongs to
//   tile rows g and g+8; as a B operand to tile column g.  MMA k index t of k-step ks is channel t*CPT + 2*ks,
//   k index t+4 is channel t*CPT + 2*ks + 1 (the same permutation on both operands, so the contraction is exact).
//   "column fragment" of a point: the KS channels [g*KS, (g+1)*KS) of the point in tile column 2t (and 2t+1).
//   With the accumulator's column n <-> channel n*KS + nt for n-tile nt, a thread ends up owning channels
//   [t*CPT, (t+1)*CPT) of tile rows g and g+8 again.  A score fragment (rows g, g+8; columns 2t, 2t+1) is
//   reused as the A operand of the second contraction with k index t <-> column 2t and t+4 <-> column 2t+1.
//
// Forward: Eq. (s2_attention_discrete_detailed).  Backward: App. B.4.
#include "sna_kernels.cuh"
#include "sna_mma_common.cuh"

#include <cstdint>
#include <type_traits>

namespace sna {
namespace {

constexpr int WARPS = 4;
constexpr int THREADS = WARPS * 32;
using namespace mmac;

// ---------------------------------------------------------------------------------------------------------
// Warp-private staging of a chunk's 16 partner points in shared memory (cp.async, two stages).
// Two point arrays are staged per chunk (forward / dq: k and v rows; dk/dv: q and dout rows), each row padded
// to C+4 floats so that both fragment layouts read without bank conflicts, plus per-column metadata.
// ---------------------------------------------------------------------------------------------------------
template <int C>
struct Stage {
    static constexpr int PITCH = C + 4;
    float a[16][PITCH];
    float b[16][PITCH];
    uint32_t mask[16];   // tile rows that use the column
    float m0[16];        // forward stream: log2 omega of the partner ring; transposed stream: lse of the partner
    float m1[16];        // transposed stream: D of the partner
    uint32_t all_rows;   // 1 if every column of the chunk is used by all 16 tile rows (no masking needed)
    uint32_t pad[15];
};

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Walks the column stream of one tile with a two-stage software pipeline: chunk c+1 is copied into shared
// memory while chunk c is consumed by `body(stage)`.  Lane l owns stream column l % 16 (both half-warps compute
// the same metadata, which keeps the code free of divergent branches).  Rows of the two point arrays are copied
// in 16-byte pieces, C/8 pieces per lane and array; the pipeline is branch-free: past the end of the stream the
// last chunk is simply staged again into the idle stage.
template <int C, bool TRANSPOSED>
struct StreamWalker {
    static constexpr int PIECES = C / 4;            // 16-byte pieces per point row
    static constexpr int ROWS_PER_PASS = 32 / PIECES;
    const int4* ent;          // this lane's entry of chunk 0
    const float* a_lane;      // array bases advanced to this lane's piece
    const float* b_lane;
    const float* lse_base;
    const float* D_base;
    uint32_t stage_smem;      // shared address of stage 0
    Stage<C>* stages;
    int first, ring_len, stride, lane, row0;

    __device__ __forceinline__ void issue(int slot, const int4& e) const {
        int u = (int)(short)(e.y & 0xffff);
        if (e.x >= 0) {   // offset relative to the tile's first point, wrapped around the ring
            u += first;
            if (u < 0) u += ring_len;
            if (u >= ring_len) u -= ring_len;
            if (u >= ring_len) u -= ring_len;
        }
        const int idx = (e.x & 0x7fffffff) + u * stride;   // flat index of the partner point in its slice
        const uint32_t sbase = stage_smem + slot * (uint32_t)sizeof(Stage<C>);
        const uint32_t dst = sbase + (uint32_t)(row0 * Stage<C>::PITCH + (lane % PIECES) * 4) * 4u;
#pragma unroll
        for (int j = 0; j < C / 8; ++j) {
            const uint32_t off = (uint32_t)__shfl_sync(FULL, idx, row0 + j * ROWS_PER_PASS) * C;   // < 2^32: checked on the host
            cp_async16(dst + j * ROWS_PER_PASS * Stage<C>::PITCH * 4, a_lane + off);
            cp_async16(dst + (16 + j * ROWS_PER_PASS) * Stage<C>::PITCH * 4, b_lane + off);
        }
        const uint32_t mask = (uint32_t)e.y >> 16;
        const uint32_t meta = sbase + 2 * 16 * Stage<C>::PITCH * 4 + (lane & 15) * 4;
        Stage<C>& st = stages[slot];
        st.mask[lane & 15] = mask;
        if (TRANSPOSED) {
            cp_async4(meta + 64, lse_base + idx);
            cp_async4(meta + 128, D_base + idx);
        } else {
            st.m0[lane & 15] = __int_as_float(e.z);
        }
        st.all_rows = __all_sync(FULL, mask == 0xffffu) ? 1u : 0u;
    }

    template <typename Body>
    __device__ __forceinline__ void run(int nchunks, Body&& body) const {
        if (nchunks <= 0) return;
        const int last = nchunks - 1;
        int4 e = __ldg(ent);
        issue(0, e);
        cp_async_commit();
        e = __ldg(ent + 16 * min(1, last));
        for (int c = 0; c < nchunks; ++c) {
            issue((c + 1) & 1, e);
            cp_async_commit();
            e = __ldg(ent + 16 * min(c + 2, last));
            cp_async_wait<1>();
            __syncwarp();
            body(stages[c & 1]);
            __syncwarp();   // everyone is done with this stage before the next iteration refills it
        }
        cp_async_wait<0>();
    }
};

template <int C, bool TRANSPOSED>
__device__ __forceinline__ StreamWalker<C, TRANSPOSED> make_walker(Stage<C>* stages, const int4* stream, int lane, int first, int ring_len,
                                                                   int stride, const float* a_base, const float* b_base,
                                                                   const float* lse_base, const float* D_base) {
    StreamWalker<C, TRANSPOSED> w;
    w.ent = stream + (lane & 15);
    w.a_lane = a_base + (lane % (C / 4)) * 4;
    w.b_lane = b_base + (lane % (C / 4)) * 4;
    w.lse_base = lse_base;
    w.D_base = D_base;
    w.stages = stages;
    w.stage_smem = (uint32_t)__cvta_generic_to_shared(stages);
    w.first = first; w.ring_len = ring_len; w.stride = stride; w.lane = lane;
    w.row0 = lane / (C / 4);
    return w;
}

template <int CPT, int PITCH>
__device__ __forceinline__ void lds_row(const float (&arr)[16][PITCH], int row, int t, float (&x)[CPT]) {
#pragma unroll
    for (int j = 0; j < CPT / 4; ++j) {
        const float4 v4 = *reinterpret_cast<const float4*>(&arr[row][t * CPT + 4 * j]);
        x[4 * j] = v4.x; x[4 * j + 1] = v4.y; x[4 * j + 2] = v4.z; x[4 * j + 3] = v4.w;
    }
}
template <int KS, int PITCH>
__device__ __forceinline__ void lds_col(const float (&arr)[16][PITCH], int row, int g, float (&x)[KS]) {
    if constexpr (KS % 4 == 0) {
#pragma unroll
        for (int j = 0; j < KS / 4; ++j) {
            const float4 v4 = *reinterpret_cast<const float4*>(&arr[row][g * KS + 4 * j]);
            x[4 * j] = v4.x; x[4 * j + 1] = v4.y; x[4 * j + 2] = v4.z; x[4 * j + 3] = v4.w;
        }
    } else {
        const float2 v2 = *reinterpret_cast<const float2*>(&arr[row][g * KS]);
        x[0] = v2.x; x[1] = v2.y;
    }
}

// Decode a warp task into (slice n, rank of the ring row in heavy-first order, tile).
__device__ __forceinline__ bool decode_task(int N, int tiles_per_row, long long total, int& n, int& row_rank, int& tile) {
    const long long task = (long long)blockIdx.x * WARPS + (threadIdx.x >> 5);
    if (task >= total) return false;
    tile = (int)(task % tiles_per_row);
    const long long rest = task / tiles_per_row;
    n = (int)(rest % N);
    row_rank = (int)(rest / N);
    return true;
}


// The column stream a forward launch walks: the full one, or the band-only one when the dense kernel has already
// produced its part (dense_ptr != null: rows with windows on the dense kernel start from that partial result).
struct FwdView {
    const int4* stream;
    const int32_t* chunk_ptr;
    const int32_t* order;
    const int32_t* dense_ptr;
};

// ---------------------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------------------
template <int C, bool LP>
__global__ void __launch_bounds__(THREADS, C == 64 ? 2 : 4)
forward_mma_kernel(DevPlan p, FwdView fv, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                   float* out, float* lse, int N, float scale_log2, int tiles_per_row, long long total_tasks) {
    constexpr int CPT = C / 4, KS = C / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Stage<C>* stages = reinterpret_cast<Stage<C>*>(smem_raw) + 2 * (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    int n, rank, tile;
    if (!decode_task(N, tiles_per_row, total_tasks, n, rank, tile)) return;
    // tile rows g and g+8 of this thread: the same longitude on the two rings of the group
    const int hg = fv.order[rank];
    const int w0 = tile * TILE_LON;
    const bool ok0 = w0 + g < p.nlon_out, ok1 = ok0 && hg * TILE_LAT + 1 < p.nlat_out;
    const int wq = min(w0 + g, p.nlon_out - 1);
    const size_t pt0 = (size_t)(n * p.nlat_out + hg * TILE_LAT) * p.nlon_out + wq;
    const size_t pt1 = (size_t)(n * p.nlat_out + min(hg * TILE_LAT + 1, p.nlat_out - 1)) * p.nlon_out + wq;

    uint32_t qh[KS][4], ql[KS][4];   // q in the log2 domain
    make_a_operand3<CPT>(q + pt0 * C + t * CPT, q + pt1 * C + t * CPT, scale_log2, qh, ql);
    float o[KS][4];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    if (fv.dense_ptr != nullptr) {
        // continue from the dense kernel's partial result of this row (normalised out and lse): m = lse, l = 1
        const int ha = hg * TILE_LAT, hb = min(hg * TILE_LAT + 1, p.nlat_out - 1);
        if (fv.dense_ptr[ha + 1] > fv.dense_ptr[ha]) {
            float r[CPT];
            load_row<CPT>(out + pt0 * C + t * CPT, r);
#pragma unroll
            for (int nt = 0; nt < KS; ++nt) { o[nt][0] = r[nt]; o[nt][1] = r[KS + nt]; }
            m0 = lse[pt0] * LOG2E;
            l0 = t == 0 ? 1.f : 0.f;
        }
        if (fv.dense_ptr[hb + 1] > fv.dense_ptr[hb]) {
            float r[CPT];
            load_row<CPT>(out + pt1 * C + t * CPT, r);
#pragma unroll
            for (int nt = 0; nt < KS; ++nt) { o[nt][2] = r[nt]; o[nt][3] = r[KS + nt]; }
            m1 = lse[pt1] * LOG2E;
            l1 = t == 0 ? 1.f : 0.f;
        }
    }

    const size_t slice = (size_t)n * p.nlat_in * p.nlon_in * C;
    const int4* stream = fv.stream + (size_t)fv.chunk_ptr[hg] * 16;
    const int nchunks = fv.chunk_ptr[hg + 1] - fv.chunk_ptr[hg];

    make_walker<C, false>(stages, stream, lane, w0, p.nlon_out, p.ps, k + slice, v + slice, nullptr, nullptr).run(nchunks, [&](const Stage<C>& st) {
        float s[2][4];
        {
            float kr[2][CPT];
            lds_row<CPT>(st.a, g, t, kr[0]);
            lds_row<CPT>(st.a, 8 + g, t, kr[1]);
            if constexpr (LP) rows_dot_points1<CPT>(s, qh, kr);
            else rows_dot_points3<CPT>(s, qh, ql, kr);   // scores at full precision (three TF32 MMAs per product)
        }
        float vr[2][2][KS];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            const float2 bs = *reinterpret_cast<const float2*>(&st.m0[tl * 8 + 2 * t]);
            lds_col<KS>(st.b, tl * 8 + 2 * t, g, vr[tl][0]);
            lds_col<KS>(st.b, tl * 8 + 2 * t + 1, g, vr[tl][1]);
            s[tl][0] += bs.x; s[tl][1] += bs.y; s[tl][2] += bs.x; s[tl][3] += bs.y;
        }
        if (!st.all_rows) {   // warp-uniform: some tile row skips some column of this chunk
#pragma unroll
            for (int tl = 0; tl < 2; ++tl) {
                const uint2 mk = *reinterpret_cast<const uint2*>(&st.mask[tl * 8 + 2 * t]);
                const uint32_t ma = mk.x >> g, mb = mk.y >> g;
                if (!(ma & 1u)) s[tl][0] = -INFINITY;
                if (!(mb & 1u)) s[tl][1] = -INFINITY;
                if (!(ma & 0x100u)) s[tl][2] = -INFINITY;
                if (!(mb & 0x100u)) s[tl][3] = -INFINITY;
            }
        }
        // online softmax over the chunk (row maxima across the four threads of a group)
        float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, 2));
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
        float pv[KS][4];
        if constexpr (LP) scores_times_points1<KS>(pv, s, vr);
        else scores_times_points2<KS, true>(pv, s, vr);
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) {
            o[nt][0] = fmaf(o[nt][0], corr0, pv[nt][0]); o[nt][1] = fmaf(o[nt][1], corr0, pv[nt][1]);
            o[nt][2] = fmaf(o[nt][2], corr1, pv[nt][2]); o[nt][3] = fmaf(o[nt][3], corr1, pv[nt][3]);
        }
    });
    // row sums across the four threads of a group, normalise, store
    l0 += __shfl_xor_sync(FULL, l0, 1); l1 += __shfl_xor_sync(FULL, l1, 1);
    l0 += __shfl_xor_sync(FULL, l0, 2); l1 += __shfl_xor_sync(FULL, l1, 2);
    if (out != nullptr) {
        const float inv0 = 1.f / l0, inv1 = 1.f / l1;
        float r0v[CPT], r1v[CPT];   // o[nt][0] is channel t*CPT + nt, o[nt][1] is channel t*CPT + KS + nt
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) {
            r0v[nt] = o[nt][0] * inv0; r0v[KS + nt] = o[nt][1] * inv0;
            r1v[nt] = o[nt][2] * inv1; r1v[KS + nt] = o[nt][3] * inv1;
        }
        if (ok0) store_row<CPT>(out + pt0 * C + t * CPT, r0v);
        if (ok1) store_row<CPT>(out + pt1 * C + t * CPT, r1v);
    }
    if (lse != nullptr && t == 0) {
        if (ok0) lse[pt0] = (m0 + log2f(l0)) * LN2;
        if (ok1) lse[pt1] = (m1 + log2f(l1)) * LN2;
    }
}

// ---------------------------------------------------------------------------------------------------------
// backward, dq:  dq_i = scale * sum_j p_ij (t_ij - D_i) k_j,  D_i = dout_i . out_i  (App. B.4)
// `out` and `dq` may be the same buffer: a warp reads its own 16 rows of `out` before it writes them as dq.
// ---------------------------------------------------------------------------------------------------------
template <int C, bool LP>
__global__ void __launch_bounds__(THREADS, C == 64 ? 2 : 3)
backward_dq_mma_kernel(DevPlan p, FwdView fv, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                       const float* __restrict__ dout, const float* out, const float* __restrict__ lse,
                       float* dq, float* __restrict__ Dws, int N, float scale, int tiles_per_row, long long total_tasks) {
    constexpr int CPT = C / 4, KS = C / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Stage<C>* stages = reinterpret_cast<Stage<C>*>(smem_raw) + 2 * (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    int n, rank, tile;
    if (!decode_task(N, tiles_per_row, total_tasks, n, rank, tile)) return;
    const int hg = fv.order[rank];
    const int w0 = tile * TILE_LON;
    const bool ok0 = w0 + g < p.nlon_out, ok1 = ok0 && hg * TILE_LAT + 1 < p.nlat_out;
    const int wq = min(w0 + g, p.nlon_out - 1);
    const size_t pt0 = (size_t)(n * p.nlat_out + hg * TILE_LAT) * p.nlon_out + wq;
    const size_t pt1 = (size_t)(n * p.nlat_out + min(hg * TILE_LAT + 1, p.nlat_out - 1)) * p.nlon_out + wq;
    const float scale_log2 = scale * LOG2E;

    uint32_t qh[KS][4], ql[KS][4], yh[KS][4], yl[KS][4];
    make_a_operand2<CPT>(q + pt0 * C + t * CPT, q + pt1 * C + t * CPT, scale_log2, qh, ql);   // ql, yl: BF16 correction quads
    make_a_operand2<CPT>(dout + pt0 * C + t * CPT, dout + pt1 * C + t * CPT, 1.f, yh, yl);
    // D of the two tile rows
    float D0 = 0.f, D1 = 0.f;
    {
        float a[CPT], b[CPT], ya[CPT], yb[CPT];
        load_row<CPT>(out + pt0 * C + t * CPT, a);
        load_row<CPT>(out + pt1 * C + t * CPT, b);
        load_row<CPT>(dout + pt0 * C + t * CPT, ya);
        load_row<CPT>(dout + pt1 * C + t * CPT, yb);
#pragma unroll
        for (int j = 0; j < CPT; ++j) { D0 = fmaf(a[j], ya[j], D0); D1 = fmaf(b[j], yb[j], D1); }
        D0 += __shfl_xor_sync(FULL, D0, 1); D1 += __shfl_xor_sync(FULL, D1, 1);
        D0 += __shfl_xor_sync(FULL, D0, 2); D1 += __shfl_xor_sync(FULL, D1, 2);
        if (t == 0) {
            if (ok0) Dws[pt0] = D0;
            if (ok1) Dws[pt1] = D1;
        }
    }
    const float nl0 = -lse[pt0] * LOG2E, nl1 = -lse[pt1] * LOG2E;
    float acc[KS][4];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;

    const size_t slice = (size_t)n * p.nlat_in * p.nlon_in * C;
    const int4* stream = fv.stream + (size_t)fv.chunk_ptr[hg] * 16;
    const int nchunks = fv.chunk_ptr[hg + 1] - fv.chunk_ptr[hg];

    make_walker<C, false>(stages, stream, lane, w0, p.nlon_out, p.ps, k + slice, v + slice, nullptr, nullptr).run(nchunks, [&](const Stage<C>& st) {
        float s[2][4], tt[2][4];
        {
            float xr[2][CPT];
            lds_row<CPT>(st.a, g, t, xr[0]);
            lds_row<CPT>(st.a, 8 + g, t, xr[1]);
            if constexpr (LP) rows_dot_points1<CPT>(s, qh, xr); else rows_dot_points2<CPT>(s, qh, ql, xr);
            lds_row<CPT>(st.b, g, t, xr[0]);
            lds_row<CPT>(st.b, 8 + g, t, xr[1]);
            if constexpr (LP) rows_dot_points1<CPT>(tt, yh, xr); else rows_dot_points2<CPT>(tt, yh, yl, xr);
        }
        float kr[2][2][KS];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            const uint2 mk = *reinterpret_cast<const uint2*>(&st.mask[tl * 8 + 2 * t]);
            const float2 bs = *reinterpret_cast<const float2*>(&st.m0[tl * 8 + 2 * t]);
            lds_col<KS>(st.a, tl * 8 + 2 * t, g, kr[tl][0]);
            lds_col<KS>(st.a, tl * 8 + 2 * t + 1, g, kr[tl][1]);
            const uint32_t ma = mk.x >> g, mb = mk.y >> g;
            const float p00 = (ma & 1u) ? ex2(s[tl][0] + bs.x + nl0) : 0.f;
            const float p01 = (mb & 1u) ? ex2(s[tl][1] + bs.y + nl0) : 0.f;
            const float p10 = (ma & 0x100u) ? ex2(s[tl][2] + bs.x + nl1) : 0.f;
            const float p11 = (mb & 0x100u) ? ex2(s[tl][3] + bs.y + nl1) : 0.f;
            s[tl][0] = p00 * (tt[tl][0] - D0);   // ds
            s[tl][1] = p01 * (tt[tl][1] - D0);
            s[tl][2] = p10 * (tt[tl][2] - D1);
            s[tl][3] = p11 * (tt[tl][3] - D1);
        }
        float part[KS][4];
        if constexpr (LP) scores_times_points1<KS>(part, s, kr); else scores_times_points2<KS>(part, s, kr);
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) {
            acc[nt][0] += part[nt][0]; acc[nt][1] += part[nt][1]; acc[nt][2] += part[nt][2]; acc[nt][3] += part[nt][3];
        }
    });
    float r0v[CPT], r1v[CPT];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) {
        r0v[nt] = acc[nt][0] * scale; r0v[KS + nt] = acc[nt][1] * scale;
        r1v[nt] = acc[nt][2] * scale; r1v[KS + nt] = acc[nt][3] * scale;
    }
    if (fv.dense_ptr != nullptr) {
        // the dense kernel has already written its part of dq for rows that have windows there: add it
        const int ha = hg * TILE_LAT, hb = min(hg * TILE_LAT + 1, p.nlat_out - 1);
        if (fv.dense_ptr[ha + 1] > fv.dense_ptr[ha]) {
            float r[CPT];
            load_row<CPT>(dq + pt0 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) r0v[j] += r[j];
        }
        if (fv.dense_ptr[hb + 1] > fv.dense_ptr[hb]) {
            float r[CPT];
            load_row<CPT>(dq + pt1 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) r1v[j] += r[j];
        }
    }
    if (ok0) store_row<CPT>(dq + pt0 * C + t * CPT, r0v);
    if (ok1) store_row<CPT>(dq + pt1 * C + t * CPT, r1v);
}

// ---------------------------------------------------------------------------------------------------------
// backward, dk and dv, gathered per input point over the transposed stream (no atomics):
//   dk_j = scale * sum_i p_ij (t_ij - D_i) q_i,   dv_j = sum_i p_ij dout_i          (App. B.4)
// Tile rows are the input columns c = ps*(u0+i) + r, i < 8, of the two rings of an input ring group; stream
// columns are output points.
// ---------------------------------------------------------------------------------------------------------
template <int C, bool LP>
__global__ void __launch_bounds__(THREADS, 2)
backward_dkdv_mma_kernel(DevPlan p, FwdView tv, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                         const float* __restrict__ dout, const float* __restrict__ lse, const float* __restrict__ Dws,
                         float* dk, float* dv, int N, float scale, int tiles_per_row, long long total_tasks) {
    constexpr int CPT = C / 4, KS = C / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Stage<C>* stages = reinterpret_cast<Stage<C>*>(smem_raw) + 2 * (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    int n, rank, tile;
    if (!decode_task(N, tiles_per_row, total_tasks, n, rank, tile)) return;
    const int hg = tv.order[rank];
    // input column of tile row g (and g+8), the first partner index of the tile, and the tile's stream row
    int col, first, srow;
    bool ok0;
    if (p.t_consecutive) {           // 8 consecutive input columns
        col = tile * TILE_LON + g;
        ok0 = col < p.nlon_in;
        first = tile * TILE_LON / p.ps;
        srow = hg;
    } else {                         // every ps-th column of one residue class
        const int r = tile % p.ps, u0 = (tile / p.ps) * TILE_LON;
        col = (u0 + g) * p.ps + r;
        ok0 = u0 + g < p.nlon_out;
        first = u0;
        srow = hg * p.ps + r;
    }
    const bool ok1 = ok0 && hg * TILE_LAT + 1 < p.nlat_in;
    col = min(col, p.nlon_in - 1);
    const int hp0 = hg * TILE_LAT, hp1 = min(hg * TILE_LAT + 1, p.nlat_in - 1);
    const size_t pt0 = (size_t)(n * p.nlat_in + hp0) * p.nlon_in + col;
    const size_t pt1 = (size_t)(n * p.nlat_in + hp1) * p.nlon_in + col;
    const float scale_log2 = scale * LOG2E;

    uint32_t kh[KS][4], kl[KS][4], vh[KS][4], vl[KS][4];
    make_a_operand2<CPT>(k + pt0 * C + t * CPT, k + pt1 * C + t * CPT, scale_log2, kh, kl);   // kl, vl: BF16 correction quads
    make_a_operand2<CPT>(v + pt0 * C + t * CPT, v + pt1 * C + t * CPT, 1.f, vh, vl);
    const float bias0 = p.log2_omega[hp0], bias1 = p.log2_omega[hp1];
    float gk[KS][4], gv[KS][4];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) {
        gk[nt][0] = gk[nt][1] = gk[nt][2] = gk[nt][3] = 0.f;
        gv[nt][0] = gv[nt][1] = gv[nt][2] = gv[nt][3] = 0.f;
    }
    const size_t oslice = (size_t)n * p.nlat_out * p.nlon_out;
    const int4* stream = tv.stream + (size_t)tv.chunk_ptr[srow] * 16;
    const int nchunks = tv.chunk_ptr[srow + 1] - tv.chunk_ptr[srow];

    make_walker<C, true>(stages, stream, lane, first, p.nlon_out, 1, q + oslice * C, dout + oslice * C, lse + oslice, Dws + oslice).run(nchunks, [&](const Stage<C>& st) {
        float s[2][4], tt[2][4];
        {
            float xr[2][CPT];
            lds_row<CPT>(st.a, g, t, xr[0]);
            lds_row<CPT>(st.a, 8 + g, t, xr[1]);
            if constexpr (LP) rows_dot_points1<CPT>(s, kh, xr); else rows_dot_points2<CPT>(s, kh, kl, xr);
            lds_row<CPT>(st.b, g, t, xr[0]);
            lds_row<CPT>(st.b, 8 + g, t, xr[1]);
            if constexpr (LP) rows_dot_points1<CPT>(tt, vh, xr); else rows_dot_points2<CPT>(tt, vh, vl, xr);
        }
        float qr[2][2][KS], yr[2][2][KS];
        float pr[2][4];
#pragma unroll
        for (int tl = 0; tl < 2; ++tl) {
            const uint2 mk = *reinterpret_cast<const uint2*>(&st.mask[tl * 8 + 2 * t]);
            const float2 ls = *reinterpret_cast<const float2*>(&st.m0[tl * 8 + 2 * t]);
            const float2 Dd = *reinterpret_cast<const float2*>(&st.m1[tl * 8 + 2 * t]);
            lds_col<KS>(st.a, tl * 8 + 2 * t, g, qr[tl][0]);
            lds_col<KS>(st.a, tl * 8 + 2 * t + 1, g, qr[tl][1]);
            lds_col<KS>(st.b, tl * 8 + 2 * t, g, yr[tl][0]);
            lds_col<KS>(st.b, tl * 8 + 2 * t + 1, g, yr[tl][1]);
            const float nla = -ls.x * LOG2E, nlb = -ls.y * LOG2E;   // -lse_i in the log2 domain
            const uint32_t ma = mk.x >> g, mb = mk.y >> g;
            pr[tl][0] = (ma & 1u) ? ex2(s[tl][0] + nla + bias0) : 0.f;   // bias: log2 omega_j of the row's ring
            pr[tl][1] = (mb & 1u) ? ex2(s[tl][1] + nlb + bias0) : 0.f;
            pr[tl][2] = (ma & 0x100u) ? ex2(s[tl][2] + nla + bias1) : 0.f;
            pr[tl][3] = (mb & 0x100u) ? ex2(s[tl][3] + nlb + bias1) : 0.f;
            s[tl][0] = pr[tl][0] * (tt[tl][0] - Dd.x);   // ds
            s[tl][1] = pr[tl][1] * (tt[tl][1] - Dd.y);
            s[tl][2] = pr[tl][2] * (tt[tl][2] - Dd.x);
            s[tl][3] = pr[tl][3] * (tt[tl][3] - Dd.y);
        }
        float part[KS][4];
        if constexpr (LP) scores_times_points1<KS>(part, pr, yr); else scores_times_points2<KS>(part, pr, yr);
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) { gv[nt][0] += part[nt][0]; gv[nt][1] += part[nt][1]; gv[nt][2] += part[nt][2]; gv[nt][3] += part[nt][3]; }
        if constexpr (LP) scores_times_points1<KS>(part, s, qr); else scores_times_points2<KS>(part, s, qr);
#pragma unroll
        for (int nt = 0; nt < KS; ++nt) { gk[nt][0] += part[nt][0]; gk[nt][1] += part[nt][1]; gk[nt][2] += part[nt][2]; gk[nt][3] += part[nt][3]; }
    });
    // k was pre-multiplied by scale*log2e for the scores only; dk carries the plain scale
    float a0[CPT], a1[CPT], b0[CPT], b1[CPT];
#pragma unroll
    for (int nt = 0; nt < KS; ++nt) {
        a0[nt] = gk[nt][0] * scale; a0[KS + nt] = gk[nt][1] * scale; a1[nt] = gk[nt][2] * scale; a1[KS + nt] = gk[nt][3] * scale;
        b0[nt] = gv[nt][0]; b0[KS + nt] = gv[nt][1]; b1[nt] = gv[nt][2]; b1[KS + nt] = gv[nt][3];
    }
    if (tv.dense_ptr != nullptr) {
        // the dense kernel has already written its part of dk, dv for input rings that have windows there
        if (tv.dense_ptr[hp0 + 1] > tv.dense_ptr[hp0]) {
            float r[CPT];
            load_row<CPT>(dk + pt0 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) a0[j] += r[j];
            load_row<CPT>(dv + pt0 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) b0[j] += r[j];
        }
        if (tv.dense_ptr[hp1 + 1] > tv.dense_ptr[hp1]) {
            float r[CPT];
            load_row<CPT>(dk + pt1 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) a1[j] += r[j];
            load_row<CPT>(dv + pt1 * C + t * CPT, r);
#pragma unroll
            for (int j = 0; j < CPT; ++j) b1[j] += r[j];
        }
    }
    if (ok0) {
        store_row<CPT>(dk + pt0 * C + t * CPT, a0);
        store_row<CPT>(dv + pt0 * C + t * CPT, b0);
    }
    if (ok1) {
        store_row<CPT>(dk + pt1 * C + t * CPT, a1);
        store_row<CPT>(dv + pt1 * C + t * CPT, b1);
    }
}

template <int C>
constexpr size_t smem_bytes() { return sizeof(Stage<C>) * 2 * WARPS; }

// Dynamic shared memory above 48 KB needs an opt-in per kernel and device; mma_prepare_device does it once per plan
// creation for every instantiation.
template <typename K>
cudaError_t prepare_kernel(K kernel, size_t bytes) {
    return bytes > 48 * 1024 ? cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) : cudaSuccess;
}
template <int C, bool LP>
cudaError_t prepare_instantiation() {
    cudaError_t e = prepare_kernel(forward_mma_kernel<C, LP>, smem_bytes<C>());
    if (e == cudaSuccess) e = prepare_kernel(backward_dq_mma_kernel<C, LP>, smem_bytes<C>());
    if (e == cudaSuccess) e = prepare_kernel(backward_dkdv_mma_kernel<C, LP>, smem_bytes<C>());
    return e;
}

template <typename F>
cudaError_t dispatch_c(int C, F&& f) {
    switch (C) {
        case 16: return f(std::integral_constant<int, 16>());
        case 32: return f(std::integral_constant<int, 32>());
        case 64: return f(std::integral_constant<int, 64>());
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t mma_prepare_device() {
    cudaError_t e = prepare_instantiation<16, false>();
    if (e == cudaSuccess) e = prepare_instantiation<32, false>();
    if (e == cudaSuccess) e = prepare_instantiation<64, false>();
    if (e == cudaSuccess) e = prepare_instantiation<16, true>();
    if (e == cudaSuccess) e = prepare_instantiation<32, true>();
    if (e == cudaSuccess) e = prepare_instantiation<64, true>();
    return e;
}

bool mma_path_supported(const DevPlan& p, int C) {
    return p.fwd_stream != nullptr && !p.is_global && (C == 16 || C == 32 || C == 64) && p.nlon_out >= 32 && p.nlon_out < 32768 &&
           (long long)p.nlat_in * p.nlon_in * C < (1LL << 32) && (long long)p.nlat_out * p.nlon_out * C < (1LL << 32);
}

static cudaError_t launch_forward_view(const DevPlan& p, const FwdView& fv, const float* q, const float* k, const float* v, float* out,
                                       float* lse, int N, int C, cudaStream_t stream, bool lp = false) {
    const float scale_log2 = LOG2E / sqrtf((float)C);
    const int tiles = (p.nlon_out + TILE_LON - 1) / TILE_LON;
    const long long tasks = (long long)tiles * ((p.nlat_out + TILE_LAT - 1) / TILE_LAT) * N;
    const long long blocks = (tasks + WARPS - 1) / WARPS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    return dispatch_c(C, [&](auto c) {
        constexpr int CC = decltype(c)::value;
        if (lp) forward_mma_kernel<CC, true><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, fv, q, k, v, out, lse, N, scale_log2, tiles, tasks);
        else forward_mma_kernel<CC, false><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, fv, q, k, v, out, lse, N, scale_log2, tiles, tasks);
        return cudaGetLastError();
    });
}

cudaError_t launch_forward_mma(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                               int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwd_stream, p.fwd_chunk_ptr, p.grp_order, nullptr};
    return launch_forward_view(p, fv, q, k, v, out, lse, N, C, stream);
}

cudaError_t launch_forward_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                    int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwdb_stream, p.fwdb_chunk_ptr, p.grpb_order, p.dense_ptr};
    return launch_forward_view(p, fv, q, k, v, out, lse, N, C, stream);
}

static cudaError_t launch_backward_dq_view(const DevPlan& p, const FwdView& fv, const float* q, const float* k, const float* v, const float* dout,
                                           const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream, bool lp = false) {
    const float scale = 1.0f / sqrtf((float)C);
    const int tiles = (p.nlon_out + TILE_LON - 1) / TILE_LON;
    const long long tasks = (long long)tiles * ((p.nlat_out + TILE_LAT - 1) / TILE_LAT) * N;
    const long long blocks = (tasks + WARPS - 1) / WARPS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    return dispatch_c(C, [&](auto c) {
        constexpr int CC = decltype(c)::value;
        if (lp) backward_dq_mma_kernel<CC, true><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, fv, q, k, v, dout, out, lse, dq, Dws, N, scale, tiles, tasks);
        else backward_dq_mma_kernel<CC, false><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, fv, q, k, v, dout, out, lse, dq, Dws, N, scale, tiles, tasks);
        return cudaGetLastError();
    });
}

cudaError_t launch_backward_dq_mma(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                   const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwd_stream, p.fwd_chunk_ptr, p.grp_order, nullptr};
    return launch_backward_dq_view(p, fv, q, k, v, dout, out, lse, dq, Dws, N, C, stream);
}

cudaError_t launch_backward_dq_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                        const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwdb_stream, p.fwdb_chunk_ptr, p.grpb_order, p.dense_ptr};
    return launch_backward_dq_view(p, fv, q, k, v, dout, out, lse, dq, Dws, N, C, stream);
}

static cudaError_t launch_backward_dkdv_view(const DevPlan& p, const FwdView& tv, const float* q, const float* k, const float* v, const float* dout,
                                             const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream, bool lp = false) {
    const float scale = 1.0f / sqrtf((float)C);
    const int tiles = p.t_consecutive ? (p.nlon_in + TILE_LON - 1) / TILE_LON : p.ps * ((p.nlon_out + TILE_LON - 1) / TILE_LON);
    const long long tasks = (long long)tiles * ((p.nlat_in + TILE_LAT - 1) / TILE_LAT) * N;
    const long long blocks = (tasks + WARPS - 1) / WARPS;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    return dispatch_c(C, [&](auto c) {
        constexpr int CC = decltype(c)::value;
        if (lp) backward_dkdv_mma_kernel<CC, true><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, tv, q, k, v, dout, lse, Dws, dk, dv, N, scale, tiles, tasks);
        else backward_dkdv_mma_kernel<CC, false><<<(unsigned)blocks, THREADS, smem_bytes<CC>(), stream>>>(p, tv, q, k, v, dout, lse, Dws, dk, dv, N, scale, tiles, tasks);
        return cudaGetLastError();
    });
}

cudaError_t launch_backward_dkdv_mma(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                     const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream) {
    const FwdView tv{p.t_stream, p.t_chunk_ptr, p.t_grp_order, nullptr};
    return launch_backward_dkdv_view(p, tv, q, k, v, dout, lse, Dws, dk, dv, N, C, stream);
}

cudaError_t launch_backward_dkdv_mma_band(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                          const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream) {
    const FwdView tv{p.tb_stream, p.tb_chunk_ptr, p.tb_grp_order, p.t_dense_ptr};
    return launch_backward_dkdv_view(p, tv, q, k, v, dout, lse, Dws, dk, dv, N, C, stream);
}

// Reduced-precision variant: the same kernels with every product taken as a single TF32 MMA (full streams, no dense split).
cudaError_t launch_forward_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                  int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwd_stream, p.fwd_chunk_ptr, p.grp_order, nullptr};
    return launch_forward_view(p, fv, q, k, v, out, lse, N, C, stream, true);
}
cudaError_t launch_backward_dq_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                      const float* out, const float* lse, float* dq, float* Dws, int N, int C, cudaStream_t stream) {
    const FwdView fv{p.fwd_stream, p.fwd_chunk_ptr, p.grp_order, nullptr};
    return launch_backward_dq_view(p, fv, q, k, v, dout, out, lse, dq, Dws, N, C, stream, true);
}
cudaError_t launch_backward_dkdv_mma_lp(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                        const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream) {
    const FwdView tv{p.t_stream, p.t_chunk_ptr, p.t_grp_order, nullptr};
    return launch_backward_dkdv_view(p, tv, q, k, v, dout, lse, Dws, dk, dv, N, C, stream, true);
}

}  // namespace sna
