// Dense forward kernel for whole-ring windows on the 5th-generation tensor cores (tcgen05 / TMEM), sm_100a.
//
// Near the poles, and in the global limit theta_cutoff = pi, an output ring attends to EVERY point of an input
// ring.  That part of Eq. (s2_attention_discrete_detailed) is an ordinary dense attention block, so it runs as
// UMMA GEMMs: one CTA owns 128 consecutive output longitudes of one ring (the M = 128 rows of the MMA), walks the
// ring's whole input rings in blocks of 64 columns, and for every block
//   1. splits the k and v rows into hi = top 11 significand bits and lo = remainder and writes them to shared
//      memory in the K-major 128-byte-swizzle layout (v transposed, so that the columns are its K dimension),
//   2. S = Q K^T as three TF32 UMMAs per k-step (q_lo k_hi + q_hi k_lo + q_hi k_hi) into TMEM,
//   3. reads its row of S from TMEM (thread r owns tile row r), does the online softmax in registers and writes
//      P_hi and P_lo back to TMEM,
//   4. O_block = P V with the A operand taken from TMEM, again three UMMAs per k-step,
//   5. folds O_block into fp32 register accumulators (the tensor core's accumulate truncates, so chains stay short).
// The result (normalised out and lse of the dense part) is the initial state of the band kernel.
// Every wait on an mbarrier is bounded; a wait that runs out sets the plan's device status word and the CTA leaves.
#include "sna_kernels.cuh"

#include <cstdint>

namespace sna {
namespace {

constexpr int DM = 128;        // tile rows (output longitudes)
constexpr int DBN = 64;        // columns per block
constexpr int DC = 32;         // channels
constexpr int TMEM_COLS = 256; // S 64 | P_hi 64 | P_lo 64 | O 32 (power of two allocation)
constexpr size_t DENSE_SMEM = 100 * 1024;   // 64 KB of tiles + alignment; sized so that two CTAs share an SM (and its 512 TMEM columns)
constexpr float LOG2E_D = 1.4426950408889634f;
constexpr float LN2_D = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ float ex2d(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// Shared-memory matrix descriptor, K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3fff) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulator, TF32 operands, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(DM >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(0u));
}
__device__ __forceinline__ void umma_ts(uint32_t d, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d), "r"(a_tmem), "l"(b), "r"(idesc), "r"(acc), "r"(0u));
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity) {
    uint32_t done = 0;
    for (int it = 0; it < (1 << 20) && !done; ++it)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
__device__ __forceinline__ void tmem_ld32(uint32_t (&r)[32], uint32_t addr) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]),"=r"(r[1]),"=r"(r[2]),"=r"(r[3]),"=r"(r[4]),"=r"(r[5]),"=r"(r[6]),"=r"(r[7]),"=r"(r[8]),"=r"(r[9]),"=r"(r[10]),"=r"(r[11]),"=r"(r[12]),"=r"(r[13]),"=r"(r[14]),"=r"(r[15]),
          "=r"(r[16]),"=r"(r[17]),"=r"(r[18]),"=r"(r[19]),"=r"(r[20]),"=r"(r[21]),"=r"(r[22]),"=r"(r[23]),"=r"(r[24]),"=r"(r[25]),"=r"(r[26]),"=r"(r[27]),"=r"(r[28]),"=r"(r[29]),"=r"(r[30]),"=r"(r[31]) : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t addr, const uint32_t (&r)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        :: "r"(addr), "r"(r[0]),"r"(r[1]),"r"(r[2]),"r"(r[3]),"r"(r[4]),"r"(r[5]),"r"(r[6]),"r"(r[7]),"r"(r[8]),"r"(r[9]),"r"(r[10]),"r"(r[11]),"r"(r[12]),"r"(r[13]),"r"(r[14]),"r"(r[15]),
           "r"(r[16]),"r"(r[17]),"r"(r[18]),"r"(r[19]),"r"(r[20]),"r"(r[21]),"r"(r[22]),"r"(r[23]),"r"(r[24]),"r"(r[25]),"r"(r[26]),"r"(r[27]),"r"(r[28]),"r"(r[29]),"r"(r[30]),"r"(r[31]) : "memory");
}
// BF16 UMMA (K = 16 per instruction) for the stacked correction terms: the 16 k-slots of a step hold
// [a_lo(8) | a_hi(8)] on the A side against [b_hi(8) ; b_lo(8)] on the B side, so one instruction adds
// a_lo*b_hi + a_hi*b_lo for 8 contraction indices.  A step is 32 bytes, like a TF32 step.
__device__ __forceinline__ uint32_t umma_idesc16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(DM >> 4) << 24);
}
__device__ __forceinline__ void umma_ss16(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(0u));
}
__device__ __forceinline__ void umma_ts16(uint32_t d, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d), "r"(a_tmem), "l"(b), "r"(idesc), "r"(acc), "r"(0u));
}
// {low half = bf16(x0), high half = bf16(x1)}, round to nearest
__device__ __forceinline__ uint32_t bf16x2(float x0, float x1) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
    return r;
}
__device__ __forceinline__ float trunc19(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }
// Eight values as one 16-byte chunk of BF16.
__device__ __forceinline__ uint4 bf16x8(const float (&x)[8]) {
    return make_uint4(bf16x2(x[0], x[1]), bf16x2(x[2], x[3]), bf16x2(x[4], x[5]), bf16x2(x[6], x[7]));
}
// A operand in TMEM for the stacked product: per group of 8 columns, 4 words of lo pairs then 4 words of hi pairs.
// src holds the fp32 values of 32 columns, dst receives the 32 packed words.
__device__ __forceinline__ void pack_a16(const uint32_t (&src)[32], uint32_t (&dst)[32]) {
#pragma unroll
    for (int gq = 0; gq < 4; ++gq) {
        float hi[8], lo[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { hi[i] = trunc19(__uint_as_float(src[gq * 8 + i])); lo[i] = __uint_as_float(src[gq * 8 + i]) - hi[i]; }
#pragma unroll
        for (int i = 0; i < 4; ++i) { dst[gq * 8 + i] = bf16x2(lo[2 * i], lo[2 * i + 1]); dst[gq * 8 + 4 + i] = bf16x2(hi[2 * i], hi[2 * i + 1]); }
    }
}
__device__ __forceinline__ void tmem_ld16(uint32_t (&r)[16], uint32_t addr) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]),"=r"(r[1]),"=r"(r[2]),"=r"(r[3]),"=r"(r[4]),"=r"(r[5]),"=r"(r[6]),"=r"(r[7]),"=r"(r[8]),"=r"(r[9]),"=r"(r[10]),"=r"(r[11]),"=r"(r[12]),"=r"(r[13]),"=r"(r[14]),"=r"(r[15]) : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&r)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        :: "r"(addr), "r"(r[0]),"r"(r[1]),"r"(r[2]),"r"(r[3]),"r"(r[4]),"r"(r[5]),"r"(r[6]),"r"(r[7]),"r"(r[8]),"r"(r[9]),"r"(r[10]),"r"(r[11]),"r"(r[12]),"r"(r[13]),"r"(r[14]),"r"(r[15]) : "memory");
}
// pack_a16 for 16 columns (two groups of 8)
__device__ __forceinline__ void pack_a16_16(const uint32_t (&src)[16], uint32_t (&dst)[16]) {
#pragma unroll
    for (int gq = 0; gq < 2; ++gq) {
        float hi[8], lo[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { hi[i] = trunc19(__uint_as_float(src[gq * 8 + i])); lo[i] = __uint_as_float(src[gq * 8 + i]) - hi[i]; }
#pragma unroll
        for (int i = 0; i < 4; ++i) { dst[gq * 8 + i] = bf16x2(lo[2 * i], lo[2 * i + 1]); dst[gq * 8 + 4 + i] = bf16x2(hi[2 * i], hi[2 * i + 1]); }
    }
}
// Byte offset of the 16-byte chunk c4 of row r inside a [rows x 128 B] swizzled block.
__device__ __forceinline__ int sw_chunk(int r, int c4) { return r * 128 + ((c4 ^ (r & 7)) << 4); }
// Eight consecutive channels (group grp) of a point as the two chunks of a stacked BF16 row tile.  A operand: lo then hi;
// B operand: hi then lo.
__device__ __forceinline__ void st_stacked8(unsigned char* tile, int row, int grp, const float (&x)[8], bool a_side) {
    float hi[8], lo[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { hi[i] = trunc19(x[i]); lo[i] = x[i] - hi[i]; }
    *reinterpret_cast<uint4*>(tile + sw_chunk(row, 2 * grp)) = a_side ? bf16x8(lo) : bf16x8(hi);
    *reinterpret_cast<uint4*>(tile + sw_chunk(row, 2 * grp + 1)) = a_side ? bf16x8(hi) : bf16x8(lo);
}
// Element (row = channel ch, partner column col) of a transposed stacked BF16 tile (B operand of a second contraction):
// per group of 8 columns 16 slots [hi(8) | lo(8)], 64 slots (32 columns) per 128-byte block.
__device__ __forceinline__ void st_stacked_t(unsigned char* tile, int ch, int col, float x) {
    const float hi = trunc19(x);
    const int kbytes = ((col >> 3) & 3) * 32 + (col & 7) * 2;
    unsigned char* blk = tile + (col >> 5) * (DC * 128);
    *reinterpret_cast<unsigned short*>(blk + sw_chunk(ch, kbytes >> 4) + (kbytes & 15)) = (unsigned short)(bf16x2(hi, 0.f) & 0xffffu);
    *reinterpret_cast<unsigned short*>(blk + sw_chunk(ch, (kbytes + 16) >> 4) + (kbytes & 15)) = (unsigned short)(bf16x2(x - hi, 0.f) & 0xffffu);
}

__global__ void __launch_bounds__(DM)
forward_dense_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                     float* __restrict__ out, float* __restrict__ lse, int N, float scale_log2, int blocks_per_row) {
    extern __shared__ unsigned char dense_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)dense_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sQh = base, *sQl = base + 16384, *sKh = base + 32768, *sKl = base + 40960, *sVh = base + 49152, *sVl = base + 57344;
    __shared__ uint64_t mbar;
    __shared__ uint32_t tmem_base;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int lb = blockIdx.x % blocks_per_row;
    const int rest = blockIdx.x / blocks_per_row;
    const int n = rest % N;
    const int h = p.dense_rows[rest / N];
    const int w = lb * DM + tid;
    const bool row_ok = w < p.nlon_out;
    const size_t opt = (size_t)(n * p.nlat_out + h) * p.nlon_out + min(w, p.nlon_out - 1);

    {   // this thread's q row, in the log2 domain, split and stored as tile row tid
        const float4* src = reinterpret_cast<const float4*>(q + opt * DC);
#pragma unroll
        for (int c4 = 0; c4 < DC / 4; ++c4) {
            float4 x = __ldg(src + c4);
            x.x *= scale_log2; x.y *= scale_log2; x.z *= scale_log2; x.w *= scale_log2;
            float4 hi;
            hi.x = __uint_as_float(__float_as_uint(x.x) & 0xffffe000u); hi.y = __uint_as_float(__float_as_uint(x.y) & 0xffffe000u);
            hi.z = __uint_as_float(__float_as_uint(x.z) & 0xffffe000u); hi.w = __uint_as_float(__float_as_uint(x.w) & 0xffffe000u);
            *reinterpret_cast<float4*>(sQh + sw_chunk(tid, c4)) = hi;
            *reinterpret_cast<float4*>(sQl + sw_chunk(tid, c4)) = make_float4(x.x - hi.x, x.y - hi.y, x.z - hi.z, x.w - hi.w);
        }
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base, lanebits = (uint32_t)(warp * 32) << 16;
    const uint32_t tS = tm, tPh = tm + 64, tPl = tm + 128, tO = tm + 192;
    const uint32_t idS = umma_idesc(DBN), idO = umma_idesc(DC), bar = smem_u32(&mbar);
    uint32_t phase = 0;
    bool ok = true;
    float m = -INFINITY, l = 0.f, o[DC];
#pragma unroll
    for (int i = 0; i < DC; ++i) o[i] = 0.f;

    const int col = tid >> 1, half = tid & 1;      // this thread's share of a 64-column block: one column, 16 channels
    const int nblk = (p.nlon_in + DBN - 1) / DBN;
    const int e_begin = p.dense_ptr[h], e_end = p.dense_ptr[h + 1];
    const int total = (e_end - e_begin) * nblk;    // blocks of this tile, over all its whole input rings
    // raw k / v rows of the next block travel in registers while the current block's MMAs and softmax run
    // k: thread = (column tid/2, 16 channels); v: thread = (channel lane, 16 columns of group warp), so that the
    // transposed v rows are written with vector stores and read from global memory as whole 128-byte rows per warp
    float4 kraw[4];
    float vraw[16];
    const int lane = tid & 31;
    auto fetch = [&](int it) {
        const int hp = p.dense_lat[e_begin + it / nblk];
        const size_t ring0 = (size_t)(n * p.nlat_in + hp) * p.nlon_in;
        const int c0n = (it % nblk) * DBN;
        const size_t pt = (ring0 + min(c0n + col, p.nlon_in - 1)) * DC + half * 16;
#pragma unroll
        for (int j = 0; j < 4; ++j) kraw[j] = __ldg(reinterpret_cast<const float4*>(k + pt) + j);
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) vraw[jj] = __ldg(v + (ring0 + min(c0n + warp * 16 + jj, p.nlon_in - 1)) * DC + lane);
    };
    if (total > 0) fetch(0);
    for (int it = 0; it < total && ok; ++it) {
        const float bias = p.log2_omega[p.dense_lat[e_begin + it / nblk]];
        {
            const int c0 = (it % nblk) * DBN;
            {   // split this block's k rows, and v rows transposed (row = channel, K index = column)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float4 x = kraw[j];
                    float4 hi;
                    hi.x = __uint_as_float(__float_as_uint(x.x) & 0xffffe000u); hi.y = __uint_as_float(__float_as_uint(x.y) & 0xffffe000u);
                    hi.z = __uint_as_float(__float_as_uint(x.z) & 0xffffe000u); hi.w = __uint_as_float(__float_as_uint(x.w) & 0xffffe000u);
                    *reinterpret_cast<float4*>(sKh + sw_chunk(col, half * 4 + j)) = hi;
                    *reinterpret_cast<float4*>(sKl + sw_chunk(col, half * 4 + j)) = make_float4(x.x - hi.x, x.y - hi.y, x.z - hi.z, x.w - hi.w);
                }
                // columns warp*16 .. +15 of channel `lane`: K block warp/2, 16-byte chunks (warp%2)*4 .. +3 of row `lane`
#pragma unroll
                for (int g4 = 0; g4 < 4; ++g4) {
                    float hi[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) hi[i] = trunc19(vraw[4 * g4 + i]);
                    const int off = (warp >> 1) * (DC * 128) + sw_chunk(lane, (warp & 1) * 4 + g4);
                    *reinterpret_cast<float4*>(sVh + off) = make_float4(hi[0], hi[1], hi[2], hi[3]);
                }
                // stacked BF16 tile (row = channel): per group of 8 columns a 16-byte chunk of hi, then one of lo
#pragma unroll
                for (int g8 = 0; g8 < 2; ++g8) {
                    float hi[8], lo[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) { hi[i] = trunc19(vraw[8 * g8 + i]); lo[i] = vraw[8 * g8 + i] - hi[i]; }
                    const int chunk = ((warp & 1) * 2 + g8) * 2;
                    *reinterpret_cast<uint4*>(sVl + (warp >> 1) * (DC * 128) + sw_chunk(lane, chunk)) = bf16x8(hi);
                    *reinterpret_cast<uint4*>(sVl + (warp >> 1) * (DC * 128) + sw_chunk(lane, chunk + 1)) = bf16x8(lo);
                }
            }
            if (it + 1 < total) fetch(it + 1);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            if (tid == 0) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t qh = umma_desc(smem_u32(sQh)), ql = umma_desc(smem_u32(sQl)), kh = umma_desc(smem_u32(sKh)), kl = umma_desc(smem_u32(sKl));
#pragma unroll
                for (int ks2 = 0; ks2 < DC / 8; ++ks2) umma_ss(tS, ql + 2 * ks2, kh + 2 * ks2, idS, ks2 > 0);
#pragma unroll
                for (int ks2 = 0; ks2 < DC / 8; ++ks2) umma_ss(tS, qh + 2 * ks2, kl + 2 * ks2, idS, 1);
#pragma unroll
                for (int ks2 = 0; ks2 < DC / 8; ++ks2) umma_ss(tS, qh + 2 * ks2, kh + 2 * ks2, idS, 1);
                umma_commit(bar);
            }
            ok = wait_bar(bar, phase);
            phase ^= 1;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float corr = 1.f;
            if (ok) {
                uint32_t s0[32], s1[32], lo[32];
                tmem_ld32(s0, tS + lanebits);
                tmem_ld32(s1, tS + lanebits + 32);
                const int nvalid = p.nlon_in - c0;   // columns of this block that exist (>= 64 except in the last block)
                float mx = m;
                if (nvalid >= DBN) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float a = __uint_as_float(s0[j]) + bias, b = __uint_as_float(s1[j]) + bias;
                        s0[j] = __float_as_uint(a); s1[j] = __float_as_uint(b);
                        mx = fmaxf(mx, fmaxf(a, b));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float a = j < nvalid ? __uint_as_float(s0[j]) + bias : -INFINITY;
                        const float b = j + 32 < nvalid ? __uint_as_float(s1[j]) + bias : -INFINITY;
                        s0[j] = __float_as_uint(a); s1[j] = __float_as_uint(b);
                        mx = fmaxf(mx, fmaxf(a, b));
                    }
                }
                corr = ex2d(m - mx);
                m = mx;
                float ps = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float pj = ex2d(__uint_as_float(s0[j]) - m);
                    ps += pj;
                    s0[j] = __float_as_uint(pj);
                }
                pack_a16(s0, lo);
                tmem_st32(tPh + lanebits, s0);
                tmem_st32(tPl + lanebits, lo);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float pj = ex2d(__uint_as_float(s1[j]) - m);
                    ps += pj;
                    s1[j] = __float_as_uint(pj);
                }
                pack_a16(s1, lo);
                tmem_st32(tPh + lanebits + 32, s1);
                tmem_st32(tPl + lanebits + 32, lo);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                l = l * corr + ps;
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            if (tid == 0 && ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t vh0 = umma_desc(smem_u32(sVh)), vl0 = umma_desc(smem_u32(sVl));
                // corrections p_lo v_hi + p_hi v_lo: one BF16 UMMA per 8 columns; main term p_hi v_hi: one TF32 UMMA per 8 columns
#pragma unroll
                for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts16(tO, tPl + ks2 * 8, vl0 + (uint64_t)((ks2 >> 2) * (DC * 128 >> 4) + (ks2 & 3) * 2), umma_idesc16(DC), ks2 > 0);
#pragma unroll
                for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts(tO, tPh + ks2 * 8, vh0 + (uint64_t)((ks2 >> 2) * (DC * 128 >> 4) + (ks2 & 3) * 2), idO, 1);
                umma_commit(bar);
            }
            if (ok) {
                ok = wait_bar(bar, phase);
                phase ^= 1;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (ok) {
                uint32_t ob[32];
                tmem_ld32(ob, tO + lanebits);
#pragma unroll
                for (int j = 0; j < DC; ++j) o[j] = fmaf(o[j], corr, __uint_as_float(ob[j]));
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();   // the tiles and the TMEM blocks are free for the next block
        }
    }
    if (!ok && tid == 0) atomicExch(p.dev_status, 1);
    if (ok && row_ok) {
        const float inv = 1.f / l;
        float4* dst = reinterpret_cast<float4*>(out + opt * DC);
#pragma unroll
        for (int c4 = 0; c4 < DC / 4; ++c4) dst[c4] = make_float4(o[4 * c4] * inv, o[4 * c4 + 1] * inv, o[4 * c4 + 2] * inv, o[4 * c4 + 3] * inv);
        lse[opt] = (m + log2f(l)) * LN2_D;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(TMEM_COLS));
}


// ---------------------------------------------------------------------------------------------------------
// Dense part of the dq stage (App. B.4): for the whole input rings of an output ring,
//   p = exp2(s + log2 omega - lse),  ds = p (t - D),  dq += scale * dS K,   s = q.k (log2 domain),  t = dout.v.
// Same tiling as the forward kernel.  S and T go to TMEM as three TF32 UMMAs per k-step each; every thread turns
// its row of (S, T) into dS, split in hi and lo, in place; the k tile is then written transposed into the space
// of the v tile (dead once T is complete) and dq_block = dS K runs with A from TMEM.
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DM)
backward_dq_dense_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                         const float* __restrict__ dout, const float* __restrict__ out, const float* __restrict__ lse,
                         float* __restrict__ dq, int N, float scale, int blocks_per_row) {
    extern __shared__ unsigned char dense_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)dense_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sQh = base, *sQl = base + 16384, *sYh = base + 32768, *sYl = base + 49152;
    unsigned char *sKh = base + 65536, *sKl = base + 73728, *sVh = base + 81920, *sVl = base + 90112;   // v tiles, later k transposed
    __shared__ uint64_t mbar;
    __shared__ uint32_t tmem_base;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int lb = blockIdx.x % blocks_per_row;
    const int rest = blockIdx.x / blocks_per_row;
    const int n = rest % N;
    const int h = p.dense_rows[rest / N];
    const int w = lb * DM + tid;
    const bool row_ok = w < p.nlon_out;
    const size_t opt = (size_t)(n * p.nlat_out + h) * p.nlon_out + min(w, p.nlon_out - 1);
    const float scale_log2 = scale * LOG2E_D;

    float D = 0.f;
    {   // this thread's q row (log2 domain) and dout row as tile row tid (fp32 hi tile + stacked BF16 tile); D = dout . out
        const float4* qs = reinterpret_cast<const float4*>(q + opt * DC);
        const float4* ys = reinterpret_cast<const float4*>(dout + opt * DC);
        const float4* os = reinterpret_cast<const float4*>(out + opt * DC);
#pragma unroll
        for (int grp = 0; grp < DC / 8; ++grp) {
            float x[8], y[8];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float4 a = __ldg(qs + 2 * grp + hh), b = __ldg(ys + 2 * grp + hh), o4 = __ldg(os + 2 * grp + hh);
                x[4 * hh] = a.x * scale_log2; x[4 * hh + 1] = a.y * scale_log2; x[4 * hh + 2] = a.z * scale_log2; x[4 * hh + 3] = a.w * scale_log2;
                y[4 * hh] = b.x; y[4 * hh + 1] = b.y; y[4 * hh + 2] = b.z; y[4 * hh + 3] = b.w;
                D = fmaf(b.x, o4.x, fmaf(b.y, o4.y, fmaf(b.z, o4.z, fmaf(b.w, o4.w, D))));
                *reinterpret_cast<float4*>(sQh + sw_chunk(tid, 2 * grp + hh)) = make_float4(trunc19(x[4 * hh]), trunc19(x[4 * hh + 1]), trunc19(x[4 * hh + 2]), trunc19(x[4 * hh + 3]));
                *reinterpret_cast<float4*>(sYh + sw_chunk(tid, 2 * grp + hh)) = make_float4(trunc19(b.x), trunc19(b.y), trunc19(b.z), trunc19(b.w));
            }
            st_stacked8(sQl, tid, grp, x, true);
            st_stacked8(sYl, tid, grp, y, true);
        }
    }
    const float nl = -__ldg(lse + opt) * LOG2E_D;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base, lanebits = (uint32_t)(warp * 32) << 16;
    const uint32_t tS = tm, tT = tm + 64, tG = tm + 128;
    const uint32_t idS = umma_idesc(DBN), idO = umma_idesc(DC), bar = smem_u32(&mbar);
    uint32_t phase = 0;
    bool ok = true;
    float acc[DC];
#pragma unroll
    for (int i = 0; i < DC; ++i) acc[i] = 0.f;

    const int col = tid >> 1, half = tid & 1;      // this thread's share of a 64-column block: one column, 16 channels
    const int nblk = (p.nlon_in + DBN - 1) / DBN;
    const int e_begin = p.dense_ptr[h], e_end = p.dense_ptr[h + 1];
    const int total = (e_end - e_begin) * nblk;
    float4 kcur[4], vcur[4], knext[4], vnext[4];
    auto fetch = [&](int it, float4 (&kk)[4], float4 (&vv)[4]) {
        const int hp = p.dense_lat[e_begin + it / nblk];
        const size_t pt = ((size_t)(n * p.nlat_in + hp) * p.nlon_in + min((it % nblk) * DBN + col, p.nlon_in - 1)) * DC + half * 16;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            kk[j] = __ldg(reinterpret_cast<const float4*>(k + pt) + j);
            vv[j] = __ldg(reinterpret_cast<const float4*>(v + pt) + j);
        }
    };
    auto hi4 = [](const float4& x) {
        return make_float4(__uint_as_float(__float_as_uint(x.x) & 0xffffe000u), __uint_as_float(__float_as_uint(x.y) & 0xffffe000u),
                           __uint_as_float(__float_as_uint(x.z) & 0xffffe000u), __uint_as_float(__float_as_uint(x.w) & 0xffffe000u));
    };
    if (total > 0) fetch(0, kcur, vcur);
    for (int it = 0; it < total && ok; ++it) {
        const float bias = p.log2_omega[p.dense_lat[e_begin + it / nblk]] + nl;
        const int c0 = (it % nblk) * DBN;
#pragma unroll
        for (int g2 = 0; g2 < 2; ++g2) {   // k and v rows of this block (channels as K dimension): fp32 hi tile + stacked BF16 tile
            float kx[8], vx[8];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float4 a = kcur[2 * g2 + hh], b = vcur[2 * g2 + hh];
                kx[4 * hh] = a.x; kx[4 * hh + 1] = a.y; kx[4 * hh + 2] = a.z; kx[4 * hh + 3] = a.w;
                vx[4 * hh] = b.x; vx[4 * hh + 1] = b.y; vx[4 * hh + 2] = b.z; vx[4 * hh + 3] = b.w;
                *reinterpret_cast<float4*>(sKh + sw_chunk(col, half * 4 + 2 * g2 + hh)) = hi4(a);
                *reinterpret_cast<float4*>(sVh + sw_chunk(col, half * 4 + 2 * g2 + hh)) = hi4(b);
            }
            st_stacked8(sKl, col, half * 2 + g2, kx, false);
            st_stacked8(sVl, col, half * 2 + g2, vx, false);
        }
        if (it + 1 < total) fetch(it + 1, knext, vnext);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t qh = umma_desc(smem_u32(sQh)), ql = umma_desc(smem_u32(sQl)), yh = umma_desc(smem_u32(sYh)), yl = umma_desc(smem_u32(sYl));
            const uint64_t kh = umma_desc(smem_u32(sKh)), kl = umma_desc(smem_u32(sKl)), vh = umma_desc(smem_u32(sVh)), vl = umma_desc(smem_u32(sVl));
            // per 8 channels: one BF16 UMMA for both correction terms, one TF32 UMMA for the main term
#pragma unroll
            for (int ks2 = 0; ks2 < DC / 8; ++ks2) { umma_ss16(tS, ql + 2 * ks2, kl + 2 * ks2, umma_idesc16(DBN), ks2 > 0); umma_ss16(tT, yl + 2 * ks2, vl + 2 * ks2, umma_idesc16(DBN), ks2 > 0); }
#pragma unroll
            for (int ks2 = 0; ks2 < DC / 8; ++ks2) { umma_ss(tS, qh + 2 * ks2, kh + 2 * ks2, idS, 1); umma_ss(tT, yh + 2 * ks2, vh + 2 * ks2, idS, 1); }
            umma_commit(bar);
        }
        ok = wait_bar(bar, phase);
        phase ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            const int nvalid = p.nlon_in - c0;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {   // dS = p (t - D), split, in place over this row of S (hi) and T (lo)
                uint32_t sv[32], tv[32];
                tmem_ld32(sv, tS + lanebits + hf * 32);
                tmem_ld32(tv, tT + lanebits + hf * 32);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float pj = hf * 32 + j < nvalid ? ex2d(__uint_as_float(sv[j]) + bias) : 0.f;
                    const float ds = pj * (__uint_as_float(tv[j]) - D);
                    sv[j] = __float_as_uint(ds);
                }
                pack_a16(sv, tv);
                tmem_st32(tS + lanebits + hf * 32, sv);
                tmem_st32(tT + lanebits + hf * 32, tv);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            // k transposed (row = channel, K index = column) into the v tiles, which the completed T MMAs no longer read
            const int kb = col >> 5, kc = col & 31;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float xv[4] = {kcur[j].x, kcur[j].y, kcur[j].z, kcur[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int ch = half * 16 + 4 * j + i;
                    *reinterpret_cast<float*>(sVh + kb * (DC * 128) + sw_chunk(ch, kc >> 2) + (kc & 3) * 4) = trunc19(xv[i]);
                    st_stacked_t(sVl, ch, col, xv[i]);
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0 && ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t th0 = umma_desc(smem_u32(sVh)), tl0 = umma_desc(smem_u32(sVl));
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts16(tG, tT + ks2 * 8, tl0 + (uint64_t)((ks2 >> 2) * (DC * 128 >> 4) + (ks2 & 3) * 2), umma_idesc16(DC), ks2 > 0);
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts(tG, tS + ks2 * 8, th0 + (uint64_t)((ks2 >> 2) * (DC * 128 >> 4) + (ks2 & 3) * 2), idO, 1);
            umma_commit(bar);
        }
        if (ok) {
            ok = wait_bar(bar, phase);
            phase ^= 1;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            uint32_t gb[32];
            tmem_ld32(gb, tG + lanebits);
#pragma unroll
            for (int j = 0; j < DC; ++j) acc[j] += __uint_as_float(gb[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) { kcur[j] = knext[j]; vcur[j] = vnext[j]; }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }
    if (!ok && tid == 0) atomicExch(p.dev_status, 1);
    if (ok && row_ok) {
        float4* dst = reinterpret_cast<float4*>(dq + opt * DC);
#pragma unroll
        for (int c4 = 0; c4 < DC / 4; ++c4) dst[c4] = make_float4(acc[4 * c4] * scale, acc[4 * c4 + 1] * scale, acc[4 * c4 + 2] * scale, acc[4 * c4 + 3] * scale);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(TMEM_COLS));
}

// ---------------------------------------------------------------------------------------------------------
// Dense part of the dk/dv stage (App. B.4), transposed roles: one CTA owns 128 consecutive input columns of an input
// ring (tile row = input point j) and walks, in blocks of 64, the output points i of the output rings that attend to
// this input ring as a whole:
//   S^T = K Q^T, T^T = V dY^T (TF32 UMMAs into TMEM);  p = exp2(s + log2 omega_j - lse_i),  ds = p (t - D_i);
//   dV += P^T dY,  dK += scale * dS^T Q   (A from TMEM, the q / dout tiles rewritten transposed once S^T, T^T are done).
// TMEM budget (256 columns): P_hi over S, P_lo over T, raw dS in a third block; after the dV MMAs dS_lo replaces P_lo
// and the raw dS block itself serves as dS_hi (the MMA reads only its top 19 bits).
// ---------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(DM)
backward_dkdv_dense_kernel(DevPlan p, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                           const float* __restrict__ dout, const float* __restrict__ lse, const float* __restrict__ Dws,
                           float* __restrict__ dk, float* __restrict__ dv, int N, float scale, int blocks_per_row) {
    extern __shared__ unsigned char dense_raw[];
    unsigned char* base = (unsigned char*)(((uintptr_t)dense_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sKh = base, *sKl = base + 16384, *sVh = base + 32768, *sVl = base + 49152;                 // persistent A tiles
    unsigned char *sQh = base + 65536, *sQl = base + 73728, *sYh = base + 81920, *sYl = base + 90112;         // per block, later transposed
    __shared__ uint64_t mbar;
    __shared__ uint32_t tmem_base;
    __shared__ float s_nl[DBN], s_D[DBN];     // per partner column: -lse (log2) and D
    const int tid = threadIdx.x, warp = tid >> 5;
    const int lb = blockIdx.x % blocks_per_row;
    const int rest = blockIdx.x / blocks_per_row;
    const int n = rest % N;
    const int hp = p.t_dense_rows[rest / N];
    const int c = lb * DM + tid;
    const bool row_ok = c < p.nlon_in;
    const size_t ipt = (size_t)(n * p.nlat_in + hp) * p.nlon_in + min(c, p.nlon_in - 1);
    const float scale_log2 = scale * LOG2E_D;
    const float bias = p.log2_omega[hp];

    {   // this thread's k row (log2 domain) and v row as tile row tid: fp32 hi tile + stacked BF16 tile
        const float4* ks = reinterpret_cast<const float4*>(k + ipt * DC);
        const float4* vs = reinterpret_cast<const float4*>(v + ipt * DC);
#pragma unroll
        for (int grp = 0; grp < DC / 8; ++grp) {
            float x[8], y[8];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float4 a = __ldg(ks + 2 * grp + hh), b = __ldg(vs + 2 * grp + hh);
                x[4 * hh] = a.x * scale_log2; x[4 * hh + 1] = a.y * scale_log2; x[4 * hh + 2] = a.z * scale_log2; x[4 * hh + 3] = a.w * scale_log2;
                y[4 * hh] = b.x; y[4 * hh + 1] = b.y; y[4 * hh + 2] = b.z; y[4 * hh + 3] = b.w;
                *reinterpret_cast<float4*>(sKh + sw_chunk(tid, 2 * grp + hh)) = make_float4(trunc19(x[4 * hh]), trunc19(x[4 * hh + 1]), trunc19(x[4 * hh + 2]), trunc19(x[4 * hh + 3]));
                *reinterpret_cast<float4*>(sVh + sw_chunk(tid, 2 * grp + hh)) = make_float4(trunc19(b.x), trunc19(b.y), trunc19(b.z), trunc19(b.w));
            }
            st_stacked8(sKl, tid, grp, x, true);
            st_stacked8(sVl, tid, grp, y, true);
        }
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tm = tmem_base, lanebits = (uint32_t)(warp * 32) << 16;
    const uint32_t tS = tm, tT = tm + 64, tX = tm + 128, tGv = tm + 192, tGk = tm + 224;
    const uint32_t idS = umma_idesc(DBN), idO = umma_idesc(DC), bar = smem_u32(&mbar);
    uint32_t phase = 0;
    bool ok = true;
    float gk[DC], gv[DC];
#pragma unroll
    for (int i = 0; i < DC; ++i) { gk[i] = 0.f; gv[i] = 0.f; }
    const int col = tid >> 1, half = tid & 1;      // this thread's share of a 64-partner block: one output point, 16 channels
    const int nblk = (p.nlon_out + DBN - 1) / DBN;
    const int e_begin = p.t_dense_ptr[hp], e_end = p.t_dense_ptr[hp + 1];
    const int total = (e_end - e_begin) * nblk;
    float4 qcur[4], ycur[4], qnext[4], ynext[4];
    auto fetch = [&](int it, float4 (&qq)[4], float4 (&yy)[4]) {
        const int h = p.t_dense_lat[e_begin + it / nblk];
        const size_t pt = ((size_t)(n * p.nlat_out + h) * p.nlon_out + min((it % nblk) * DBN + col, p.nlon_out - 1)) * DC + half * 16;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            qq[j] = __ldg(reinterpret_cast<const float4*>(q + pt) + j);
            yy[j] = __ldg(reinterpret_cast<const float4*>(dout + pt) + j);
        }
    };
    auto hi4 = [](const float4& x) {
        return make_float4(__uint_as_float(__float_as_uint(x.x) & 0xffffe000u), __uint_as_float(__float_as_uint(x.y) & 0xffffe000u),
                           __uint_as_float(__float_as_uint(x.z) & 0xffffe000u), __uint_as_float(__float_as_uint(x.w) & 0xffffe000u));
    };
    // element (row = channel, K index = partner column) of a transposed tile: fp32 hi tile and stacked BF16 tile
    auto st_t = [&](unsigned char* th, unsigned char* tl, int ch, float x) {
        *reinterpret_cast<float*>(th + (col >> 5) * (DC * 128) + sw_chunk(ch, (col & 31) >> 2) + (col & 3) * 4) = trunc19(x);
        st_stacked_t(tl, ch, col, x);
    };
    if (total > 0) fetch(0, qcur, ycur);
    for (int it = 0; it < total && ok; ++it) {
        const int h = p.t_dense_lat[e_begin + it / nblk];
        const int w0 = (it % nblk) * DBN;
#pragma unroll
        for (int g2 = 0; g2 < 2; ++g2) {   // q and dout rows of the partner points (channels as K dimension)
            float qx[8], yx[8];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float4 a = qcur[2 * g2 + hh], b = ycur[2 * g2 + hh];
                qx[4 * hh] = a.x; qx[4 * hh + 1] = a.y; qx[4 * hh + 2] = a.z; qx[4 * hh + 3] = a.w;
                yx[4 * hh] = b.x; yx[4 * hh + 1] = b.y; yx[4 * hh + 2] = b.z; yx[4 * hh + 3] = b.w;
                *reinterpret_cast<float4*>(sQh + sw_chunk(col, half * 4 + 2 * g2 + hh)) = hi4(a);
                *reinterpret_cast<float4*>(sYh + sw_chunk(col, half * 4 + 2 * g2 + hh)) = hi4(b);
            }
            st_stacked8(sQl, col, half * 2 + g2, qx, false);
            st_stacked8(sYl, col, half * 2 + g2, yx, false);
        }
        if (tid < DBN) {
            const size_t o = (size_t)(n * p.nlat_out + h) * p.nlon_out + min(w0 + tid, p.nlon_out - 1);
            s_nl[tid] = fmaf(-__ldg(lse + o), LOG2E_D, bias);
            s_D[tid] = __ldg(Dws + o);
        }
        if (it + 1 < total) fetch(it + 1, qnext, ynext);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t kh = umma_desc(smem_u32(sKh)), kl = umma_desc(smem_u32(sKl)), vh = umma_desc(smem_u32(sVh)), vl = umma_desc(smem_u32(sVl));
            const uint64_t qh = umma_desc(smem_u32(sQh)), ql = umma_desc(smem_u32(sQl)), yh = umma_desc(smem_u32(sYh)), yl = umma_desc(smem_u32(sYl));
#pragma unroll
            for (int ks2 = 0; ks2 < DC / 8; ++ks2) { umma_ss16(tS, kl + 2 * ks2, ql + 2 * ks2, umma_idesc16(DBN), ks2 > 0); umma_ss16(tT, vl + 2 * ks2, yl + 2 * ks2, umma_idesc16(DBN), ks2 > 0); }
#pragma unroll
            for (int ks2 = 0; ks2 < DC / 8; ++ks2) { umma_ss(tS, kh + 2 * ks2, qh + 2 * ks2, idS, 1); umma_ss(tT, vh + 2 * ks2, yh + 2 * ks2, idS, 1); }
            umma_commit(bar);
        }
        ok = wait_bar(bar, phase);
        phase ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            const int nvalid = p.nlon_out - w0;
#pragma unroll
            for (int qt = 0; qt < 4; ++qt) {   // P (fp32 over S, stacked packs over T) and raw dS for this row; 16 columns at a
                uint32_t sv[16], tv[16], xv[16];   // time keeps the kernel free of register spills (worth 19 % here)
                tmem_ld16(sv, tS + lanebits + qt * 16);
                tmem_ld16(tv, tT + lanebits + qt * 16);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float pj = qt * 16 + j < nvalid ? ex2d(__uint_as_float(sv[j]) + s_nl[qt * 16 + j]) : 0.f;
                    xv[j] = __float_as_uint(pj * (__uint_as_float(tv[j]) - s_D[qt * 16 + j]));
                    sv[j] = __float_as_uint(pj);
                }
                pack_a16_16(sv, tv);
                tmem_st16(tS + lanebits + qt * 16, sv);
                tmem_st16(tT + lanebits + qt * 16, tv);
                tmem_st16(tX + lanebits + qt * 16, xv);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            // the q / dout tiles are dead: rewrite them transposed (row = channel, K index = partner)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float qv[4] = {qcur[j].x, qcur[j].y, qcur[j].z, qcur[j].w}, yv[4] = {ycur[j].x, ycur[j].y, ycur[j].z, ycur[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    st_t(sQh, sQl, half * 16 + 4 * j + i, qv[i]);
                    st_t(sYh, sYl, half * 16 + 4 * j + i, yv[i]);
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        const auto tdesc = [](uint64_t d0, int ks2) { return d0 + (uint64_t)((ks2 >> 2) * (DC * 128 >> 4) + (ks2 & 3) * 2); };
        if (tid == 0 && ok) {   // dV_block = P^T dY
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t yh = umma_desc(smem_u32(sYh)), yl = umma_desc(smem_u32(sYl));
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts16(tGv, tT + ks2 * 8, tdesc(yl, ks2), umma_idesc16(DC), ks2 > 0);
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts(tGv, tS + ks2 * 8, tdesc(yh, ks2), idO, 1);
            umma_commit(bar);
        }
        if (ok) { ok = wait_bar(bar, phase); phase ^= 1; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {   // the stacked packs of dS replace those of P; the raw dS block is the main-term operand
#pragma unroll
            for (int qt = 0; qt < 4; ++qt) {
                uint32_t xv[16], pk[16];
                tmem_ld16(xv, tX + lanebits + qt * 16);
                pack_a16_16(xv, pk);
                tmem_st16(tT + lanebits + qt * 16, pk);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0 && ok) {   // dK_block = dS^T Q
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t qh = umma_desc(smem_u32(sQh)), ql = umma_desc(smem_u32(sQl));
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts16(tGk, tT + ks2 * 8, tdesc(ql, ks2), umma_idesc16(DC), ks2 > 0);
#pragma unroll
            for (int ks2 = 0; ks2 < DBN / 8; ++ks2) umma_ts(tGk, tX + ks2 * 8, tdesc(qh, ks2), idO, 1);
            umma_commit(bar);
        }
        if (ok) { ok = wait_bar(bar, phase); phase ^= 1; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok) {
            uint32_t gb[32];
            tmem_ld32(gb, tGv + lanebits);
#pragma unroll
            for (int j = 0; j < DC; ++j) gv[j] += __uint_as_float(gb[j]);
            tmem_ld32(gb, tGk + lanebits);
#pragma unroll
            for (int j = 0; j < DC; ++j) gk[j] += __uint_as_float(gb[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) { qcur[j] = qnext[j]; ycur[j] = ynext[j]; }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
    }
    if (!ok && tid == 0) atomicExch(p.dev_status, 1);
    if (ok && row_ok) {
        float4* dkp = reinterpret_cast<float4*>(dk + ipt * DC);
        float4* dvp = reinterpret_cast<float4*>(dv + ipt * DC);
#pragma unroll
        for (int c4 = 0; c4 < DC / 4; ++c4) {
            dkp[c4] = make_float4(gk[4 * c4] * scale, gk[4 * c4 + 1] * scale, gk[4 * c4 + 2] * scale, gk[4 * c4 + 3] * scale);
            dvp[c4] = make_float4(gv[4 * c4], gv[4 * c4 + 1], gv[4 * c4 + 2], gv[4 * c4 + 3]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(TMEM_COLS));
}
}  // namespace

cudaError_t dense_prepare_device() {
    cudaError_t e = cudaFuncSetAttribute(forward_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DENSE_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(backward_dq_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DENSE_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(backward_dkdv_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DENSE_SMEM);
    return e;
}

bool dense_path_supported(const DevPlan& p, int C) {
    return C == DC && p.dense_ptr != nullptr && p.n_dense_rows > 0 && p.fwdb_stream != nullptr && mma_path_supported(p, C);
}

cudaError_t launch_forward_dense(const DevPlan& p, const float* q, const float* k, const float* v, float* out, float* lse,
                                 int N, int C, cudaStream_t stream) {
    if (C != DC || lse == nullptr) return cudaErrorInvalidValue;
    const int blocks_per_row = (p.nlon_out + DM - 1) / DM;
    const long long blocks = (long long)blocks_per_row * p.n_dense_rows * N;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    forward_dense_kernel<<<(unsigned)blocks, DM, DENSE_SMEM, stream>>>(p, q, k, v, out, lse, N, LOG2E_D / sqrtf((float)C), blocks_per_row);
    return cudaGetLastError();
}

cudaError_t launch_backward_dq_dense(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                     const float* out, const float* lse, float* dq, int N, int C, cudaStream_t stream) {
    if (C != DC || out == nullptr || lse == nullptr || out == dq) return cudaErrorInvalidValue;
    const int blocks_per_row = (p.nlon_out + DM - 1) / DM;
    const long long blocks = (long long)blocks_per_row * p.n_dense_rows * N;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    backward_dq_dense_kernel<<<(unsigned)blocks, DM, DENSE_SMEM, stream>>>(p, q, k, v, dout, out, lse, dq, N, 1.0f / sqrtf((float)C), blocks_per_row);
    return cudaGetLastError();
}

cudaError_t launch_backward_dkdv_dense(const DevPlan& p, const float* q, const float* k, const float* v, const float* dout,
                                       const float* lse, const float* Dws, float* dk, float* dv, int N, int C, cudaStream_t stream) {
    if (C != DC) return cudaErrorInvalidValue;
    const int blocks_per_row = (p.nlon_in + DM - 1) / DM;
    const long long blocks = (long long)blocks_per_row * p.n_t_dense_rows * N;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    backward_dkdv_dense_kernel<<<(unsigned)blocks, DM, DENSE_SMEM, stream>>>(p, q, k, v, dout, lse, Dws, dk, dv, N, 1.0f / sqrtf((float)C), blocks_per_row);
    return cudaGetLastError();
}

}  // namespace sna
