// Dynamic Top-K block mask (Appendix A.1, Steps 1-2): per (batch, head) and query block, the k key
// blocks whose mean has the largest average similarity with the block's queries,
//     s[i][j] = < mean of query block i , mean of key block j > ,
// written as the CSR lists the attention kernel consumes (every row keeps kk = min(k, nKb) blocks,
// ascending; a tie goes to the lower block index).
//
//   block_mean_kernel   HBM-bound: Q and K are read once (4*N*d bytes per head).  One CTA per token
//                       block; a thread owns one 16-byte channel group of every G-th row, so a warp
//                       instruction reads 512 contiguous bytes; the row groups are added in a fixed
//                       order through shared memory (deterministic), fp32.
//   topk_score_kernel   s for a 32 x 128 tile of (query block, key block) pairs per CTA: register-tiled
//                       fp32 FMAs in channel order from channel-major shared memory; the scores go
//                       to the workspace as order-preserving 32-bit images.
//   topk_pick_kernel    per query block (a warp takes two): the kk-th largest score by bisection on
//                       the bits of its image, then an ordered compaction into the CSR row.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace salad {

constexpr int kMeanThreads = 256;

struct MeanJob {
    const uint4* x;      // bf16 [BH][N][d]
    float* mean;         // fp32 [BH][nB][d], or channel-major [BH][d][ld] when ld > 0
    int block, nB;       // tokens per block, blocks per head
    int ld;              // 0: block-major rows of d channels; > 0: channel-major rows of ld blocks
};

// grid (max nB, BH, 2): z selects the job (queries / keys)
__global__ void __launch_bounds__(kMeanThreads)
block_mean_kernel(MeanJob jq, MeanJob jk, int N, int d)
{
    const MeanJob job = (blockIdx.z == 0) ? jq : jk;
    const int blk = blockIdx.x, bh = blockIdx.y;
    if (blk >= job.nB) return;
    __shared__ float part[kMeanThreads / 8][8 * 16 + 1];      // [row group][channel] (d <= 128)
    const int chunks = d / 8;                                 // 16-byte groups per row: 8 or 16
    const int groups = kMeanThreads / chunks;                 // row groups: 32 or 16
    const int tid = threadIdx.x, c = tid % chunks, g = tid / chunks;
    const int n0 = blk * job.block, n1 = min(N, n0 + job.block);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const uint4* base = job.x + (size_t(bh) * N) * chunks + c;
#pragma unroll 4
    for (int n = n0 + g; n < n1; n += groups) {               // this thread's rows, in token order
        const uint4 v = __ldg(base + size_t(n) * chunks);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            acc[2 * e] += f.x; acc[2 * e + 1] += f.y;
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) part[g][c * 8 + e] = acc[e];
    __syncthreads();
    if (tid < d) {
        float s = 0.f;
        for (int gg = 0; gg < groups; ++gg) s += part[gg][tid];      // fixed order
        const float m = s / float(n1 - n0);
        if (job.ld > 0) job.mean[(size_t(bh) * d + tid) * job.ld + blk] = m;
        else            job.mean[(size_t(bh) * job.nB + blk) * d + tid] = m;
    }
}

constexpr int kScoreRows = 32;        // query blocks per CTA (eight warps, four each)
constexpr int kScoreTile = 128;       // key blocks per CTA (four per lane)

// fp32 -> uint32 such that a < b  <=>  image(a) < image(b)  (for non-NaN a, b; -0 is stored as +0)
__device__ __forceinline__ uint32_t ordered_bits(float s) {
    const uint32_t u = __float_as_uint(s + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// grid (ceil(nKb / 128), ceil(nQb / 32), BH), 256 threads, dynamic shared memory d * (32 + 128) * 4
// bytes: As [d][32] query-block means | Bs [d][128] key-block means, both channel-major.
//   qmean  [BH][nQb][d]      kmeanT [BH][d][ldk] (ldk a multiple of 128: whole tiles are readable)
//   score  [BH][nQb][nKb]    images of s[i][j] = sum_c qmean[i][c] * kmean[j][c], c ascending
__global__ void __launch_bounds__(256)
topk_score_kernel(const float* __restrict__ qmean, const float* __restrict__ kmeanT, int nQb, int nKb, int ldk,
                  int d, uint32_t* __restrict__ score)
{
    extern __shared__ __align__(16) float sc_smem[];
    float* As = sc_smem;
    float* Bs = As + d * kScoreRows;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j0 = blockIdx.x * kScoreTile, i0 = blockIdx.y * kScoreRows, bh = blockIdx.z;
    const int d4 = d / 4;
    grid_dependency_wait();
    grid_launch_dependents();
    {   // key-block means: rows of 128 contiguous floats per channel, 16-byte asynchronous copies
        const float* src = kmeanT + size_t(bh) * d * ldk + j0;
        for (int idx = tid; idx < d * (kScoreTile / 4); idx += 256) {
            const int c = idx / (kScoreTile / 4), f = idx % (kScoreTile / 4);
            cp_async_16(Bs + c * kScoreTile + f * 4, src + size_t(c) * ldk + f * 4);
        }
    }
    {   // query-block means, transposed on the way in
        const int r = tid % kScoreRows, ii = min(i0 + r, nQb - 1);
        const float4* src = reinterpret_cast<const float4*>(qmean + (size_t(bh) * nQb + ii) * d);
        for (int c4 = tid / kScoreRows; c4 < d4; c4 += 256 / kScoreRows) {
            const float4 v = __ldg(src + c4);
            As[(c4 * 4 + 0) * kScoreRows + r] = v.x; As[(c4 * 4 + 1) * kScoreRows + r] = v.y;
            As[(c4 * 4 + 2) * kScoreRows + r] = v.z; As[(c4 * 4 + 3) * kScoreRows + r] = v.w;
        }
    }
    cp_async_wait_all();
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[r][u] = 0.f;
#pragma unroll 4
    for (int c = 0; c < d; ++c) {                              // channel order
        const float4 q4 = *reinterpret_cast<const float4*>(As + c * kScoreRows + warp * 4);
        const float4 k4 = *reinterpret_cast<const float4*>(Bs + c * kScoreTile + lane * 4);
        const float qv[4] = {q4.x, q4.y, q4.z, q4.w}, kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[r][u] = fmaf(qv[r], kv[u], acc[r][u]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + warp * 4 + r;
        if (i >= nQb) break;
        uint32_t* out = score + (size_t(bh) * nQb + i) * nKb + j0 + lane * 4;
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (j0 + lane * 4 + u < nKb) out[u] = ordered_bits(acc[r][u]);
    }
}

// grid ceil(rows_total / 8), 128 threads: a warp selects for two consecutive rows (query blocks) at
// a time: the kk-th largest score by bisection on the 32 bits of its image (32 counting passes,
// whatever kk), everything above it, and of the scores equal to it the lowest block indices -- the
// same set as kk rounds of "largest remaining, ties to the lower index".
// KPL > 0: the lane's share of a row (block j = lane + 32 t, t < KPL) is held in registers during
// the bisection (needs nKb <= 32 KPL); KPL = 0: it is re-read (from L1/L2) in every pass.
template <int KPL>
__global__ void __launch_bounds__(128)
topk_pick_kernel(const uint32_t* __restrict__ score, int nKb, int kk, int32_t* __restrict__ row_ptr,
                 int32_t* __restrict__ col_idx, long long rows_total)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dependency_wait();
    grid_launch_dependents();
    {
        const long long ra = ((long long)blockIdx.x * 4 + warp) * 2;
        if (ra >= rows_total) return;
        const bool two = ra + 1 < rows_total;
        const uint32_t* ka = score + ra * nKb;
        const uint32_t* kb = ka + (two ? nKb : 0);
        uint32_t ma[KPL > 0 ? KPL : 1], mb[KPL > 0 ? KPL : 1];
        if (KPL > 0) {
#pragma unroll
            for (int t = 0; t < KPL; ++t) {
                const bool in = lane + 32 * t < nKb;
                ma[t] = in ? ka[lane + 32 * t] : 0u; mb[t] = in ? kb[lane + 32 * t] : 0u;
            }
        }
        // image of the kk-th largest score: the largest T with #{key >= T} >= kk.  (Absent
        // entries are 0 and every candidate is > 0, so they are never counted.)
        uint32_t Ta = 0, Tb = 0;
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t ca = Ta | (1u << bit), cb = Tb | (1u << bit);
            int na = 0, nb = 0;
            if (KPL > 0) {
#pragma unroll
                for (int t = 0; t < KPL; ++t) { na += (ma[t] >= ca) ? 1 : 0; nb += (mb[t] >= cb) ? 1 : 0; }
            } else {
                for (int j = lane; j < nKb; j += 32) { na += (ka[j] >= ca) ? 1 : 0; nb += (kb[j] >= cb) ? 1 : 0; }
            }
            na = __reduce_add_sync(0xffffffffu, na); nb = __reduce_add_sync(0xffffffffu, nb);
            if (na >= kk) Ta = ca;
            if (nb >= kk) Tb = cb;
        }
        for (int e = 0; e < (two ? 2 : 1); ++e) {
            const uint32_t* kr = e ? kb : ka;
            const uint32_t T = e ? Tb : Ta;
            int n_gt = 0;
            for (int j = lane; j < nKb; j += 32) n_gt += (kr[j] > T) ? 1 : 0;
            n_gt = __reduce_add_sync(0xffffffffu, n_gt);
            const int need_eq = kk - n_gt;                     // of the scores equal to T, the first need_eq
            // ordered compaction
            const long long row = ra + e;
            int32_t* out = col_idx + row * kk;
            int count = 0, eq_seen = 0;
            for (int j0 = 0; j0 < nKb; j0 += 32) {
                const int j = j0 + lane;
                const uint32_t v = (j < nKb) ? kr[j] : 0u;
                const bool eq = (j < nKb) && v == T;
                const unsigned m_eq = __ballot_sync(0xffffffffu, eq);
                const int my_eq = eq_seen + __popc(m_eq & ((1u << lane) - 1u));
                const bool take = (j < nKb) && (v > T || (eq && my_eq < need_eq));
                const unsigned m = __ballot_sync(0xffffffffu, take);
                if (take) out[count + __popc(m & ((1u << lane) - 1u))] = j;
                count += __popc(m); eq_seen += __popc(m_eq);
            }
            if (lane == 0) {
                row_ptr[row] = int32_t(row * kk);
                if (row == rows_total - 1) row_ptr[rows_total] = int32_t(rows_total * kk);
            }
        }
    }
}

}  // namespace salad
