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
//   topk_pick_row_kernel  per query block (a CTA each): the kk-th largest score by radix selection on
//                       the bytes of its image, then an ordered compaction into the CSR row.
//                       (topk_pick_kernel: the same by bisection, a warp per two rows, for rows of more
//                       than 1024 key blocks.)
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
#pragma unroll 8
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

constexpr int kScoreRows = 32;        // query blocks per CTA (four warps, eight each)
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

constexpr int kScoreChunk = 32;       // channels per shared-memory stage
constexpr int kScoreSmemBytes = 2 * kScoreChunk * (kScoreRows + kScoreTile) * 4;      // two stages: 40 KB

// grid (ceil(nKb / 128), ceil(nQb / 32), BH), 128 threads (an 8 x 4 tile of scores each), 40 KB of dynamic shared memory: two stages of
// 32 channels each, As [32][32] query-block means | Bs [32][128] key-block means, both channel-major; the
// next stage is fetched (asynchronous 16-byte copies) while the current one is multiplied, and five CTAs
// fit on an SM, so the whole grid is resident at once.
//   qmean  [BH][nQb][d]      kmeanT [BH][d][ldk] (ldk a multiple of 128: whole tiles are readable)
//   score  [BH][nQb][nKb]    images of s[i][j] = sum_c qmean[i][c] * kmean[j][c], c ascending
__global__ void __launch_bounds__(128)
topk_score_kernel(const float* __restrict__ qmean, const float* __restrict__ kmeanT, int nQb, int nKb, int ldk,
                  int d, uint32_t* __restrict__ score)
{
    extern __shared__ __align__(16) float sc_smem[];
    constexpr int STAGE = kScoreChunk * (kScoreRows + kScoreTile);       // floats per stage
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j0 = blockIdx.x * kScoreTile, i0 = blockIdx.y * kScoreRows, bh = blockIdx.z;
    grid_dependency_wait();
    grid_launch_dependents();
    const float* ksrc = kmeanT + size_t(bh) * d * ldk + j0;
    const int r_q = tid % kScoreRows, ii = min(i0 + r_q, nQb - 1);
    const float* qsrc = qmean + (size_t(bh) * nQb + ii) * d;
    auto fetch = [&](int chunk, int stage) {
        float* As = sc_smem + stage * STAGE;
        float* Bs = As + kScoreChunk * kScoreRows;
        const int c0 = chunk * kScoreChunk;
        // key-block means: rows of 128 contiguous floats per channel
        for (int idx = tid; idx < kScoreChunk * (kScoreTile / 4); idx += 128) {
            const int c = idx / (kScoreTile / 4), f = idx % (kScoreTile / 4);
            cp_async_16(Bs + c * kScoreTile + f * 4, ksrc + size_t(c0 + c) * ldk + f * 4);
        }
        // query-block means, transposed on the way in: this thread's row, one float4 of channels
        for (int c4 = tid / kScoreRows; c4 < kScoreChunk / 4; c4 += 128 / kScoreRows) {     // channels 4 c4 .. 4 c4 + 3 of the chunk
            const float4 v = __ldg(reinterpret_cast<const float4*>(qsrc + c0) + c4);
            As[(c4 * 4 + 0) * kScoreRows + r_q] = v.x; As[(c4 * 4 + 1) * kScoreRows + r_q] = v.y;
            As[(c4 * 4 + 2) * kScoreRows + r_q] = v.z; As[(c4 * 4 + 3) * kScoreRows + r_q] = v.w;
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int u = 0; u < 4; ++u) acc[r][u] = 0.f;
    const int chunks = d / kScoreChunk;
    fetch(0, 0);
    for (int ch = 0; ch < chunks; ++ch) {
        if (ch + 1 < chunks) {
            fetch(ch + 1, (ch + 1) & 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const float* As = sc_smem + (ch & 1) * STAGE;
        const float* Bs = As + kScoreChunk * kScoreRows;
#pragma unroll 8
        for (int c = 0; c < kScoreChunk; ++c) {                    // channel order
            const float4 qa = *reinterpret_cast<const float4*>(As + c * kScoreRows + warp * 8);
            const float4 qb = *reinterpret_cast<const float4*>(As + c * kScoreRows + warp * 8 + 4);
            const float4 k4 = *reinterpret_cast<const float4*>(Bs + c * kScoreTile + lane * 4);
            const float qv[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w}, kv[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int r = 0; r < 8; ++r)
#pragma unroll
                for (int u = 0; u < 4; ++u) acc[r][u] = fmaf(qv[r], kv[u], acc[r][u]);
        }
        __syncthreads();                                           // the stage is fetched into again two chunks on
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const int i = i0 + warp * 8 + r;
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
// The lane's share of a row is re-read (from L1/L2) in every pass: this is the kernel for rows too long for
// topk_pick_row_kernel below (more than 1024 key blocks).
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
        // image of the kk-th largest score: the largest T with #{key >= T} >= kk.  (Absent
        // entries are 0 and every candidate is > 0, so they are never counted.)
        uint32_t Ta = 0, Tb = 0;
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t ca = Ta | (1u << bit), cb = Tb | (1u << bit);
            int na = 0, nb = 0;
            for (int j = lane; j < nKb; j += 32) { na += (ka[j] >= ca) ? 1 : 0; nb += (kb[j] >= cb) ? 1 : 0; }
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

// One CTA (four warps) per row: with a warp per two rows only ten warps ran on an SM and the selection was a
// chain of dependent steps (measured 18-20 us for 3072 rows of 512 scores); a CTA per row puts sixteen rows on
// an SM at a time and shortens every step by a factor of four.
//   1. radix selection of the kk-th largest image from the top byte down: four passes, each a 256-bin
//      histogram (shared-memory atomics) of the byte among the keys that still share the bytes chosen so far,
//      then the bin in which the count from the top reaches what is still needed (every warp does that scan
//      for itself, so a pass needs one barrier; the histograms rotate through three buffers).  Absent
//      entries are 0 and every real image is > 0, so they are never counted.
//   2. ties: if more keys equal the threshold than the selection takes, warp 0 finds the index up to which
//      they belong to it (a tie goes to the lower block index).
//   3. ordered compaction: per 128-key chunk a ballot per warp, one table of counts, every thread places its keys.
// KPT keys per thread in registers (key j = tid + 128 i); needs nKb <= 128 KPT and nKb <= 128 * kPickMaxChunks.
constexpr int kPickMaxChunks = 8;

template <int KPT>
__global__ void __launch_bounds__(128)
topk_pick_row_kernel(const uint32_t* __restrict__ score, int nKb, int kk, int32_t* __restrict__ row_ptr,
                     int32_t* __restrict__ col_idx, long long rows_total)
{
    __shared__ int hist[3][256];
    __shared__ int wcnt[kPickMaxChunks][4];
    __shared__ int cut_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long row = blockIdx.x;
    hist[0][tid] = 0; hist[0][tid + 128] = 0;
    grid_dependency_wait();
    grid_launch_dependents();
    const uint32_t* kr = score + row * nKb;
    uint32_t key[KPT];
#pragma unroll
    for (int i = 0; i < KPT; ++i) key[i] = (tid + 128 * i < nKb) ? kr[tid + 128 * i] : 0u;
    __syncthreads();
    uint32_t T = 0;
    int need = kk, n_eq = 0;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
        int* h = hist[pass % 3];
        // for the next pass (that buffer was last read two passes ago: every warp is past the barrier since)
        hist[(pass + 1) % 3][tid] = 0; hist[(pass + 1) % 3][tid + 128] = 0;
#pragma unroll
        for (int i = 0; i < KPT; ++i)
            if (key[i] != 0u && (key[i] & mask) == T) atomicAdd(&h[(key[i] >> shift) & 255u], 1);
        __syncthreads();
        // lane l looks at bins [8 l, 8 l + 8); counts from the top: the lanes above first, then the lane's bins downwards
        int c[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { c[i] = h[8 * lane + i]; sum += c[i]; }
        int incl = sum;                                     // this lane's bins and all higher ones
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int v = __shfl_down_sync(0xffffffffu, incl, off);
            if (lane + off < 32) incl += v;
        }
        const int above = incl - sum;
        const bool hit = above < need && incl >= need;     // exactly one lane
        int bin = 0, above_bin = 0, in_bin = 0;
        if (hit) {
            int acc = above;
#pragma unroll
            for (int i = 7; i >= 0; --i) {
                if (acc < need && acc + c[i] >= need) { bin = 8 * lane + i; above_bin = acc; in_bin = c[i]; }
                acc += c[i];
            }
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, hit)) - 1;
        bin = __shfl_sync(0xffffffffu, bin, src);
        above_bin = __shfl_sync(0xffffffffu, above_bin, src);
        n_eq = __shfl_sync(0xffffffffu, in_bin, src);      // after the last pass: keys equal to the threshold
        T |= uint32_t(bin) << shift;
        need -= above_bin;
    }
    // `need` of the n_eq keys equal to T belong to the selection: those with the lowest indices
    int cut = nKb;                                          // equal keys with an index below `cut` are taken
    if (n_eq > need) {                                      // (uniform over the CTA)
        if (warp == 0) {
            int seen = 0;
            for (int j0 = 0; j0 < nKb && cut == nKb; j0 += 32) {
                const int j = j0 + lane;
                const bool eq = j < nKb && kr[j] == T;
                const unsigned m = __ballot_sync(0xffffffffu, eq);
                if (seen + __popc(m) >= need) {
                    // the need-th equal key is in this group: find its lane
                    unsigned mm = m;
                    for (int r = seen + 1; r < need; ++r) mm &= mm - 1;       // drop the lowest set bits
                    cut = j0 + (__ffs(mm) - 1) + 1;
                }
                seen += __popc(m);
            }
            if (lane == 0) cut_s = cut;
        }
        __syncthreads();
        cut = cut_s;
    }
    // ordered compaction
    bool take[KPT];
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
        const int j = tid + 128 * i;
        take[i] = key[i] != 0u && (key[i] > T || (key[i] == T && j < cut));
        const unsigned m = __ballot_sync(0xffffffffu, take[i]);
        if (lane == 0 && i < kPickMaxChunks) wcnt[i][warp] = __popc(m);
    }
    __syncthreads();
    int32_t* out = col_idx + row * kk;
    int base = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
        const unsigned m = __ballot_sync(0xffffffffu, take[i]);
        int pos = base;
        for (int w = 0; w < warp; ++w) pos += wcnt[i][w];
        if (take[i]) out[pos + __popc(m & ((1u << lane) - 1u))] = tid + 128 * i;
        base += wcnt[i][0] + wcnt[i][1] + wcnt[i][2] + wcnt[i][3];
    }
    if (tid == 0) {
        row_ptr[row] = int32_t(row * kk);
        if (row == rows_total - 1) row_ptr[rows_total] = int32_t(rows_total * kk);
    }
}

}  // namespace salad
