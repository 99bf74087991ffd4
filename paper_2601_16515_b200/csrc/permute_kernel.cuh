// Token permutation for attention heads with temporal locality (Appendix A.1): the flattening with
// time slowest, n = t*S + s (S = Hs*Ws spatial positions), is replaced by m = s*T + t, which puts the
// temporal neighbours of a token next to it, so that a 1-D sliding window reaches them.
//   forward   y[b,h,m,:] = x[b,h,n,:]        inverse   y[b,h,n,:] = x[b,h,m,:]
// for the heads whose flag bit is set; the other heads are copied.  HBM-bound: 4*N*d bytes per head
// (one read, one write).  A CTA writes 128 consecutive destination rows; a thread moves 16 bytes, so
// every row (2*d bytes) is read and written as one contiguous segment.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace salad {

constexpr int kPermuteThreads = 256;
constexpr int kPermuteRows = 128;
constexpr int kPermuteMaxHeads = 1024;

struct PermuteParams {
    int N, T, S, H;
    int vec_per_row;                          // d / 8: 8 or 16
    int inverse;
    uint32_t flag_bits[kPermuteMaxHeads / 32];
};

// grid (ceil(N / 128), B*H)
__global__ void __launch_bounds__(kPermuteThreads)
permute_tokens_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, const PermuteParams p)
{
    const int bh = blockIdx.y, h = bh % p.H;
    const bool flagged = (p.flag_bits[h >> 5] >> (h & 31)) & 1u;
    const int rows_per_pass = kPermuteThreads / p.vec_per_row;       // 32 or 16
    const int c = threadIdx.x % p.vec_per_row, r0 = threadIdx.x / p.vec_per_row;
    const int base = blockIdx.x * kPermuteRows;
    const size_t head = size_t(bh) * p.N * p.vec_per_row;
    constexpr int UNROLL = 8;
    for (int pass0 = 0; pass0 < kPermuteRows / rows_per_pass; pass0 += UNROLL) {
        uint4 v[UNROLL];
        int dst[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int row = base + (pass0 + u) * rows_per_pass + r0;         // destination row
            dst[u] = (row < p.N && pass0 + u < kPermuteRows / rows_per_pass) ? row : -1;
            if (dst[u] >= 0) {
                int src = row;
                if (flagged) {
                    // forward: destination m = s*T + t takes source n = t*S + s; inverse: the other way round
                    if (!p.inverse) { const int s = row / p.T, t = row % p.T; src = t * p.S + s; }
                    else            { const int t = row / p.S, s = row % p.S; src = s * p.T + t; }
                }
                v[u] = __ldg(x + head + size_t(src) * p.vec_per_row + c);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (dst[u] >= 0) y[head + size_t(dst[u]) * p.vec_per_row + c] = v[u];
    }
}

}  // namespace salad
