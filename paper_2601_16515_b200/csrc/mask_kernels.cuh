// Static 3-D sliding-window block mask -> CSR lists of kept key blocks
// (Sec. 3 static sparse attention; Appendix A.1 token flattening, time slowest).
//
// Block pair (i, j) is kept iff some query token of block i and some key token of block j
// lie within (wt, wh, ww) of each other on the T x Hs x Ws grid.  Token pairs are not
// enumerated: a block is a contiguous range of flat token ids, i.e. a few grid rows (t, h)
// each contributing one contiguous run of w.  For every (query row, key row) pair whose t and
// h differ by at most wt and wh, two w-runs [wa, wb] and [ka, kb] hold a pair within ww iff
// ka - wb <= ww and wa - kb <= ww.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace salad {

struct MaskGeom {
    int T, Hs, Ws, N, Bq, Bk, nQb, nKb, Hm;
    // second block geometry, used by the mask heads whose bit is set in MaskWindows::alt (the heads with
    // temporal locality of salad_stswa_mask_build: blocks of whole spatial positions); nQb stays the number of
    // list rows per mask head, rows beyond a head's own blocks are empty
    int Bq2, Bk2, nQb2, nKb2, nQb1;     // nQb1: query blocks of the heads that use (Bq, Bk)
};

// Window sizes (wt, wh, ww) per mask head, passed by value as a kernel argument so that the
// builder needs no device scratch.
struct MaskWindows {
    int32_t w[3 * 256];
    uint32_t alt[8];          // bit hm: mask head hm uses the second block geometry
};

__device__ __forceinline__ bool block_pair_kept(const MaskGeom& g, int Bq, int Bk, int i, int j, int wt, int wh, int ww) {
    const int q0 = i * Bq, q1 = min(g.N, q0 + Bq) - 1;    // inclusive token ranges
    const int k0 = j * Bk, k1 = min(g.N, k0 + Bk) - 1;
    const int qrow0 = q0 / g.Ws, qrow1 = q1 / g.Ws;            // grid rows (t*Hs + h) touched
    const int krow0 = k0 / g.Ws, krow1 = k1 / g.Ws;
    for (int r = qrow0; r <= qrow1; ++r) {
        const int t = r / g.Hs, h = r - t * g.Hs;
        const int wa = (r == qrow0) ? q0 - r * g.Ws : 0;
        const int wb = (r == qrow1) ? q1 - r * g.Ws : g.Ws - 1;
        for (int r2 = krow0; r2 <= krow1; ++r2) {
            const int t2 = r2 / g.Hs, h2 = r2 - t2 * g.Hs;
            if (abs(t2 - t) > wt || abs(h2 - h) > wh) continue;
            const int ka = (r2 == krow0) ? k0 - r2 * g.Ws : 0;
            const int kb = (r2 == krow1) ? k1 - r2 * g.Ws : g.Ws - 1;
            if (ka - wb <= ww && wa - kb <= ww) return true;
        }
    }
    return false;
}

// One warp per CSR row.  FILL = false: write the row's count to counts[row + 1].
// FILL = true: write the kept key-block ids, ascending, at row_ptr[row].
template <bool FILL>
__global__ void __launch_bounds__(256) mask_rows_kernel(const MaskGeom g, const __grid_constant__ MaskWindows windows,
                                                        int32_t* __restrict__ row_ptr,
                                                        int32_t* __restrict__ col_idx) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int rows = g.Hm * g.nQb;
    if (warp >= rows) return;
    const int hm = warp / g.nQb, i = warp - hm * g.nQb;
    const int wt = windows.w[3 * hm], wh = windows.w[3 * hm + 1], ww = windows.w[3 * hm + 2];
    const bool alt = (windows.alt[(hm >> 5) & 7] >> (hm & 31)) & 1u;
    const int Bq = alt ? g.Bq2 : g.Bq, Bk = alt ? g.Bk2 : g.Bk;
    const int nKb = alt ? g.nKb2 : g.nKb, nQb_own = alt ? g.nQb2 : g.nQb1;
    int base = FILL ? row_ptr[warp] : 0;
    int count = 0;
    for (int j0 = 0; j0 < nKb && i < nQb_own; j0 += 32) {
        const int j = j0 + lane;
        const bool keep = (j < nKb) && block_pair_kept(g, Bq, Bk, i, j, wt, wh, ww);
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        if (FILL && keep) col_idx[base + count + __popc(m & ((1u << lane) - 1u))] = j;
        count += __popc(m);
    }
    if (!FILL && lane == 0) row_ptr[warp + 1] = count;
}

// In-place exclusive scan of counts stored at row_ptr[1..rows] (row_ptr[0] = 0 afterwards,
// row_ptr[rows] = nnz).  Single block.  If the total does not fit in int32, row_ptr[rows]
// is set to -1.
__global__ void __launch_bounds__(1024) mask_scan_kernel(int32_t* __restrict__ row_ptr, int rows) {
    __shared__ long long part[1024];
    const int tid = threadIdx.x;
    const int per = (rows + 1023) / 1024;
    const int lo = min(rows, tid * per), hi = min(rows, lo + per);
    long long s = 0;
    for (int r = lo; r < hi; ++r) s += row_ptr[r + 1];
    part[tid] = s;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        long long add = (tid >= off) ? part[tid - off] : 0;
        __syncthreads();
        part[tid] += add;
        __syncthreads();
    }
    long long run = part[tid] - s;   // exclusive prefix of this thread's segment
    for (int r = lo; r < hi; ++r) {
        const int c = row_ptr[r + 1];
        run += c;
        row_ptr[r + 1] = (int32_t)run;   // inclusive value belongs at index r + 1
    }
    __syncthreads();
    if (tid == 0) {
        row_ptr[0] = 0;
        if (part[1023] > 2147483647ll) row_ptr[rows] = -1;
    }
}

}  // namespace salad
