// First kernel of every call with a sparse branch (Eq. 2 on the block mask M):
//   - clears the status words the later kernels test (unless the list validator, which then runs
//     before it, has done so),
//   - checks what it reads of the mask anyway: the row offsets of every mask head must be
//     non-negative and non-decreasing; otherwise it records SALAD_ERR_BAD_MASK and the later kernels
//     of the call return at once,
//   - writes the launch order of the attention kernel's work items: for every mask head, the query
//     blocks sorted by decreasing length of their kept list, so that the long items start first and
//     the short ones fill the tail.  Counting sort in shared memory; one CTA per mask head.  The
//     order among equal costs is arbitrary (it only affects scheduling).
//
// csr_validate_kernel is the full check of the lists (salad_csr_validate): offsets start at 0, are
// non-decreasing and end within the capacity of col_idx; every row's block ids are strictly
// ascending and inside [0, nKb).  It reads nothing beyond row_ptr[0..rows] and
// col_idx[0..col_capacity), so corrupted lists cannot make it fault.
#pragma once
#include "ptx.cuh"

namespace salad {

__global__ void __launch_bounds__(1024) work_order_kernel(const int32_t* __restrict__ row_ptr, int nQb, int Hm,
                                                          int32_t* __restrict__ order,
                                                          int32_t* __restrict__ ws_status,
                                                          int32_t* __restrict__ user_status, int clear_status) {
    grid_launch_dependents();         // the next kernel of the call may be placed now; it waits for this one
    constexpr int BINS = 2048;
    __shared__ int hist[BINS];
    const int hm = blockIdx.x, tid = threadIdx.x;
    if (hm == 0) {
        // The first CTA is the only writer of the status words in this kernel (so a clear can never
        // overtake a report): it checks the offsets of every mask head.
        int bad = 0;
        for (long long r = tid; r < (long long)Hm * nQb; r += blockDim.x)
            bad |= (row_ptr[r] < 0 || row_ptr[r + 1] < row_ptr[r]) ? 1 : 0;
        bad = __syncthreads_or(bad);
        if (tid == 0) {
            if (bad) {
                *ws_status = SALAD_ERR_BAD_MASK;
                if (user_status) *user_status = SALAD_ERR_BAD_MASK;
            } else if (clear_status) {       // (otherwise the list validator, which ran before, owns the words)
                *ws_status = 0;
                if (user_status) *user_status = 0;
            }
        }
    }
    const int32_t* rp = row_ptr + size_t(hm) * nQb;
    // the length of a list, clamped to a bin: a corrupted offset must not index outside the histogram
    // (the order written for a rejected mask is never used: every later kernel of the call returns at once)
    auto cost_of = [&](int qb) { return max(0, min(BINS - 1, rp[qb + 1] - rp[qb])); };
    for (int i = tid; i < BINS; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int qb = tid; qb < nQb; qb += blockDim.x) atomicAdd(&hist[cost_of(qb)], 1);
    __syncthreads();
    // start position of every cost, largest cost first: an exclusive suffix sum over the bins,
    // two bins per thread, Hillis-Steele over the per-thread totals
    __shared__ int part[1024];
    const int h0 = hist[2 * tid], h1 = hist[2 * tid + 1];
    part[tid] = h0 + h1;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        const int add = (tid + off < 1024) ? part[tid + off] : 0;
        __syncthreads();
        part[tid] += add;
        __syncthreads();
    }
    const int above = part[tid] - (h0 + h1);      // items with a cost in a higher pair of bins
    hist[2 * tid + 1] = above;
    hist[2 * tid] = above + h1;
    __syncthreads();
    for (int qb = tid; qb < nQb; qb += blockDim.x)
        order[size_t(hm) * nQb + atomicAdd(&hist[cost_of(qb)], 1)] = qb;
}

// One warp per CSR row.  The status words (either may be null) receive SALAD_ERR_BAD_MASK when a check
// fails; the host clears them, in stream order, before this kernel.
__global__ void __launch_bounds__(256) csr_validate_kernel(const int32_t* __restrict__ row_ptr,
                                                           const int32_t* __restrict__ col_idx,
                                                           long long col_capacity, int rows, int nKb,
                                                           int32_t* __restrict__ status_a,
                                                           int32_t* __restrict__ status_b) {
    grid_launch_dependents();
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (row >= rows) return;
    const long long a = row_ptr[row], b = row_ptr[row + 1];
    bool bad = (row == 0 && a != 0) || a < 0 || b < a || b > col_capacity;
    if (!bad) {
        for (long long i = a + lane; i < b; i += 32) {
            const int c = col_idx[i];
            if (c < 0 || c >= nKb) bad = true;
            if (i > a && col_idx[i - 1] >= c) bad = true;        // strictly ascending: sorted and unique
        }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) {
        if (status_a) atomicExch(status_a, SALAD_ERR_BAD_MASK);
        if (status_b) atomicExch(status_b, SALAD_ERR_BAD_MASK);
    }
}

}  // namespace salad
