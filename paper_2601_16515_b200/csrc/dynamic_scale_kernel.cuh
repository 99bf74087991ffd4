// Input- and timestep-aware dynamic scaling factor (Algorithm 1, Level 2; Sec. 4.2):
//     s[b] = Mean_n sigmoid( <X_t[b, n, :], w> + bias ).
// HBM-bound: X_t (bf16 [B, N, D]) is read exactly once, 2*N*D bytes per batch item.
// One warp per token at a time: the lanes read the token's D channels as 16-byte vectors
// (512 contiguous bytes per warp instruction), multiply with w held as fp32 in shared memory,
// reduce with shuffles, and lane 0 adds the sigmoid to the warp's running sum.  Each CTA writes
// one partial per (batch item, CTA); a second, tiny kernel adds the partials of a batch item in
// a fixed order (deterministic) and divides by N.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace salad {

constexpr int kDynScaleThreads = 256;

// dot product of eight bf16 channels (one 16-byte vector) with eight fp32 weights, added to acc
__device__ __forceinline__ float dot8(const uint4& v, const float4& w0, const float4& w1, float acc) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
    const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
    const float2 f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
    acc = fmaf(f0.x, w0.x, acc); acc = fmaf(f0.y, w0.y, acc);
    acc = fmaf(f1.x, w0.z, acc); acc = fmaf(f1.y, w0.w, acc);
    acc = fmaf(f2.x, w1.x, acc); acc = fmaf(f2.y, w1.y, acc);
    acc = fmaf(f3.x, w1.z, acc); acc = fmaf(f3.y, w1.w, acc);
    return acc;
}

__global__ void __launch_bounds__(kDynScaleThreads)
dynamic_scale_partial_kernel(const uint4* __restrict__ x, const float* __restrict__ w, float bias,
                             int N, int D, float* __restrict__ partial)
{
    extern __shared__ float w_s[];                     // D floats
    __shared__ float warp_sum[kDynScaleThreads / 32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.y, G = gridDim.x;
    for (int c = tid; c < D; c += kDynScaleThreads) w_s[c] = w[c];
    __syncthreads();

    const int chunks = D / 8;                          // 16-byte vectors per token
    const int warps_total = G * (kDynScaleThreads / 32);
    float acc = 0.f;                                   // lane 0: sum of sigmoids of this warp's tokens
    // two tokens per trip: twice the loads in flight per warp
    for (int n = blockIdx.x * (kDynScaleThreads / 32) + warp; n < N; n += 2 * warps_total) {
        const int n1 = n + warps_total;
        const bool two = n1 < N;
        const uint4* row0 = x + (size_t(b) * N + n) * chunks;
        const uint4* row1 = x + (size_t(b) * N + (two ? n1 : n)) * chunks;
        float dot0 = 0.f, dot1 = 0.f;
#pragma unroll 2
        for (int c = lane; c < chunks; c += 32) {
            const uint4 v0 = __ldg(row0 + c);
            const uint4 v1 = __ldg(row1 + c);
            const float4 w0 = *reinterpret_cast<const float4*>(w_s + c * 8);
            const float4 w1 = *reinterpret_cast<const float4*>(w_s + c * 8 + 4);
            dot0 = dot8(v0, w0, w1, dot0);
            dot1 = dot8(v1, w0, w1, dot1);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            dot0 += __shfl_xor_sync(0xffffffffu, dot0, off);
            dot1 += __shfl_xor_sync(0xffffffffu, dot1, off);
        }
        acc += 1.0f / (1.0f + __expf(-(dot0 + bias)));
        if (two) acc += 1.0f / (1.0f + __expf(-(dot1 + bias)));
    }
    if (lane == 0) warp_sum[warp] = acc;
    __syncthreads();
    if (tid == 0) {
        float s = 0.f;
        for (int i = 0; i < kDynScaleThreads / 32; ++i) s += warp_sum[i];
        partial[size_t(b) * G + blockIdx.x] = s;
    }
}

__global__ void __launch_bounds__(32)
dynamic_scale_finalize_kernel(const float* __restrict__ partial, int G, int N, float* __restrict__ s_out)
{
    const int b = blockIdx.x, lane = threadIdx.x;
    float s = 0.f;
    for (int g = lane; g < G; g += 32) s += partial[size_t(b) * G + g];     // fixed assignment and order
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) s_out[b] = s / float(N);
}

}  // namespace salad
