// Rotation table of a 3-D rotary position embedding for the tokens of a T x Hs x Ws latent grid, the
// input of the rotary linear branch (Sec. 4.1): fp16 (cos, sin) per token and channel pair.
//
// The d/2 channel pairs are shared out among the axes: floor(d/6) pairs each for h and w (after the t
// pairs), the rest for t; pair j of an axis with P pairs turns by  position * base^(-j / P).  A table is
// built once per grid (like a static mask), so the angles are formed in double precision: the fp16 value is
// then the correctly rounded one, identical to a float64 host computation.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace salad {

struct RopeGeom {
    int T, Hs, Ws, pairs, p_t, p_hw;
    long long entries;      // N * pairs
    double log2_base;
};

__global__ void __launch_bounds__(256) rope3d_table_kernel(const RopeGeom g, __half2* __restrict__ table) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= g.entries) return;
    const int n = int(idx / g.pairs), i = int(idx % g.pairs);
    int pos, j, P;
    if (i < g.p_t)               { pos = n / (g.Hs * g.Ws); j = i;                   P = g.p_t; }
    else if (i < g.p_t + g.p_hw) { pos = (n / g.Ws) % g.Hs; j = i - g.p_t;           P = g.p_hw; }
    else                         { pos = n % g.Ws;          j = i - g.p_t - g.p_hw;  P = g.p_hw; }
    const double angle = double(pos) * exp2(-g.log2_base * double(j) / double(P));
    double sn, cs;
    sincos(angle, &sn, &cs);
    table[idx] = __halves2half2(__double2half(cs), __double2half(sn));
}

}  // namespace salad
