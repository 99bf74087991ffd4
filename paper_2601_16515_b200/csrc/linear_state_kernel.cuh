// Linear-attention state (Eq. 3):  KV = sum_j ReLU(K_j)^T V_j  (d x d),  Z = sum_j ReLU(K_j).
//
// HBM-bound: K and V are read exactly once.  The token axis of every (batch, head) is cut
// into `chunks` contiguous ranges of key blocks (64 tokens); one CTA per SM streams one range
// through a ring of stages (linear-only calls: six, 192 KB in flight per SM; fused calls: three,
// so that a CTA of the attention kernel fits on the SM beside it and starts meanwhile):
//   warp 0      TMA producer, K and V tiles through a ring of stages
//   warp 1      tcgen05 MMA issuer; per 16 tokens one MMA  D[d x d] += ReLU(K)^T V with both
//               operands token-major in shared memory (MN-major descriptors), plus one
//               N = 16 MMA against an all-ones tile whose columns all equal Z
//   warps 2-5   apply ReLU to the K tile in place in shared memory (16-byte vectors), and at
//               the end move the fp32 accumulator from TMEM to this chunk's partial in global
//               memory
// A second, tiny kernel adds the partials of a head in a fixed order (deterministic), and
// emits the fp32 state plus the bf16, transposed copy that the fused attention kernel
// multiplies with ReLU(Q).
//
// ROPE variant (linear branch with a rotary position embedding, Sec. 4.1): the ReLU warps rotate the
// channel pairs of ReLU(K) before the MMA reads them, with the fp16 rotation rows (cosine, sine per
// channel pair) of the tile's tokens, which ride in the stage behind K and V (a third TMA load; fetching
// them from L2 with plain loads one tile ahead left the L2 latency exposed on every tile); Z, which takes
// the un-rotated values, they form in registers (a thread always meets the same 8 channels of a 64-channel
// chunk) and sum in a fixed order.  The rotation doubles the work per element: eight ReLU warps.
//
// For d = 64 the MMA still uses M = 128: the "rows 64..127" of the MN-major A operand are
// addressed through the leading-byte-offset, which is pointed at the V tile that follows
// the K tile in the stage; those accumulator rows are ignored.
#pragma once
#include "ptx.cuh"

namespace salad {

template <int D, bool OVERLAP, bool ROPE = false>
struct StateCfg {
    static constexpr int BK = 64;
    static constexpr int CH = D / 64;
    static constexpr int T_CHUNK = BK * 128;           // bytes of one 64-column chunk of a tile
    static constexpr int T_BYTES = CH * T_CHUNK;       // one K or V tile
    static constexpr int R_BYTES = ROPE ? BK * D * 2 : 0;          // fp16 rotation rows of the tile's tokens
    static constexpr int STAGE_BYTES = 2 * T_BYTES + R_BYTES;      // K, V, then the rotation rows
    static constexpr int STAGES = ROPE ? ((D == 128) ? 4 : 8) : (OVERLAP ? 3 : ((D == 128) ? 6 : 8));
    static constexpr int OFF_ONES = STAGES * STAGE_BYTES;
    static constexpr int SMEM_BYTES = OFF_ONES + 2048 + 1024;
    static constexpr int RELU_THREADS = ROPE ? 256 : 128;   // the rotation doubles the work per element
    static constexpr int THREADS = 64 + RELU_THREADS;
    static constexpr int TMEM_COLS = 256;
};

struct StateParams {
    int N, nKb, chunks, blocks_per_chunk;
    float* kv_part;       // [BH][chunks][D][D]
    float* z_part;        // [BH][chunks][D]
    int32_t* ws_status;
    int32_t* user_status;
    int clear_status;         // 1: this kernel is the first of its call and clears the status words itself
    const float* dyn_scale;   // [B] or null: with drop_tau, batch items whose scale is below it are skipped
    float drop_tau;
    int H;
};

// Post-tuning branch dropping (Sec. 4.3): the linear branch of a batch item is skipped when its
// dynamic scale is below the threshold.  Decided on the device, so no host synchronisation.
__device__ __forceinline__ bool branch_dropped(const float* dyn_scale, float tau, int b) {
    return dyn_scale != nullptr && __ldg(dyn_scale + b) < tau;
}

template <int D, bool OVERLAP, bool ROPE>
__global__ void __launch_bounds__(64 + (ROPE ? 256 : 128))
salad_linear_state_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                          const __grid_constant__ CUtensorMap map_r, const StateParams p)
{
    using C = StateCfg<D, OVERLAP, ROPE>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[C::STAGES], relu_done[C::STAGES], empty[C::STAGES], acc_done, z_staged;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunk = blockIdx.x, bh = blockIdx.y;
    // First kernel of a linear-only call (an ordinary launch, so everything before it in the stream is done):
    // its first CTA, which is in the first wave, clears the status words at once; a CTA sets them only after
    // a bounded wait of a second has run out.  No CTA of this kernel reads them (there is no earlier kernel of
    // the call whose failure it would have to honour).
    if (p.clear_status && chunk == 0 && bh == 0 && tid == 0) {
        p.ws_status[0] = 0; p.ws_status[1] = 0;
        if (p.user_status) *p.user_status = 0;
    }
    if (branch_dropped(p.dyn_scale, p.drop_tau, bh / p.H)) {           // whole CTA, before any allocation
        grid_dependency_wait();        // an exit releases the kernels after this one: not before the kernel before it is done
        return;
    }
    const int kb0 = chunk * p.blocks_per_chunk;
    const int kb1 = min(p.nKb, kb0 + p.blocks_per_chunk);
    const int nblk = max(0, kb1 - kb0);

    // K and V are inputs of the call, not products of the kernel before this one in the stream: the
    // producer thread starts the first loads at once, ahead of the set-up below and of the dependency
    // wait (this kernel is launched so that it may begin while its predecessor still runs).
    auto load_stage = [&](int g) {
        const int s = g % C::STAGES;
        const uint32_t bar = smem_u32(&full[s]);
        mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
        const uint32_t dst = s_base + s * C::STAGE_BYTES;
        for (int ch = 0; ch < C::CH; ++ch) {
            tma_load_3d(dst + ch * C::T_CHUNK, &map_k, bar, ch * 64, (kb0 + g) * C::BK, bh);
            tma_load_3d(dst + C::T_BYTES + ch * C::T_CHUNK, &map_v, bar, ch * 64, (kb0 + g) * C::BK, bh);
        }
        if (ROPE) tma_load_3d(dst + 2 * C::T_BYTES, &map_r, bar, 0, (kb0 + g) * C::BK, 0);   // [BK tokens][D halves]
    };
    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&relu_done[s]), C::RELU_THREADS);
            mbar_init(smem_u32(&empty[s]), 1);
        }
        mbar_init(smem_u32(&acc_done), 1);
        mbar_init(smem_u32(&z_staged), C::RELU_THREADS);
        fence_mbar_init();
        prefetch_tmap(&map_k); prefetch_tmap(&map_v);
        if (ROPE) prefetch_tmap(&map_r);
        for (int g = 0; g < min(nblk, C::STAGES); ++g) load_stage(g);
    }
    // all-ones bf16 tile (0x3F80 = 1.0)
    for (int i = tid; i < 2048 / 4; i += C::THREADS)
        reinterpret_cast<uint32_t*>(smem + C::OFF_ONES)[i] = 0x3F803F80u;
    fence_proxy_async_smem();
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS); tmem_relinquish(); }
    // Invariant the attention kernel of a fused call relies on: this kernel releases its dependents only AFTER
    // its own dependency wait (here, and in the early exit of a dropped batch item above).  The attention
    // kernel reads the launch order and the status word, both written by the first kernel of the call,
    // without a wait of its own; it can be placed only once every CTA of the finalize kernel has started,
    // which needs every CTA of this kernel to have got here, i.e. past the wait for that first kernel.
    grid_dependency_wait();            // the status word is cleared by the kernel before
    grid_launch_dependents();
    // 2: the first kernel of the call has reported a failure (a rejected mask): do nothing, report nothing
    if (tid == 0) abort_flag = (!p.clear_status && *reinterpret_cast<volatile int32_t*>(p.ws_status) != 0) ? 2 : 0;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;

    if (abort_flag == 0) {
    if (warp == 0) {
        if (lane == 0) {
            for (int g = C::STAGES; g < nblk; ++g) {          // the first STAGES blocks are already on their way
                const int s = g % C::STAGES;
                if (!mbar_wait(smem_u32(&empty[s]), ((g / C::STAGES) & 1) ^ 1, abortp)) break;
                load_stage(g);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_kv = make_idesc_bf16(128, D, 1, 1);
            const uint32_t idesc_z = make_idesc_bf16(128, 16, 1, 0);
            const uint64_t ones = make_sdesc_sw128(s_base + C::OFF_ONES, 16, 1024);
            bool ok = true;
            for (int g = 0; g < nblk && ok; ++g) {
                const int s = g % C::STAGES;
                ok = mbar_wait(smem_u32(&relu_done[s]), (g / C::STAGES) & 1, abortp);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t ka = s_base + s * C::STAGE_BYTES, va = ka + C::T_BYTES;
#pragma unroll
                for (int k = 0; k < C::BK / 16; ++k) {
                    // 16 tokens = 2 groups of 8 rows of 128 B; next 64 channels one chunk further
                    const uint64_t da = make_sdesc_sw128(ka + k * 2048, C::T_CHUNK, 1024);
                    const uint64_t db = make_sdesc_sw128(va + k * 2048, C::T_CHUNK, 1024);
                    const uint32_t acc = (g > 0 || k > 0) ? 1u : 0u;
                    mma_ss(tmem, da, db, idesc_kv, acc);
                    if (!ROPE) mma_ss(tmem + D, da, ones, idesc_z, acc);
                }
                tc_commit(smem_u32(&empty[s]));
            }
            if (ok) tc_commit(smem_u32(&acc_done));
        }
    } else {
        constexpr int RW = C::RELU_THREADS;
        const int wt = tid - 64;                       // 0..RW-1 within the ReLU/epilogue group
        bool ok = true;
        float zacc[C::CH][8];                          // ROPE: this thread's share of Z
#pragma unroll
        for (int ch = 0; ch < C::CH; ++ch)
#pragma unroll
            for (int e = 0; e < 8; ++e) zacc[ch][e] = 0.f;
        // Vector i*RW + wt of a tile (512 vectors per 64-channel chunk): chunk i*RW / 512, token row
        // (i*RW % 512) / 8 + wt / 8, 16-byte group wt % 8 of the swizzled row = channels 8 * (group ^ (row & 7))
        // .. + 7.  ROPE: its rotation values ((cos, sin) of four channel pairs) are 16 bytes of the stage's
        // rotation rows.
        constexpr int NV = C::T_BYTES / 16 / RW;
        for (int g = 0; g < nblk && ok; ++g) {
            const int s = g % C::STAGES;
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&full[s]), (g / C::STAGES) & 1, abortp));
            if (!ok) break;
            uint4* kt = reinterpret_cast<uint4*>(smem + s * C::STAGE_BYTES);
            const __nv_bfloat162 zero = __float2bfloat162_rn(0.f);
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                uint4 v = kt[i * RW + wt];
                __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&v);
                hv[0] = __hmax2(hv[0], zero); hv[1] = __hmax2(hv[1], zero);
                hv[2] = __hmax2(hv[2], zero); hv[3] = __hmax2(hv[3], zero);
                if (ROPE) {
                    const int row = ((i * RW) % 512) / 8 + (wt >> 3);
                    const int grp = (wt & 7) ^ (row & 7);
                    const uint4 tv = *reinterpret_cast<const uint4*>(
                        smem + s * C::STAGE_BYTES + 2 * C::T_BYTES + (row * D + ((i * RW) / 512) * 64 + grp * 8) * 2);
                    const __half2* th = reinterpret_cast<const __half2*>(&tv);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 x = __bfloat1622float2(hv[e]);
                        zacc[(i * RW) / 512][2 * e] += x.x; zacc[(i * RW) / 512][2 * e + 1] += x.y;
                        const float2 cs = __half22float2(th[e]);
                        hv[e] = __floats2bfloat162_rn(cs.x * x.x - cs.y * x.y, cs.y * x.x + cs.x * x.y);
                    }
                }
                kt[i * RW + wt] = v;
            }
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&relu_done[s]));
        }
        // accumulator -> this chunk's partial.  TMEM lane = key channel a; columns [0,D) = KV
        // row a, column D = Z[a].
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&acc_done), 0, abortp));
        if (ok) {
            tc_fence_after_sync();
            const int a = (warp & 3) * 32 + lane;       // lanes this warp may access
            const uint32_t t_row = tmem + (uint32_t((warp & 3) * 32) << 16);
            float* kv_row = p.kv_part + ((size_t(bh) * p.chunks + chunk) * D + a) * D;
            // (ROPE: eight warps, two per group of 32 lanes: each takes half of the columns)
            constexpr int NCC = (D / 32) / (RW / 128);
            const int cc0 = ((warp - 2) / 4) * NCC;
#pragma unroll
            for (int cc = cc0; cc < cc0 + NCC; ++cc) {
                uint32_t r[32];
                if (nblk > 0) { tmem_ld32(t_row + cc * 32, r); tmem_wait_ld(); }
                if (a < D) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        float4 o = nblk > 0 ? make_float4(__uint_as_float(r[c]), __uint_as_float(r[c + 1]),
                                                          __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
                        *reinterpret_cast<float4*>(kv_row + cc * 32 + c) = o;
                    }
                }
            }
            if (!ROPE) {
                uint32_t zr[32];
                if (nblk > 0) { tmem_ld32(t_row + D, zr); tmem_wait_ld(); }   // reads 32 columns, uses the first
                if (a < D)
                    p.z_part[(size_t(bh) * p.chunks + chunk) * D + a] = nblk > 0 ? __uint_as_float(zr[0]) : 0.f;
            }
        }
        if (ROPE && ok) {
            // Z of this chunk: the threads' register sums, staged in the (now idle) first stage and added
            // per channel over the RW / 8 threads that met it, in a fixed order
            float* zs = reinterpret_cast<float*>(smem);
#pragma unroll
            for (int ch = 0; ch < C::CH; ++ch)
#pragma unroll
                for (int e = 0; e < 8; ++e) zs[wt * (C::CH * 8) + ch * 8 + e] = zacc[ch][e];
            mbar_arrive(smem_u32(&z_staged));
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&z_staged), 0, abortp));
            if (ok && wt < D) {
                const int ch = wt / 64, grp = (wt % 64) / 8, e = wt % 8;
                float sum = 0.f;
#pragma unroll
                for (int r8 = 0; r8 < RW / 8; ++r8)
                    sum += zs[(r8 * 8 + (grp ^ (r8 & 7))) * (C::CH * 8) + ch * 8 + e];
                p.z_part[(size_t(bh) * p.chunks + chunk) * D + wt] = sum;
            }
        }
    }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0) {
        if (tid == 0 && abort_flag == 1) {            // a bounded wait of this CTA ran out
            atomicExch(p.ws_status, SALAD_ERR_TIMEOUT);
            if (p.user_status) atomicExch(p.user_status, SALAD_ERR_TIMEOUT);
        }
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, C::TMEM_COLS);
}

// Sum the partials of each head in chunk order; emit
//   kv_out  fp32 [BH][D][D]  (optional)      z fp32 [BH][D]  (+ optional user copy)
//   kvt     bf16 [BH][D][D]  transposed: kvt[c][a] = KV[a][c], the K-major B operand of
//           num = ReLU(Q) KV in the fused kernel.
template <int D, int ROWS>
__global__ void __launch_bounds__(32 * ROWS)
salad_linear_finalize_kernel(const float* __restrict__ kv_part, const float* __restrict__ z_part, int chunks,
                             float* __restrict__ kv_out, float* __restrict__ z_ws, float* __restrict__ z_out,
                             __nv_bfloat16* __restrict__ kvt, const float* __restrict__ dyn_scale, float drop_tau, int H)
{
    // The kernel after this one may be placed at once (it waits for this one before it touches the
    // state).  In fused calls ROWS = 8: a block is small, 256 threads and few registers, so that while it
    // waits for the state kernel it does not keep a CTA of the attention kernel off its SM.  In linear-only
    // calls, where this kernel's latency counts, ROWS = 32: one element per thread.
    grid_launch_dependents();
    grid_dependency_wait();
    if (branch_dropped(dyn_scale, drop_tau, blockIdx.z / H)) return;
    // grid (D/32, D/32, BH), block (32, ROWS): one 32 x 32 tile of KV per block, 32 / ROWS elements per
    // thread, transposed through shared memory so that both the partial reads and the bf16
    // writes are coalesced
    __shared__ float tile[32][33];
    const int bh = blockIdx.z;
    const int a0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
    for (int r = 0; r < 32 / ROWS; ++r) {
        const int a = a0 + ty + ROWS * r;
        const float* src = kv_part + size_t(bh) * chunks * D * D + size_t(a) * D + c0 + tx;
        // fixed order: ((p0+p4+..)+(p1+p5+..))+((p2+..)+(p3+..)), the chunks % 4 last partials into the first
        // sum; sixteen loads are issued before the first add (the kernel is a chain of L2 round trips otherwise)
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        const int full = chunks & ~3;
        for (int ch0 = 0; ch0 < chunks; ch0 += 16) {
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = (ch0 + u < chunks) ? src[size_t(ch0 + u) * D * D] : 0.f;
#pragma unroll
            for (int u = 0; u < 16; u += 4) {
                if (ch0 + u + 4 <= full) { s0 += v[u]; s1 += v[u + 1]; s2 += v[u + 2]; s3 += v[u + 3]; }
                else if (ch0 + u < chunks) { s0 += v[u]; s0 += v[u + 1]; s0 += v[u + 2]; }    // absent ones are zero
            }
        }
        const float s = (s0 + s1) + (s2 + s3);
        if (kv_out) kv_out[size_t(bh) * D * D + size_t(a) * D + c0 + tx] = s;
        tile[ty + ROWS * r][tx] = s;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 32 / ROWS; ++r)
        kvt[size_t(bh) * D * D + size_t(c0 + ty + ROWS * r) * D + a0 + tx] = __float2bfloat16(tile[tx][ty + ROWS * r]);
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        for (int a = ty * 32 + tx; a < D; a += 32 * ROWS) {
            const float* src = z_part + size_t(bh) * chunks * D + a;
            float s = 0.f;
            for (int ch = 0; ch < chunks; ++ch) s += src[size_t(ch) * D];
            z_ws[size_t(bh) * D + a] = s;
            if (z_out) z_out[size_t(bh) * D + a] = s;
        }
    }
}

// The finalize step with a block-diagonal Level-1 projection (Algorithm 1; Sec. 4.2) folded into the linear
// state: with one d x d block W_h per head on the linear branch,
//     W_h (ReLU(Q_n) KV)^T = (KV W_h^T)^T ReLU(Q_n)^T ,   i.e.   num' = ReLU(Q_n) KV'  with  KV' = KV W_h^T,
// so projecting the state once per head (a d x d x d product) projects every output row for free; the
// normaliser Z is applied before the projection and stays as it is.  The bf16 transposed state the attention
// kernel multiplies with becomes
//     kvt[c][a'] = KV'[a'][c] = sum_a KV[a'][a] * W_h[c][a] ,
// KV summed from the partials in chunk order as in the plain finalize kernel, w [H][D][D] bf16 = W_h[c_out][a_in],
// fp32 arithmetic, one rounding.  kv_out (optional) receives the un-projected fp32 state.
// grid (D/8, BH), 256 threads: a block owns eight rows a' of the state.  It sums them from the partials once
// (every load issued before the first add: one L2 round trip) and keeps them in shared memory; a thread then
// forms the outputs of one output channel c for some of the rows, reading row c of W_h straight from memory
// (32 channels = four 16-byte vectors at a time, the next four fetched while the current ones are used).
// Blocks of this kernel wait on every SM while the state kernel runs, next to a CTA of the attention kernel
// that has started early: 4 KB of shared memory and few registers, so that all three fit.
template <int D>
__global__ void __launch_bounds__(256)
salad_linear_finalize_proj_kernel(const float* __restrict__ kv_part, const float* __restrict__ z_part, int chunks,
                                  const __nv_bfloat16* __restrict__ w, float* __restrict__ kv_out,
                                  float* __restrict__ z_ws, float* __restrict__ z_out, __nv_bfloat16* __restrict__ kvt,
                                  const float* __restrict__ dyn_scale, float drop_tau, int H)
{
    grid_launch_dependents();
    grid_dependency_wait();
    const int bh = blockIdx.y, a0 = blockIdx.x * 8, tid = threadIdx.x;
    if (branch_dropped(dyn_scale, drop_tau, bh / H)) return;
    __shared__ float ks[8][D + 4];
    {
        // the eight rows of KV: D * 8 / 256 elements per thread, the partials of the head in chunk order
        constexpr int EPT = D * 8 / 256;
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int idx = tid + 256 * e, r = idx / D, a = idx % D;
            const float* src = kv_part + size_t(bh) * chunks * D * D + size_t(a0 + r) * D + a;
            float s0 = 0.f, s1 = 0.f;
            for (int ch0 = 0; ch0 < chunks; ch0 += 16) {
                float pv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pv[j] = (ch0 + j < chunks) ? src[size_t(ch0 + j) * D * D] : 0.f;
#pragma unroll
                for (int j = 0; j < 16; j += 2) { s0 += pv[j]; s1 += pv[j + 1]; }
            }
            ks[r][a] = s0 + s1;
            if (kv_out) kv_out[size_t(bh) * D * D + size_t(a0 + r) * D + a] = s0 + s1;
        }
    }
    __syncthreads();
    // outputs of this thread: c = tid % D, rows a' = a0 + OPT * (tid / D) + (0 .. OPT-1)
    constexpr int OPT = D * 8 / 256;
    const int c = tid % D, r0 = (tid / D) * OPT;
    const uint4* wrow = reinterpret_cast<const uint4*>(w + (size_t(bh % H) * D + c) * D);     // row c of W_h: D bf16
    float acc[OPT];
#pragma unroll
    for (int j = 0; j < OPT; ++j) acc[j] = 0.f;
    uint4 cur[4], nxt[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) cur[u] = __ldg(wrow + u);
#pragma unroll
    for (int k0 = 0; k0 < D; k0 += 32) {
        if (k0 + 32 < D) {
#pragma unroll
            for (int u = 0; u < 4; ++u) nxt[u] = __ldg(wrow + (k0 + 32) / 8 + u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&cur[u]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 wv = __bfloat1622float2(h2[e]);
                const int a = k0 + u * 8 + e * 2;
#pragma unroll
                for (int j = 0; j < OPT; ++j) {
                    acc[j] = fmaf(ks[r0 + j][a], wv.x, acc[j]);
                    acc[j] = fmaf(ks[r0 + j][a + 1], wv.y, acc[j]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) cur[u] = nxt[u];
    }
#pragma unroll
    for (int j = 0; j < OPT; ++j)
        kvt[size_t(bh) * D * D + size_t(c) * D + a0 + r0 + j] = __float2bfloat16(acc[j]);
    if (blockIdx.x == 0) {
        for (int a = tid; a < D; a += 256) {
            const float* src = z_part + size_t(bh) * chunks * D + a;
            float sum = 0.f;
            for (int ch = 0; ch < chunks; ++ch) sum += src[size_t(ch) * D];
            z_ws[size_t(bh) * D + a] = sum;
            if (z_out) z_out[size_t(bh) * D + a] = sum;
        }
    }
}

}  // namespace salad
