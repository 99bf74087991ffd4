// Full projection of the linear branch and the residual sum (Algorithm 1, Level 1 + integration):
//     out[b, :, n, :] = O_s[b, :, n, :] + s_b * ( concat_h O_l[b, h, n, :] . W^T + bias )
// a [B*N x D] x [D x D] GEMM (D = H*d) with a fused epilogue, on tcgen05 tensor cores.
//
// The head-major layout [B, H, N, d] needs no transposition on either side: a 64-channel K step of
// the concatenated activation is a [128 tokens x 64] box of one head (3-D TMA map), and a 256-column
// output tile is two (d = 128) or four (d = 64) heads of the output tensor.
//   warp 0      TMA producer: A = O_l tile [128 x 64] and B = W tile [256 x 64] per K step, ring of
//               four 48 KB stages
//   warp 1      MMA issuer: four 128 x 256 x 16 tcgen05.mma per K step into accumulator it & 1
//               (2 x 256 TMEM columns: the epilogue of one tile overlaps the main loop of the next)
//   warps 2-5   epilogue, thread = token row: accumulator -> registers, + bias, * s_b, + O_s, bf16,
//               16-byte stores
// Persistent: one CTA per SM walks the tiles with the output-column tile fastest, so the 128-token
// activation panel and W are shared through L2.  Every wait is bounded.
#pragma once
#include "ptx.cuh"

namespace salad {

struct ProjCfg {
    static constexpr int BM = 128, BN = 256, BK = 64;
    static constexpr int A_BYTES = BM * 128, B_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;           // 48 KB
    static constexpr int STAGES = 4;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024;  // + alignment slack
    static constexpr int THREADS = 192;
};

struct ProjParams {
    int B, H, N, d, D;              // D = H * d
    int nMt, nNt, ksteps;           // token tiles per batch item, output-column tiles, D / 64
    long long tiles;                // B * nMt * nNt
    const __nv_bfloat16* o_s;       // [B, H, N, d]
    __nv_bfloat16* out;             // [B, H, N, d]
    const float* bias;              // [D] or null
    const float* s_b;               // [B] or null (1)
    int32_t* status;                // optional device status word
};

__global__ void __launch_bounds__(192)
salad_proj_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                       const ProjParams p)
{
    using C = ProjCfg;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[C::STAGES], empty[C::STAGES], acc_full[2], acc_free[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_free[i]), 128); }
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int chunks_per_head = p.d / 64;

    if (warp == 0) {
        // ============================================================== TMA producer
        if (lane == 0) {
            prefetch_tmap(&map_a); prefetch_tmap(&map_w);
            long long g = 0;
            for (long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
                const int nt = int(tile % p.nNt), mt = int((tile / p.nNt) % p.nMt), b = int(tile / (p.nNt * (long long)p.nMt));
                bool ok = true;
                for (int kk = 0; kk < p.ksteps && ok; ++kk, ++g) {
                    const int s = int(g % C::STAGES);
                    ok = mbar_wait(smem_u32(&empty[s]), (uint32_t(g / C::STAGES) & 1) ^ 1, abortp);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&full[s]);
                    mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                    const uint32_t dst = s_base + s * C::STAGE_BYTES;
                    tma_load_3d(dst, &map_a, bar, (kk % chunks_per_head) * 64, mt * C::BM, b * p.H + kk / chunks_per_head);
                    tma_load_3d(dst + C::A_BYTES, &map_w, bar, kk * 64, nt * C::BN, 0);
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ============================================================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, C::BN, 0, 0);
            constexpr uint32_t HI = sdesc_hi_sw128(1024);
            long long g = 0;
            int it = 0;
            bool ok = true;
            for (long long tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
                const int ab = it & 1;
                ok = mbar_wait(smem_u32(&acc_free[ab]), ((it >> 1) & 1) ^ 1, abortp);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kk = 0; kk < p.ksteps; ++kk, ++g) {
                    const int s = int(g % C::STAGES);
                    ok = mbar_wait(smem_u32(&full[s]), uint32_t(g / C::STAGES) & 1, abortp);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_lo = sdesc_lo(s_base + s * C::STAGE_BYTES, 16);
                    const uint32_t b_lo = sdesc_lo(s_base + s * C::STAGE_BYTES + C::A_BYTES, 16);
#pragma unroll
                    for (int k = 0; k < C::BK / 16; ++k)
                        mma_ss_lohi(tmem + ab * C::BN, a_lo + ((k * 32) >> 4), HI, b_lo + ((k * 32) >> 4), HI, idesc,
                                    (kk > 0 || k > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&empty[s]));
                }
                if (ok) tc_commit(smem_u32(&acc_full[ab]));
            }
        }
    } else {
        // ============================================================== epilogue
        const int row = (warp & 3) * 32 + lane;                     // = TMEM lane this thread may read
        const uint32_t t_row = tmem + (uint32_t((warp & 3) * 32) << 16);
        int it = 0;
        bool ok = true;
        for (long long tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++it) {
            const int nt = int(tile % p.nNt), mt = int((tile / p.nNt) % p.nMt), b = int(tile / (p.nNt * (long long)p.nMt));
            const int ab = it & 1;
            ok = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&acc_full[ab]), (it >> 1) & 1, abortp));
            if (!ok) break;
            tc_fence_after_sync();
            const int n = mt * C::BM + row;
            const float sb = p.s_b ? __ldg(p.s_b + b) : 1.0f;
#pragma unroll 1
            for (int cc = 0; cc < C::BN / 32; ++cc) {
                uint32_t acc[32];
                tmem_ld32(t_row + ab * C::BN + cc * 32, acc);
                tmem_wait_ld();
                const int j0 = nt * C::BN + cc * 32;                // first output channel of this chunk
                if (n < p.N && j0 < p.D) {
                    const size_t idx = ((size_t(b) * p.H + j0 / p.d) * p.N + n) * p.d + j0 % p.d;
                    const uint4* src = reinterpret_cast<const uint4*>(p.o_s + idx);
                    uint4* dst = reinterpret_cast<uint4*>(p.out + idx);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        const uint4 os = src[v4];                       // plain load: out may alias o_s
                        const __nv_bfloat162* oh = reinterpret_cast<const __nv_bfloat162*>(&os);
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int c = v4 * 8 + e * 2;
                            float y0 = __uint_as_float(acc[c]), y1 = __uint_as_float(acc[c + 1]);
                            if (p.bias) { y0 += __ldg(p.bias + j0 + c); y1 += __ldg(p.bias + j0 + c + 1); }
                            const float2 o = __bfloat1622float2(oh[e]);
                            w[e] = pack_bf16x2(fmaf(sb, y0, o.x), fmaf(sb, y1, o.y));
                        }
                        dst[v4] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&acc_free[ab]));
        }
    }

    // ------------------------------------------------------------------ tear-down
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0) {
        if (tid == 0 && p.status) atomicExch(p.status, SALAD_ERR_TIMEOUT);
        const uint64_t ts = global_timer_ns();
        while (global_timer_ns() - ts < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---------------------------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs.  The kernel above is bound by the L2-to-SM operand traffic of a 128 x 256 tile
// (48 KB per 512 tensor cycles and SM); a pair of CTAs on the two SMs of a TPC works on a 256 x 256 tile
// instead (tcgen05.mma.cta_group::2, M = 256): every CTA loads its own 128 token rows of the activation and HALF
// of the 256 W rows of the tile, 32 KB per K step for the same tensor work per SM, which also leaves room for a
// ring of six stages.  No multicast: each CTA fetches its own bytes; their completion is signalled on the
// barrier of the first CTA (cluster rank 0), whose MMA thread issues the products for both; a commit arrives on
// the barriers of both CTAs.  The epilogue of a CTA covers its own 128 rows; the accumulator is handed back to
// the issuing CTA by arrivals from both.
template <int BN_>
struct Proj2Cfg {
    static constexpr int BM = 128, BN = BN_, BK = 64;              // per CTA: BM rows of the pair's 256; BN output columns
    static constexpr int A_BYTES = BM * 128, B_BYTES = (BN / 2) * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;           // 32 KB
    static constexpr int STAGES = 6;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024;  // + alignment slack
    static constexpr int EPI_WARPS = 8;                             // two per quarter of the TMEM lanes: half of the columns each
                                                                    // (sixteen warps were measured slower, four much slower)
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
};

template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(Proj2Cfg<256>::THREADS)
salad_proj_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                            const ProjParams p)
{
    using C = Proj2Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full[C::STAGES], empty[C::STAGES], acc_full[2], acc_free[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                      // 0: issues the products of the pair
    const long long pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(smem_u32(&full[s]), 1); mbar_init(smem_u32(&empty[s]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_free[i]), 2 * 32 * C::EPI_WARPS); }
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc_pair(smem_u32(&tmem_base_slot), 512); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                   // the other CTA's barriers are initialised before anything is signalled on them
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int chunks_per_head = p.d / 64;
    const int nMt2 = (p.N + 2 * C::BM - 1) / (2 * C::BM);          // 256-token tiles per batch item
    const int nNt = (p.D + C::BN - 1) / C::BN;
    const long long tiles = (long long)p.B * nMt2 * nNt;

    if (warp == 0) {
        // ============================================================== TMA producer (each CTA its own part)
        if (lane == 0) {
            prefetch_tmap(&map_a); prefetch_tmap(&map_w);
            long long g = 0;
            for (long long tile = pair; tile < tiles; tile += pairs) {
                const int nt = int(tile % nNt), mt = int((tile / nNt) % nMt2), b = int(tile / (nNt * (long long)nMt2));
                bool ok = true;
                for (int kk = 0; kk < p.ksteps && ok; ++kk, ++g) {
                    const int s = int(g % C::STAGES);
                    ok = mbar_wait(smem_u32(&empty[s]), (uint32_t(g / C::STAGES) & 1) ^ 1, abortp);
                    if (!ok) break;
                    // the bytes of both CTAs are expected on the first CTA's barrier
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&full[s]), 2 * C::STAGE_BYTES);
                    const uint32_t bar = map_to_cta(smem_u32(&full[s]), 0);
                    const uint32_t dst = s_base + s * C::STAGE_BYTES;
                    tma_load_3d_pair(dst, &map_a, bar, (kk % chunks_per_head) * 64, mt * 2 * C::BM + int(rank) * C::BM,
                                     b * p.H + kk / chunks_per_head);
                    tma_load_3d_pair(dst + C::A_BYTES, &map_w, bar, kk * 64, nt * C::BN + int(rank) * (C::BN / 2), 0);
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ============================================================== MMA issuer (first CTA of the pair only)
        if (rank == 0 && lane == 0) {
            const uint32_t idesc = make_idesc_bf16(2 * C::BM, C::BN, 0, 0);
            constexpr uint32_t HI = sdesc_hi_sw128(1024);
            long long g = 0;
            int it = 0;
            bool ok = true;
            for (long long tile = pair; tile < tiles && ok; tile += pairs, ++it) {
                const int ab = it & 1;
                ok = mbar_wait(smem_u32(&acc_free[ab]), ((it >> 1) & 1) ^ 1, abortp);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kk = 0; kk < p.ksteps; ++kk, ++g) {
                    const int s = int(g % C::STAGES);
                    ok = mbar_wait(smem_u32(&full[s]), uint32_t(g / C::STAGES) & 1, abortp);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_lo = sdesc_lo(s_base + s * C::STAGE_BYTES, 16);
                    const uint32_t b_lo = sdesc_lo(s_base + s * C::STAGE_BYTES + C::A_BYTES, 16);
#pragma unroll
                    for (int k = 0; k < C::BK / 16; ++k)
                        mma_ss_lohi_pair(tmem + ab * 256, a_lo + ((k * 32) >> 4), HI, b_lo + ((k * 32) >> 4), HI, idesc,
                                         (kk > 0 || k > 0) ? 1u : 0u);
                    tc_commit_pair(smem_u32(&empty[s]));             // frees the stage in both CTAs
                }
                if (ok) tc_commit_pair(smem_u32(&acc_full[ab]));     // both epilogues may read
            }
        }
    } else {
        // ============================================================== epilogue (each CTA its own 128 rows)
        const int row = (warp & 3) * 32 + lane;                     // = TMEM lane this thread may read
        const uint32_t t_row = tmem + (uint32_t((warp & 3) * 32) << 16);
        constexpr int CC_PER_WARP = (C::BN / 32) / (C::EPI_WARPS / 4);
        const int cc0 = ((warp - 2) / 4) * CC_PER_WARP;              // this warp's share of the 32-column chunks
        int it = 0;
        bool ok = true;
        for (long long tile = pair; tile < tiles; tile += pairs, ++it) {
            const int nt = int(tile % nNt), mt = int((tile / nNt) % nMt2), b = int(tile / (nNt * (long long)nMt2));
            const int ab = it & 1;
            const int n = mt * 2 * C::BM + int(rank) * C::BM + row;
            const float sb = p.s_b ? __ldg(p.s_b + b) : 1.0f;
            // the O_s values of this thread's outputs are fetched while the products of the tile still run
            // (plain loads: out may alias o_s; every element is read by the thread that later writes it)
            uint4 osr[CC_PER_WARP][4];
#pragma unroll
            for (int u = 0; u < CC_PER_WARP; ++u) {
                const int j0 = nt * C::BN + (cc0 + u) * 32;
                if (n < p.N && j0 < p.D) {
                    const uint4* src = reinterpret_cast<const uint4*>(
                        p.o_s + ((size_t(b) * p.H + j0 / p.d) * p.N + n) * p.d + j0 % p.d);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) osr[u][v4] = src[v4];
                }
            }
            ok = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&acc_full[ab]), (it >> 1) & 1, abortp));
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int u = 0; u < CC_PER_WARP; ++u) {
                const int cc = cc0 + u;
                uint32_t acc[32];
                tmem_ld32(t_row + ab * 256 + cc * 32, acc);
                tmem_wait_ld();
                const int j0 = nt * C::BN + cc * 32;                // first output channel of this chunk
                if (n < p.N && j0 < p.D) {
                    const size_t idx = ((size_t(b) * p.H + j0 / p.d) * p.N + n) * p.d + j0 % p.d;
                    uint4* dst = reinterpret_cast<uint4*>(p.out + idx);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        const uint4 os = osr[u][v4];
                        const __nv_bfloat162* oh = reinterpret_cast<const __nv_bfloat162*>(&os);
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int c = v4 * 8 + e * 2;
                            float y0 = __uint_as_float(acc[c]), y1 = __uint_as_float(acc[c + 1]);
                            if (p.bias) { y0 += __ldg(p.bias + j0 + c); y1 += __ldg(p.bias + j0 + c + 1); }
                            const float2 o = __bfloat1622float2(oh[e]);
                            w[e] = pack_bf16x2(fmaf(sb, y0, o.x), fmaf(sb, y1, o.y));
                        }
                        dst[v4] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            // the accumulator goes back to the issuing CTA: an arrival from every epilogue thread of the pair
            tc_fence_before_sync();
            mbar_arrive_cluster(map_to_cta(smem_u32(&acc_free[ab]), 0));
        }
    }

    // ------------------------------------------------------------------ tear-down
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0) {
        if (tid == 0 && p.status) atomicExch(p.status, SALAD_ERR_TIMEOUT);
        const uint64_t ts = global_timer_ns();
        while (global_timer_ns() - ts < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    cluster_sync_all();                   // neither CTA leaves while the other may still signal one of its barriers
    if (warp == 1) tmem_dealloc_pair(tmem, 512);
}

}  // namespace salad
