// Linear-attention apply (Eq. 3), standing alone:  O_l = ReLU(Q) KV / (ReLU(Q) . Z + eps).
//
// Used by the linear-only entry points (in the fused call the same arithmetic runs in the epilogue
// of the attention kernel and costs no HBM traffic of its own).  HBM-bound: Q is read once and
// O_l written once, 4*N*d bytes per (batch, head); the per-head state (bf16 d x d, fp32 Z) comes
// from L2.  One persistent CTA per SM walks a contiguous range of 128-row query tiles; loads,
// arithmetic and stores of neighbouring tiles overlap through rings of shared-memory stages and
// two TMEM accumulators:
//   warp 0      TMA producer: Q tiles (ring of NQ stages), the state tile when the head changes
//               (two buffers)
//   warp 1      tcgen05 MMA issuer: num[128 x d] = ReLU(Q) KV, accumulator j & 1
//   warps 2-5   one thread per query row: ReLU of the Q row in place, the denominator by FMAs
//               against Z, the row's coefficient c / (den + eps) into a small ring
//   warps 6-9   one thread per query row: accumulator -> registers, times the coefficient, bf16,
//               swizzled staging tile, TMA store (the tile is free again as soon as the store
//               has read it, long before the next accumulator is ready)
// Every hand-over is an mbarrier with a bounded wait.
//
// ROPE variant (rotary position embedding in the linear branch, Sec. 4.1): a Q stage also holds the fp16
// rotation rows (cos, sin per channel pair) of the tile's 128 tokens, laid out like the Q tile itself (same
// 128-byte swizzle), so a row thread reads the four (cos, sin) values of a 16-byte Q vector from the same
// offset; the denominator takes the un-rotated ReLU values, the MMA the rotated ones.  The ring is two
// stages of 64 KB then, and the state has one buffer (a CTA meets a second head at most once or twice).
#pragma once
#include "ptx.cuh"

namespace salad {

template <int D, bool ROPE = false>
struct ApplyCfg {
    static constexpr int CH = D / 64;                  // 128-byte chunks per row
    static constexpr int Q_CHUNK = 128 * 128;          // bytes of one 64-column chunk of a 128-row tile
    static constexpr int Q_BYTES = CH * Q_CHUNK;
    static constexpr int ST_CHUNK = D * 128;
    static constexpr int ST_BYTES = CH * ST_CHUNK;     // bf16 state [d][d], transposed
    static constexpr int NQ = ROPE ? 2 : 3;            // Q stages
    static constexpr int STAGE_BYTES = ROPE ? 2 * Q_BYTES : Q_BYTES;   // Q tile, then its rotation rows
    static constexpr int NST = ROPE ? 1 : 2;           // state buffers
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_ST = NQ * STAGE_BYTES;
    static constexpr int OFF_O = OFF_ST + NST * ST_BYTES;
    static constexpr int SMEM_BYTES = OFF_O + Q_BYTES + 1024;       // + alignment slack
    static constexpr int THREADS = 320;
    static constexpr int TMEM_COLS = 2 * D;            // 256 or 128: a power of two
    static constexpr int NCOEF = 8;                    // coefficient ring (tiles in flight < 8)
};

struct ApplyParams {
    int N, nQb, H;                // nQb = 128-row tiles per head
    long long tiles;              // B*H*nQb
    const float* z;               // [BH][D]
    const float* static_scale;    // [H] or null
    const float* dyn_scale;       // [B] or null
    float eps;
    int32_t* ws_status;
    int32_t* user_status;
};

struct ApplyBarriers {
    uint64_t q_full[3], q_empty[3], relu_done[3];
    uint64_t st_full[2], st_empty[2], z_ready[2];
    uint64_t acc_full[2], acc_free[2], out_staged, out_free;
};

template <int D, bool ROPE>
__global__ void __launch_bounds__(320)
salad_linear_apply_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_st,
                          const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_r,
                          const ApplyParams p)
{
    using C = ApplyCfg<D, ROPE>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ ApplyBarriers bars;
    __shared__ float z_s[2][D];
    __shared__ float coef_s[C::NCOEF][128];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // contiguous, balanced range of tiles (head-major, so the state changes rarely)
    const long long t0 = p.tiles * blockIdx.x / gridDim.x, t1 = p.tiles * (blockIdx.x + 1) / gridDim.x;

    grid_dependency_wait();
    grid_launch_dependents();
    if (tid == 0) {
        abort_flag = (*reinterpret_cast<volatile int32_t*>(p.ws_status) != 0) ? 2 : 0;    // 2: reported by an earlier kernel
        for (int s = 0; s < C::NQ; ++s) {
            mbar_init(smem_u32(&bars.q_full[s]), 1);
            mbar_init(smem_u32(&bars.q_empty[s]), 1);
            mbar_init(smem_u32(&bars.relu_done[s]), 128);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.st_full[i]), 1);
            mbar_init(smem_u32(&bars.st_empty[i]), 1);
            mbar_init(smem_u32(&bars.z_ready[i]), 128);
            mbar_init(smem_u32(&bars.acc_full[i]), 1);
            mbar_init(smem_u32(&bars.acc_free[i]), 128);
        }
        mbar_init(smem_u32(&bars.out_staged), 128);
        mbar_init(smem_u32(&bars.out_free), 1);
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;

    if (abort_flag == 0) {
    if (warp == 0) {
        // ============================================================== TMA producer
        if (lane == 0) {
            prefetch_tmap(&map_q); prefetch_tmap(&map_st); prefetch_tmap(&map_o);
            if (ROPE) prefetch_tmap(&map_r);
            int prev_bh = -1, n_st = 0, j = 0;
            for (long long t = t0; t < t1; ++t, ++j) {
                const int bh = int(t / p.nQb), qb = int(t % p.nQb);
                if (bh != prev_bh) {
                    const int sb = n_st % C::NST;
                    if (!mbar_wait(smem_u32(&bars.st_empty[sb]), ((n_st / C::NST) & 1) ^ 1, abortp)) break;
                    const uint32_t bar = smem_u32(&bars.st_full[sb]);
                    mbar_arrive_expect_tx(bar, C::ST_BYTES);
                    for (int ch = 0; ch < C::CH; ++ch)
                        tma_load_3d(s_base + C::OFF_ST + sb * C::ST_BYTES + ch * C::ST_CHUNK, &map_st, bar,
                                    ch * 64, 0, bh);
                    ++n_st; prev_bh = bh;
                }
                const int s = j % C::NQ;
                if (!mbar_wait(smem_u32(&bars.q_empty[s]), ((j / C::NQ) & 1) ^ 1, abortp)) break;
                const uint32_t bar = smem_u32(&bars.q_full[s]);
                mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                for (int ch = 0; ch < C::CH; ++ch) {
                    tma_load_3d(s_base + C::OFF_Q + s * C::STAGE_BYTES + ch * C::Q_CHUNK, &map_q, bar,
                                ch * 64, qb * 128, bh);
                    if (ROPE)
                        tma_load_3d(s_base + C::OFF_Q + s * C::STAGE_BYTES + C::Q_BYTES + ch * C::Q_CHUNK, &map_r, bar,
                                    ch * 64, qb * 128, 0);
                }
            }
        }
    } else if (warp == 1) {
        // ============================================================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, D, 0, 0);
            constexpr uint32_t HI = sdesc_hi_sw128(1024);
            int prev_bh = -1, n_st = 0, j = 0, sb = 0;
            bool ok = true;
            for (long long t = t0; t < t1 && ok; ++t, ++j) {
                const int bh = int(t / p.nQb);
                if (bh != prev_bh) {
                    // the MMAs that read the previous state buffer are all issued: hand it back
                    if (prev_bh >= 0) tc_commit(smem_u32(&bars.st_empty[sb]));
                    sb = n_st % C::NST;
                    ok = mbar_wait(smem_u32(&bars.st_full[sb]), (n_st / C::NST) & 1, abortp);
                    if (!ok) break;
                    ++n_st; prev_bh = bh;
                }
                const int s = j % C::NQ, ab = j & 1;
                ok = mbar_wait(smem_u32(&bars.relu_done[s]), (j / C::NQ) & 1, abortp);
                if (ok) ok = mbar_wait(smem_u32(&bars.acc_free[ab]), ((j >> 1) & 1) ^ 1, abortp);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t q_lo = sdesc_lo(s_base + C::OFF_Q + s * C::STAGE_BYTES, 16);
                const uint32_t st_lo = sdesc_lo(s_base + C::OFF_ST + sb * C::ST_BYTES, 16);
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    mma_ss_lohi(tmem + ab * D, q_lo + (((k / 4) * C::Q_CHUNK + (k % 4) * 32) >> 4), HI,
                                st_lo + (((k / 4) * C::ST_CHUNK + (k % 4) * 32) >> 4), HI, idesc, k > 0);
                tc_commit(smem_u32(&bars.q_empty[s]));
                tc_commit(smem_u32(&bars.acc_full[ab]));
            }
        }
    } else if (warp < 6) {
        // ============================================================== ReLU(Q) in place, denominators
        const int row = tid - 64;
        int prev_bh = -1, n_z = 0, j = 0, zb = 0;
        float c_scale = 1.f;
        bool ok = true;
        for (long long t = t0; t < t1 && ok; ++t, ++j) {
            const int bh = int(t / p.nQb);
            if (bh != prev_bh) {
                // Z of the new head into the other buffer; nobody reads that one any more (each
                // thread arrives here only after its last read of the head before the previous one)
                zb = n_z & 1;
                for (int a = row; a < D; a += 128) z_s[zb][a] = __ldg(p.z + size_t(bh) * D + a);
                mbar_arrive(smem_u32(&bars.z_ready[zb]));
                ok = mbar_wait(smem_u32(&bars.z_ready[zb]), (n_z >> 1) & 1, abortp);
                if (!ok) break;
                ++n_z; prev_bh = bh;
                c_scale = 1.f;
                if (p.static_scale) c_scale *= __ldg(p.static_scale + bh % p.H);
                if (p.dyn_scale) c_scale *= __ldg(p.dyn_scale + bh / p.H);
            }
            const int s = j % C::NQ;
            ok = mbar_wait(smem_u32(&bars.q_full[s]), (j / C::NQ) & 1, abortp);
            if (!ok) break;
            uint8_t* qtile = smem + C::OFF_Q + s * C::STAGE_BYTES;
            const float* zz = z_s[zb];
            float den = 0.f;
#pragma unroll
            for (int ch = 0; ch < C::CH; ++ch) {
#pragma unroll
                for (int c16 = 0; c16 < 8; ++c16) {
                    uint4* ptr = reinterpret_cast<uint4*>(qtile + ch * C::Q_CHUNK + row * 128 + ((c16 ^ (row & 7)) << 4));
                    uint4 v = *ptr;
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&v);
                    uint4 tv = make_uint4(0, 0, 0, 0);
                    if (ROPE) tv = *reinterpret_cast<const uint4*>(reinterpret_cast<uint8_t*>(ptr) + C::Q_BYTES);
                    const __half2* th = reinterpret_cast<const __half2*>(&tv);      // (cos, sin) of four pairs
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        hv[e] = __hmax2(hv[e], __float2bfloat162_rn(0.f));
                        const float2 f = __bfloat1622float2(hv[e]);
                        const int a = ch * 64 + c16 * 8 + e * 2;
                        den = fmaf(f.x, zz[a], den);
                        den = fmaf(f.y, zz[a + 1], den);
                        if (ROPE) {
                            const float2 cs = __half22float2(th[e]);
                            hv[e] = __floats2bfloat162_rn(cs.x * f.x - cs.y * f.y, cs.y * f.x + cs.x * f.y);
                        }
                    }
                    *ptr = v;
                }
            }
            // a row with ReLU(Q_n) = 0 and eps = 0 is 0/0: defined as 0 (the numerator is 0 as well)
            coef_s[j % C::NCOEF][row] = (den + p.eps > 0.f) ? c_scale / (den + p.eps) : 0.f;
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&bars.relu_done[s]));
        }
    } else {
        // ============================================================== accumulator -> bf16 -> TMA store
        const int row = (warp & 3) * 32 + lane;                     // = TMEM lane this thread may read
        const uint32_t t_row = tmem + (uint32_t((warp & 3) * 32) << 16);
        int j = 0;
        bool ok = true;
        for (long long t = t0; t < t1; ++t, ++j) {
            const int bh = int(t / p.nQb), qb = int(t % p.nQb);
            const int ab = j & 1;                                   // accumulator
            ok = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&bars.acc_full[ab]), (j >> 1) & 1, abortp));
            if (!ok) break;
            tc_fence_after_sync();
            if (j >= 1) {
                // the store of the previous tile must have read the staging tile before it is overwritten
                if (row == 0) { tma_store_wait_read_all(); mbar_arrive(smem_u32(&bars.out_free)); }
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.out_free), (j - 1) & 1, abortp));
                if (!ok) break;
            }
            const float coef = coef_s[j % C::NCOEF][row];
            uint8_t* otile = smem + C::OFF_O;
#pragma unroll
            for (int cc = 0; cc < D / 16; ++cc) {
                uint32_t nr[16];
                tmem_ld16(t_row + ab * D + cc * 16, nr);
                tmem_wait_ld();
#pragma unroll
                for (int c8 = 0; c8 < 2; ++c8) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = c8 * 8 + e * 2;
                        w[e] = pack_bf16x2(coef * __uint_as_float(nr[c]), coef * __uint_as_float(nr[c + 1]));
                    }
                    const int col16 = cc * 2 + c8;                  // 16-byte chunk index within the row
                    const int ch = col16 / 8, c16 = col16 % 8;
                    *reinterpret_cast<uint4*>(otile + ch * C::Q_CHUNK + row * 128 + ((c16 ^ (row & 7)) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&bars.acc_free[ab]));
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&bars.out_staged));
            if (row == 0) {
                if (mbar_wait(smem_u32(&bars.out_staged), j & 1, abortp)) {
                    for (int ch = 0; ch < C::CH; ++ch)
                        tma_store_3d(&map_o, s_base + C::OFF_O + ch * C::Q_CHUNK, ch * 64,
                                     qb * 128, bh);
                    tma_store_commit();
                } else {
                    ok = false;
                }
            }
        }
        if (row == 0) tma_store_wait_read_all();      // the staging tile must outlive the last store's read
    }
    }  // abort_flag == 0

    // ------------------------------------------------------------------ tear-down
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0) {
        if (tid == 0 && abort_flag == 1) {            // a bounded wait of this CTA ran out
            atomicExch(p.ws_status, SALAD_ERR_TIMEOUT);
            if (p.user_status) atomicExch(p.user_status, SALAD_ERR_TIMEOUT);
        }
        const uint64_t ts = global_timer_ns();
        while (global_timer_ns() - ts < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace salad
