// Block-sparse softmax attention (Eq. 2) fused with the apply step of ReLU linear attention
// (Eq. 3) and the scaled residual sum of Algorithm 1, for sm_100a.
//
// One CTA owns two consecutive query blocks of one (batch, head): two 128-row MMA tiles.
//   warp 0        TMA producer: Q tiles, linear-state tile, K/V tiles of the kept key blocks
//   warp 1, 2     tcgen05 MMA issuers of tile 0 and tile 1 (one thread each); warp 1 owns TMEM
//   warps 4-11    softmax + epilogue of tile 0: two warpgroups, thread = (query row, half of the
//                 64 key columns); the two threads of a row exchange their block max through
//                 shared memory and a two-warp mbarrier
//   warps 12-19   the same for tile 1
// The kept lists of the two query blocks are walked as one sorted merge, so a key block that
// both keep is fetched once and multiplied against both tiles.  Masked blocks are never
// loaded.
//
// A single thread can issue a tcgen05.mma only every ~60 cycles, whatever its size, so the
// work per instruction is kept large: whenever a tile's next kept block is also the next entry
// of the merged list the two blocks form one step, S = Q [K_a; K_b]^T is one 128x128x16 MMA
// series (the K ring is laid out chunk-major so that consecutive stages are contiguous rows),
// and the softmax warps, the P hand-over and O += P V (with P read from TMEM, bf16, over the
// S columns) all work on 128 keys at a time.  Per tile the chain S -> softmax -> O += P V is
// serial; the two tiles have their own issuing threads and run out of phase, so the tensor
// pipe works for one tile while the other tile's warps are in their softmax.
// In a two-block step the two warpgroups of a tile take one block each (64 columns of every
// row); in a one-block step the second warpgroup idles.  The running max lives in the log2
// domain; exponentials start against the max of the earlier steps and the O accumulator is
// rescaled only when the max grows by more than 2^8.  After the last block the warps apply
// ReLU to their Q rows in shared memory, compute the linear denominator with plain FMAs, the
// issuing thread multiplies ReLU(Q) with the bf16 linear state, and the epilogue writes
//     O = O_acc / l + (s_b lambda_h / (den + eps)) * num
// once, as bf16, through a TMA store.
//
// TMEM columns (512 allocated), tile i at 256 i:  [0,128) S of up to two blocks, the first 32
// columns of each 64 reused for P;  [128,128+D) O.  The linear numerator reuses [0,D).
#pragma once
#include "ptx.cuh"

namespace salad {

#ifdef SALAD_TRACE
#define TRACE(role, step, k) do { if (blockIdx.x == 700 && (step) < 64) reinterpret_cast<long long*>(p.lse)[((role) * 64 + (step)) * 8 + (k)] = clock64(); } while (0)
#define TRACE_CTA(k) do { reinterpret_cast<long long*>(p.lse)[4096 + blockIdx.x * 8 + (k)] = (long long)global_timer_ns(); } while (0)
#else
#define TRACE(role, step, k) do {} while (0)
#define TRACE_CTA(k) do {} while (0)
#endif

enum FusedMode { MODE_SPARSE = 1, MODE_LINEAR = 2, MODE_FUSED = 3 };

struct FusedParams {
    int N, H, nQb, nKb, nPairs, Bq, Hm, mode;
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const float* static_scale;   // [H] or null (=1)
    const float* dyn_scale;      // [B] or null (=1)
    const float* z;              // [B*H, D] linear normaliser state
    float* lse;                  // optional [B*H, N]
    float scale_log2;            // softmax_scale * log2(e)
    float eps;
    int32_t* ws_status;          // library status word (never null)
    int32_t* user_status;        // optional
};

template <int D>
struct FusedCfg {
    static constexpr int BK = 64;
    static constexpr int CH = D / 64;               // 128-byte chunks per row
    static constexpr int Q_CHUNK = 128 * 128;       // bytes of one 64-column chunk of a Q tile
    static constexpr int Q_BYTES = CH * Q_CHUNK;
    static constexpr int KV_CHUNK = BK * 128;
    static constexpr int KV_BYTES = CH * KV_CHUNK;  // one K or V tile
    static constexpr int ST_CHUNK = D * 128;
    static constexpr int ST_BYTES = CH * ST_CHUNK;  // linear state, bf16 [D][D]
#ifdef SALAD_EXPERIMENT_RINGS   /* sparse-only experiment: the state tile's space goes to the V ring */
    static constexpr int NK = 4, NV = 5;
    static constexpr int K_CH_STRIDE = NK * KV_CHUNK;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_ST = 2 * Q_BYTES;
    static constexpr int OFF_K = OFF_ST;
#else
    static constexpr int NK = 4, NV = 3;
    static constexpr int K_CH_STRIDE = NK * KV_CHUNK;   // K ring is [chunk][stage][64 rows x 128 B]
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_ST = 2 * Q_BYTES;
    static constexpr int OFF_K = OFF_ST + ST_BYTES;
#endif
    static constexpr int OFF_V = OFF_K + NK * KV_BYTES;
    static constexpr int OFF_X = OFF_V + NV * KV_BYTES;               // row exchange between column halves
    static constexpr int X_BYTES = 2 * 2 * 4 * 128 * 4;              // [tile][half][slot][row] floats
    static constexpr int SMEM_BYTES = OFF_X + X_BYTES + 1024;         // + alignment slack
    static constexpr int THREADS = 640;
    // TMEM columns within a tile's 256
    static constexpr uint32_t COL_S = 0, COL_O = 128;
};

struct FusedBarriers {
    uint64_t q_full[2], st_full, k_full[8], k_empty[8], v_full[8], v_empty[8];
    uint64_t s_full[2], p_ready[2], o_final[2], lin_ready[2], lin_done[2], out_staged[2];
    uint64_t pair[2][4];   // the two warps that share a 32-row TMEM lane quarter of a tile
};

// Sorted merge of the two kept lists.  tag bit i set: tile i keeps this key block.
struct MergeWalk {
    const int32_t* col;
    int e0, end0, e1, end1;
    __device__ __forceinline__ bool next(int& c, int& tag) {
        const int c0 = (e0 < end0) ? __ldg(col + e0) : 0x7fffffff;
        const int c1 = (e1 < end1) ? __ldg(col + e1) : 0x7fffffff;
        c = min(c0, c1);
        if (c == 0x7fffffff) return false;
        tag = (c0 == c ? 1 : 0) | (c1 == c ? 2 : 0);
        e0 += (c0 == c); e1 += (c1 == c);
        return true;
    }
};

template <int D>
__global__ void __launch_bounds__(640, 1)
salad_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                   const __grid_constant__ CUtensorMap map_st, const FusedParams p)
{
    using C = FusedCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ FusedBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int mma_turn;     // taken by the issuing thread whose MMA series owns the tensor pipe

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    const int pair = blockIdx.x % p.nPairs, bh = blockIdx.x / p.nPairs;
    const int h = bh % p.H, b = bh / p.H;
    const int hm = (p.Hm == 1) ? 0 : h;
    const bool sparse = (p.mode & MODE_SPARSE) != 0, linear = (p.mode & MODE_LINEAR) != 0;

    // kept lists of the two tiles
    int qb[2], ls[2], le[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        qb[i] = 2 * pair + i;
        ls[i] = le[i] = 0;
        if (sparse && qb[i] < p.nQb) {
            ls[i] = __ldg(p.row_ptr + hm * p.nQb + qb[i]);
            le[i] = __ldg(p.row_ptr + hm * p.nQb + qb[i] + 1);
        }
    }

    // ------------------------------------------------------------------ set-up
    if (tid == 0) {
        TRACE_CTA(0);
#ifdef SALAD_TRACE
        { uint32_t smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); reinterpret_cast<long long*>(p.lse)[4096 + blockIdx.x * 8 + 7] = smid; }
#endif
        abort_flag = (*reinterpret_cast<volatile int32_t*>(p.ws_status) != 0) ? 1 : 0;
        mma_turn = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.q_full[i]), 1);
            mbar_init(smem_u32(&bars.s_full[i]), 1);
            mbar_init(smem_u32(&bars.p_ready[i]), 8);        // one arrival per softmax warp
            mbar_init(smem_u32(&bars.o_final[i]), 1);
            mbar_init(smem_u32(&bars.lin_ready[i]), 8);
            mbar_init(smem_u32(&bars.lin_done[i]), 1);
            mbar_init(smem_u32(&bars.out_staged[i]), 8);
            for (int qd = 0; qd < 4; ++qd) mbar_init(smem_u32(&bars.pair[i][qd]), 2);
        }
        mbar_init(smem_u32(&bars.st_full), 1);
        for (int s = 0; s < 8; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 2);     // released by both issuing threads
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 2);
        }
        fence_mbar_init();
    }
    if (p.Bq < 128) {
        // rows [Bq, 128) of the Q tiles are never written by TMA: zero them so the unused
        // half of the MMA tile holds finite numbers
        for (int i = tid; i < 2 * C::CH * (128 - p.Bq) * 8; i += C::THREADS) {
            const int chunk = i / ((128 - p.Bq) * 8), rest = i % ((128 - p.Bq) * 8);
            *reinterpret_cast<uint4*>(smem + C::OFF_Q + chunk * C::Q_CHUNK + p.Bq * 128 + rest * 16) =
                make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    if (tid == 0) TRACE_CTA(1);

    if (abort_flag == 0) {
    if (warp == 0) {
        // ============================================================== TMA producer
        if (lane == 0) {
            prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
            for (int i = 0; i < 2; ++i) {
                if (qb[i] >= p.nQb) continue;
                const uint32_t bar = smem_u32(&bars.q_full[i]);
                mbar_arrive_expect_tx(bar, uint32_t(p.Bq) * D * 2);
                for (int ch = 0; ch < C::CH; ++ch)
                    tma_load_3d(s_base + C::OFF_Q + i * C::Q_BYTES + ch * C::Q_CHUNK, &map_q, bar,
                                ch * 64, qb[i] * p.Bq, bh);
            }
            if (linear) {
                const uint32_t bar = smem_u32(&bars.st_full);
                mbar_arrive_expect_tx(bar, C::ST_BYTES);
                for (int ch = 0; ch < C::CH; ++ch)
                    tma_load_3d(s_base + C::OFF_ST + ch * C::ST_CHUNK, &map_st, bar, ch * 64, 0, bh);
            }
            MergeWalk wk{p.col_idx, ls[0], le[0], ls[1], le[1]};
            int col, tag, gk = 0, gv = 0, prev_col = -1;
            bool ok = true;
            auto load_tile = [&](bool is_k, int g, int c) -> bool {
                const int n_stage = is_k ? C::NK : C::NV;
                uint64_t* full = is_k ? bars.k_full : bars.v_full;
                uint64_t* empty = is_k ? bars.k_empty : bars.v_empty;
                const int s = g % n_stage;
                if (!mbar_wait(smem_u32(&empty[s]), ((g / n_stage) & 1) ^ 1, abortp)) return false;
                const uint32_t bar = smem_u32(&full[s]);
                mbar_arrive_expect_tx(bar, C::KV_BYTES);
                for (int ch = 0; ch < C::CH; ++ch) {
                    const uint32_t dst = is_k ? s_base + C::OFF_K + ch * C::K_CH_STRIDE + s * C::KV_CHUNK
                                              : s_base + C::OFF_V + s * C::KV_BYTES + ch * C::KV_CHUNK;
                    tma_load_3d(dst, is_k ? &map_k : &map_v, bar, ch * 64, c * C::BK, bh);
                }
                return true;
            };
            // order of need: K(0), K(1), V(0), K(2), V(1), ...
            while (ok && wk.next(col, tag)) {
                ok = load_tile(true, gk++, col);
                if (ok && prev_col >= 0)
                    ok = load_tile(false, gv++, prev_col);
                prev_col = col;
            }
            if (ok && prev_col >= 0)
                ok = load_tile(false, gv++, prev_col);
        }
    } else if (warp == 1 || warp == 2) {
        // ============================================================== MMA issuer of tile i
        // Walks every entry of the merged list in order: entries of its own tile are multiplied,
        // the others are only released (each K/V stage needs both issuers' release), always
        // after waiting for the stage to be full so that a release can never run a phase ahead.
        if (lane == 0) {
            const int i = warp - 1;
            const uint32_t idesc_qk64 = make_idesc_bf16(128, 64, 0, 0);
            const uint32_t idesc_qk128 = make_idesc_bf16(128, 128, 0, 0);
            const uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
            const uint32_t idesc_lin = make_idesc_bf16(128, D, 0, 0);
            constexpr uint32_t HI = sdesc_hi_sw128(1024);   // the high descriptor word is one constant here
            const uint32_t q_lo = sdesc_lo(s_base + C::OFF_Q + i * C::Q_BYTES, 16);
            const uint32_t k_lo0 = sdesc_lo(s_base + C::OFF_K, 16);
            const uint32_t v_lo0 = sdesc_lo(s_base + C::OFF_V, C::KV_CHUNK);
            const uint32_t t_tile = tmem + i * 256;
            const int len = le[i] - ls[i];
            bool ok = true;
            if (len > 0) {
                ok = mbar_wait(smem_u32(&bars.q_full[i]), 0, abortp);
                tc_fence_after_sync();
            }
            MergeWalk wk{p.col_idx, ls[0], le[0], ls[1], le[1]};
            int col, tag, ncol = 0, ntag = 0, g = 0, t = 0, steps = 0;
            // S[:, d_col .. d_col + N) = Q K^T for N/64 consecutive K stages starting at sk
            auto qk = [&](int sk, uint32_t d_col, uint32_t idesc) {
#pragma unroll
                for (int k = 0; k < D / 16; ++k)   // 16 channels: 32 bytes of each Q and K row, chunk k/4
                    mma_ss_lohi(d_col, q_lo + (((k / 4) * C::Q_CHUNK + (k % 4) * 32) >> 4), HI,
                                k_lo0 + (((k / 4) * C::K_CH_STRIDE + sk * C::KV_CHUNK + (k % 4) * 32) >> 4), HI,
                                idesc, k > 0);
            };
            // O += P V for one block: P (bf16 pairs) at TMEM column p_col, V in stage sv
            auto pv = [&](int sv, uint32_t p_col, bool first) {
                const uint32_t vb_lo = v_lo0 + sv * (C::KV_BYTES >> 4);
#pragma unroll
                for (int k = 0; k < C::BK / 16; ++k)      // 16 keys = 16 rows of 128 bytes
                    mma_ts_lohi(t_tile + C::COL_O, p_col + k * 8, vb_lo + ((k * 2048) >> 4), HI, idesc_pv,
                                (!first || k > 0) ? 1u : 0u);
            };
            // The two tiles' MMA series must not interleave in the tensor pipe: interleaved, both
            // tiles finish their products together, run their softmax together and the tensor
            // and exponential units are never busy at the same time.  An issuing thread holds
            // `mma_turn` for the duration of one series (never across a wait on a barrier), which
            // keeps the tiles out of phase.
            bool holding = false;
            auto take_turn = [&]() -> bool {
                if (holding) return true;
                const uint64_t t0 = global_timer_ns();
                while (atomicCAS(&mma_turn, 0, 1) != 0) {
                    if (*abortp != 0) return false;
                    if (global_timer_ns() - t0 > 1000000000ull) { *abortp = 1; return false; }
                }
                holding = true;
                return true;
            };
            auto give_turn = [&]() {
                if (holding) { atomicExch(&mma_turn, 0); holding = false; }
            };
            // the current and the next entry of the merged list are always known here
            bool have = ok && wk.next(col, tag);
            bool have_n = have && wk.next(ncol, ntag);
            while (ok && have) {
                const bool mine = (tag >> i) & 1;
                const int sk = g % C::NK, sv = g % C::NV;
                TRACE(2 + i, g, 0);
                if (!mine) {
                    // a block of the other tile only: release its stages, after they were filled
                    ok = mbar_wait(smem_u32(&bars.k_full[sk]), (g / C::NK) & 1, abortp);
                    if (!ok) break;
                    mbar_arrive(smem_u32(&bars.k_empty[sk]));
                    have = have_n; col = ncol; tag = ntag;
                    have_n = have && wk.next(ncol, ntag);
                    ok = mbar_wait(smem_u32(&bars.v_full[sv]), (g / C::NV) & 1, abortp);
                    if (!ok) break;
                    mbar_arrive(smem_u32(&bars.v_empty[sv]));
                    ++g;
                    continue;
                }
                const bool paired = have_n && ((ntag >> i) & 1);
                const int sk2 = (g + 1) % C::NK, sv2 = (g + 1) % C::NV;
                ok = mbar_wait(smem_u32(&bars.k_full[sk]), (g / C::NK) & 1, abortp);
                if (ok && paired) ok = mbar_wait(smem_u32(&bars.k_full[sk2]), ((g + 1) / C::NK) & 1, abortp);
                if (ok) ok = take_turn();
                if (!ok) break;
                tc_fence_after_sync();
                if (paired && sk2 == sk + 1) {
                    qk(sk, t_tile + C::COL_S, idesc_qk128);            // both blocks in one series
                } else {
                    qk(sk, t_tile + C::COL_S, idesc_qk64);
                    if (paired) qk(sk2, t_tile + C::COL_S + 64, idesc_qk64);   // ring wrapped between them
                }
                tc_commit(smem_u32(&bars.s_full[i]));
                tc_commit(smem_u32(&bars.k_empty[sk]));
                if (paired) tc_commit(smem_u32(&bars.k_empty[sk2]));
                give_turn();
                TRACE(2 + i, g, 1);
                // advance the list while the softmax runs
                if (paired) { have = wk.next(col, tag); have_n = have && wk.next(ncol, ntag); }
                else { have = have_n; col = ncol; tag = ntag; have_n = have && wk.next(ncol, ntag); }
                ok = mbar_wait(smem_u32(&bars.p_ready[i]), steps & 1, abortp);
                if (ok) ok = mbar_wait(smem_u32(&bars.v_full[sv]), (g / C::NV) & 1, abortp);
                if (ok && paired) ok = mbar_wait(smem_u32(&bars.v_full[sv2]), ((g + 1) / C::NV) & 1, abortp);
                if (ok) ok = take_turn();
                if (!ok) break;
                TRACE(2 + i, g, 2);
                tc_fence_after_sync();
                pv(sv, t_tile + C::COL_S, t == 0);
                tc_commit(smem_u32(&bars.v_empty[sv]));
                if (paired) {
                    pv(sv2, t_tile + C::COL_S + 64, false);
                    tc_commit(smem_u32(&bars.v_empty[sv2]));
                }
                give_turn();
                TRACE(2 + i, g, 3);
                const int nb = paired ? 2 : 1;
                g += nb; t += nb; ++steps;
                if (t == len) tc_commit(smem_u32(&bars.o_final[i]));
            }
            give_turn();
            if (ok && linear && qb[i] < p.nQb) {
                ok = mbar_wait(smem_u32(&bars.st_full), 0, abortp);
                if (ok) ok = mbar_wait(smem_u32(&bars.lin_ready[i]), 0, abortp);
                if (ok) {
                    tc_fence_after_sync();
                    const uint32_t st_lo = sdesc_lo(s_base + C::OFF_ST, 16);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        mma_ss_lohi(t_tile, q_lo + (((k / 4) * C::Q_CHUNK + (k % 4) * 32) >> 4), HI,
                                    st_lo + (((k / 4) * C::ST_CHUNK + (k % 4) * 32) >> 4), HI, idesc_lin, k > 0);
                    tc_commit(smem_u32(&bars.lin_done[i]));
                }
            }
        }
    } else if (warp >= 4) {
        // ============================================================== softmax + epilogue
        const int sw = warp - 4;
        const int i = sw >> 3;                    // tile
        const int hf = (sw >> 2) & 1;             // which half of the key columns / output channels
        const int quarter = warp & 3;             // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;      // query row within the tile = TMEM lane
        const uint32_t t_tile = tmem + i * 256 + (uint32_t(quarter * 32) << 16);
        const bool tile_valid = qb[i] < p.nQb;
        const int len = le[i] - ls[i];
        uint8_t* qtile = smem + C::OFF_Q + i * C::Q_BYTES;
        float* xch = reinterpret_cast<float*>(smem + C::OFF_X);        // [tile][half][slot][row]
        float* x_mine = xch + ((i * 2 + hf) * 4) * 128 + row;
        float* x_other = xch + ((i * 2 + (hf ^ 1)) * 4) * 128 + row;
        uint64_t* pair_bar = &bars.pair[i][quarter];
        constexpr int HD = D / 2;                 // output channels per thread
        float m_run = -INFINITY, l_part = 0.f;
        bool ok = true;
        // every lane of a warp must take the same path around the warp-collective tcgen05
        // loads/stores, so the outcome of a bounded wait is made warp-uniform
        auto wait_uniform = [&](uint64_t* bar, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(smem_u32(bar), parity, abortp));
        };
        auto warp_arrive = [&](uint64_t* bar) {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(bar));
        };

        const bool ragged_keys = (p.N % C::BK) != 0;
        // Steps take one or two blocks.  Two when the tile's next kept block is also the next
        // entry of the merged list (no block of the other tile in between), the same rule the
        // issuing thread applies.
        const int32_t* own = p.col_idx + ls[i];
        const int32_t* oth = p.col_idx + ls[i ^ 1];
        const int oth_len = le[i ^ 1] - ls[i ^ 1];
        int eo = 0;                               // cursor into the other tile's list
        int steps = 0;                            // also the phase count of pair_bar
        for (int t = 0; t < len && ok; ) {
            const int col_a = __ldg(own + t);
            int col_b = col_a;
            bool paired = false;
            if (t + 1 < len) {
                col_b = __ldg(own + t + 1);
                while (eo < oth_len && __ldg(oth + eo) <= col_a) ++eo;
                paired = (eo == oth_len) || (__ldg(oth + eo) >= col_b);
            }
            const bool active = (hf == 0) || paired;          // warpgroup hf takes block hf of the step
            const int valid = p.N - (hf == 0 ? col_a : col_b) * C::BK;   // keys of this block that exist
            const uint32_t t_blk = t_tile + C::COL_S + hf * 64;
            if (row == 0 && hf == 0) TRACE(i, steps, 0);
            ok = wait_uniform(&bars.s_full[i], steps & 1);
            if (!ok) break;
            if (row == 0 && hf == 0) TRACE(i, steps, 1);
            tc_fence_after_sync();

            uint32_t pk[32];
            float lm = -INFINITY, row_sum = 0.f;
            // one pass over this thread's 64 scores, 32 at a time: block max, and (optionally)
            // P = exp2(x * scale - m_ref) as bf16 pairs with its row sum
            auto pass = [&](float m_ref, bool do_exp) {
                lm = -INFINITY; row_sum = 0.f;
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                float sm[2] = {0.f, 0.f};
                uint32_t xa[16], xb[16];
                // 16 columns at a time; the next 16 are in flight while these are processed
                auto chunk = [&](uint32_t* xr, int cc) {
                    float* x = reinterpret_cast<float*>(xr);
                    if (ragged_keys && valid - cc * 16 < 16) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) if (c >= valid - cc * 16) x[c] = -INFINITY;
                    }
#pragma unroll
                    for (int c = 0; c < 16; c += 4) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) mx[e] = fmaxf(mx[e], x[c + e]);
                    }
                    if (do_exp) {
#pragma unroll
                        for (int c = 0; c < 16; c += 2) {
                            const float p0 = ex2_approx(fmaf(x[c], p.scale_log2, -m_ref));
                            const float p1 = ex2_approx(fmaf(x[c + 1], p.scale_log2, -m_ref));
                            sm[0] += p0; sm[1] += p1;
                            pk[cc * 8 + (c >> 1)] = pack_bf16x2(p0, p1);
                        }
                    }
                };
                tmem_ld16(t_blk, xa);
                tmem_wait_ld();
                tmem_ld16(t_blk + 16, xb);
                chunk(xa, 0);
                tmem_wait_ld();
                tmem_ld16(t_blk + 32, xa);
                chunk(xb, 1);
                tmem_wait_ld();
                tmem_ld16(t_blk + 48, xb);
                chunk(xa, 2);
                tmem_wait_ld();
                chunk(xb, 3);
                lm = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                row_sum = sm[0] + sm[1];
            };
            // exponentials against the running max of the earlier steps start at once; the max
            // of this step only matters if it is more than 2^8 larger.  The first step has no
            // earlier max and reduces first.
            if (active) pass(m_run, steps > 0);
            if (row == 0 && hf == 0) TRACE(i, steps, 2);
            x_mine[(steps & 1) * 128] = lm;
            warp_arrive(pair_bar);
            ok = wait_uniform(pair_bar, steps & 1);
            if (!ok) break;
            const float msc = fmaxf(lm, x_other[(steps & 1) * 128]) * p.scale_log2;   // same in both halves
            if (steps == 0) {
                m_run = msc;
                if (active) pass(m_run, true);
            } else if (__any_sync(0xffffffffu, msc > m_run + 8.0f)) {
                // bring this thread's half of the accumulator to the new running max.  Every
                // earlier P V product is complete: it was issued before this step's Q K^T by the
                // same thread, and that product's completion was just observed.  The scores are
                // still in TMEM (P has not been stored yet) and are read again.
                const float m_new = fmaxf(m_run, msc);
                const float alpha = ex2_approx(m_run - m_new);
                l_part *= alpha;
                m_run = m_new;
#pragma unroll
                for (int cc = 0; cc < HD / 16; ++cc) {
                    uint32_t orr[16];
                    tmem_ld16(t_tile + C::COL_O + hf * HD + cc * 16, orr);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 16; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                    tmem_st16(t_tile + C::COL_O + hf * HD + cc * 16, orr);
                }
                tmem_wait_st();
                if (active) pass(m_run, true);
            }
            l_part += row_sum;
            if (row == 0 && hf == 0) TRACE(i, steps, 4);
            // P over the first 32 of this block's 64 S columns (read by this thread only)
            if (active) { tmem_st32(t_blk, pk); tmem_wait_st(); }
            tc_fence_before_sync();
            warp_arrive(&bars.p_ready[i]);
            if (row == 0 && hf == 0) TRACE(i, steps, 5);
            t += paired ? 2 : 1;
            ++steps;
        }
        const int bar_phase = steps;
        if (ok && len > 0) {
            ok = wait_uniform(&bars.o_final[i], 0);
            tc_fence_after_sync();
        }
        if (row == 0 && hf == 0) TRACE_CTA(2 + i);

        // row sum and linear denominator: add the two halves
        float den_part = 0.f;
        if (ok && tile_valid && linear) {
            // ReLU of this thread's half of its Q row, in place, and its share of ReLU(Q_n) . Z
            ok = wait_uniform(&bars.q_full[i], 0);
            if (ok) {
                const float* zrow = p.z + size_t(bh) * D;
#pragma unroll
                for (int j = 0; j < HD / 8; ++j) {
                    const int c16g = hf * (HD / 8) + j;
                    uint4* ptr = reinterpret_cast<uint4*>(qtile + (c16g / 8) * C::Q_CHUNK + row * 128 +
                                                          (((c16g % 8) ^ (row & 7)) << 4));
                    uint4 v = *ptr;
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        hv[e] = __hmax2(hv[e], __float2bfloat162_rn(0.f));
                        const float2 f = __bfloat1622float2(hv[e]);
                        const int a = c16g * 8 + e * 2;
                        den_part = fmaf(f.x, __ldg(zrow + a), den_part);
                        den_part = fmaf(f.y, __ldg(zrow + a + 1), den_part);
                    }
                    *ptr = v;
                }
                fence_proxy_async_smem();
            }
        }
        float l_run = l_part, den = den_part;
        if (ok && tile_valid) {
            x_mine[2 * 128] = l_part;
            x_mine[3 * 128] = den_part;
            warp_arrive(pair_bar);
            ok = wait_uniform(pair_bar, bar_phase & 1);
            if (ok) { l_run += x_other[2 * 128]; den += x_other[3 * 128]; }
        }

        float lin_coef = 0.f;
        if (ok && tile_valid && linear) {
            float c_scale = 1.f;
            if (p.static_scale) c_scale *= __ldg(p.static_scale + h);
            if (p.dyn_scale) c_scale *= __ldg(p.dyn_scale + b);
            lin_coef = c_scale / (den + p.eps);
            warp_arrive(&bars.lin_ready[i]);       // ReLU(Q) is in shared memory (fenced above)
            ok = wait_uniform(&bars.lin_done[i], 0);
            tc_fence_after_sync();
        }

        if (ok && tile_valid) {
            // O = O_acc / l + lin_coef * num for this thread's channels, rounded once to bf16,
            // staged in the Q tile (128-byte swizzle) for the TMA store
            const float inv_l = (len > 0) ? 1.0f / l_run : 0.f;
#pragma unroll
            for (int cc = 0; cc < HD / 16; ++cc) {
                uint32_t orr[16], nr[16];
                if (len > 0) tmem_ld16(t_tile + C::COL_O + hf * HD + cc * 16, orr);
                if (linear) tmem_ld16(t_tile + hf * HD + cc * 16, nr);
                tmem_wait_ld();
#pragma unroll
                for (int c8 = 0; c8 < 2; ++c8) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = c8 * 8 + e * 2;
                        float o0 = (len > 0) ? __uint_as_float(orr[c]) * inv_l : 0.f;
                        float o1 = (len > 0) ? __uint_as_float(orr[c + 1]) * inv_l : 0.f;
                        if (linear) {
                            o0 = fmaf(lin_coef, __uint_as_float(nr[c]), o0);
                            o1 = fmaf(lin_coef, __uint_as_float(nr[c + 1]), o1);
                        }
                        w[e] = pack_bf16x2(o0, o1);
                    }
                    const int c16g = (hf * HD + cc * 16 + c8 * 8) / 8;      // 16-byte chunk index within the row
                    *reinterpret_cast<uint4*>(qtile + (c16g / 8) * C::Q_CHUNK + row * 128 +
                                              (((c16g % 8) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            fence_proxy_async_smem();
            warp_arrive(&bars.out_staged[i]);
            if (row == 0 && hf == 0 && mbar_wait(smem_u32(&bars.out_staged[i]), 0, abortp)) {
                for (int ch = 0; ch < C::CH; ++ch)
                    tma_store_3d(&map_o, s_base + C::OFF_Q + i * C::Q_BYTES + ch * C::Q_CHUNK, ch * 64,
                                 qb[i] * p.Bq, bh);
                tma_store_commit();
                tma_store_wait_all();
            }
#ifndef SALAD_TRACE
            if (p.lse != nullptr && hf == 0) {
                const int n = qb[i] * p.Bq + row;
                if (row < p.Bq && n < p.N)
                    p.lse[size_t(bh) * p.N + n] =
                        (len > 0) ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            }
#endif
        }
    }
    }  // abort_flag == 0

    // ------------------------------------------------------------------ tear-down
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) TRACE_CTA(4);
    if (abort_flag != 0) {
        // a bounded wait expired somewhere: report, give copies in flight time to land, leave
        if (tid == 0) {
            atomicExch(p.ws_status, 1);
            if (p.user_status) atomicExch(p.user_status, -6);
        }
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, 512);
}

}  // namespace salad
