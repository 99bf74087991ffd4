// Block-sparse softmax attention (Eq. 2) fused with the apply step of ReLU linear attention
// (Eq. 3) and the scaled residual sum of Algorithm 1, for sm_100a.
//
// One CTA owns one query block of one (batch, head): a 128-row MMA tile.  Two CTAs share an SM
// (each takes half of its shared memory, registers and tensor memory), so the set-up, the first
// loads and the epilogue of one overlap the main loop of the other, and the two tiles of an SM run
// independently of each other.
//   warp 0        TMA producer of the Q tile, the K ring and (at the end) the linear-state tile
//   warp 1        TMA producer of the V ring (independent of the K ring, so neither ring can
//                 stall the other)
//   warp 2        tcgen05 issuer of S = Q K^T; owns the TMEM allocation
//   warp 3        tcgen05 issuer of O += P V and of the linear numerator
//                 (an issuing warp walks its loop as a whole, every lane polling the barriers, and one
//                 elected lane issues: the operands of a product are then warp-uniform values, which
//                 keeps the cost of issuing one low -- measured 27 against 45 cycles per instruction
//                 when a single lane runs the loop alone)
//   warps 4-11    softmax + epilogue warps: a warp works on 16 query rows (TMEM lanes) with the
//                 16-lane load/store shapes, four threads share a row and each thread serves two
//                 rows; row maxima and sums are combined with two shuffles
// Masked blocks are never loaded.
//
// S = Q K^T (128x64xd, operands in shared memory) of block t lands in TMEM score buffer t & 1;
// the softmax warps copy it to registers and write P = exp2(.), as bf16, over the first half of
// the same buffer, which O += P V then reads.  The scores of block t + 1 go to the other buffer
// as soon as the P V product of block t - 1 has read it, so both products of the neighbouring
// blocks overlap the softmax of block t.  The running max lives in the log2 domain; exponentials
// start against the max of the earlier blocks and the O accumulator is rescaled only when the max
// grows by more than 2^8.  The two products have their own issuing warps: each waits only for
// what its next MMA series needs, so it reacts as soon as that arrives.  One commit per series: the
// barrier that announces the scores of block t also frees the K-ring stage for block t + 2, the one
// that announces the completion of P V the V-ring stage.
// The four producer / issuer warps (one warpgroup) hand registers to the eight softmax warps
// (setmaxnreg: 40 against 96 per thread), which keeps the softmax loop free of spills.
// After the last block the softmax warps apply ReLU to the Q rows in shared memory and compute the
// linear denominator with plain FMAs; the linear state (bf16, transposed) is loaded over the K
// ring, which is idle by then; the issuing thread multiplies ReLU(Q) with it, and the epilogue
// writes
//     O = O_acc / l + (s_b lambda_h / (den + eps)) * num
// once, as bf16, through a TMA store.
// The kernels that make the linear state come before this one in the stream and run beside it: this
// kernel is launched to start early and waits for them only in warp 0, just before the state tile and
// the normaliser Z are fetched, so the softmax attention of the first tiles hides the state pass.
//
// TMEM columns (256 allocated):  [0,64) and [64,128) two score buffers (block t uses buffer
// t & 1; its probabilities, packed bf16, overwrite the first 32 columns of the same buffer);
// [128,128+D) O.  The linear numerator reuses [0,D).
#pragma once
#include "ptx.cuh"

namespace salad {

enum FusedMode { MODE_SPARSE = 1, MODE_LINEAR = 2, MODE_FUSED = 3 };

// Heads with temporal locality (Appendix A.1): their tokens are taken in the order that groups them by spatial
// position, m = s * T + t for token n = t * S + s, through 4-D tensor maps, without a re-ordering pass.  A
// key block of such a head is the T tokens of ks spatial positions (ks * T <= 64 rows of the 64-row tile), a
// query block those of kq positions (kq * T <= 128 rows); the unused rows of the tiles hold zeros and their
// keys are masked.
struct TemporalHeads {
    int T, S;                    // T == 0: no head is re-ordered
    int kq, ks;                  // spatial positions per query / key block
    int nQb, nKb;                // blocks per head: ceil(S / kq), ceil(S / ks)
    uint32_t flags[8];           // bit h: head h is temporal (H <= 256)
};

struct FusedParams {
    int N, H, nQb, nKb, Bq, Hm, mode;     // nQb: list rows per mask head; nKb: key blocks of a head in token order
    int nQb_tok;                 // query blocks of a head in token order (== nQb unless temporal heads have more)
    TemporalHeads th;
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* order;        // [Hm][nQb] launch order of the query blocks, or null (identity)
    int BH;                      // batch * heads
    const float* static_scale;   // [H] or null (=1)
    const float* dyn_scale;      // [B] or null (=1)
    const float* z;              // [B*H, D] linear normaliser state
    float* lse;                  // optional [B*H, N]
    float scale_log2;            // softmax_scale * log2(e)
    float eps;
    float drop_tau;              // linear branch of batch item b skipped when dyn_scale[b] < drop_tau
    const __half* rope;          // [N][D] fp16: (cos, sin) per token and channel pair of the rotary linear branch, or null
    int wait_at_top;             // 1: wait for the kernel before this one at once (calls without state kernels)
    int32_t* ws_status;          // library status word (never null)
    int32_t* user_status;        // optional
};

template <int D>
struct FusedCfg {
    static constexpr int BK = 64;
    static constexpr int CH = D / 64;               // 128-byte chunks per row
    static constexpr int Q_CHUNK = 128 * 128;       // bytes of one 64-column chunk of the Q tile
    static constexpr int Q_BYTES = CH * Q_CHUNK;
    static constexpr int KV_CHUNK = BK * 128;
    static constexpr int KV_BYTES = CH * KV_CHUNK;  // one K or V tile
    static constexpr int ST_CHUNK = D * 128;
    static constexpr int ST_BYTES = CH * ST_CHUNK;  // linear state, bf16 [D][D]: as large as the K ring
    static constexpr int NK = 2, NV = 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = Q_BYTES;
    static constexpr int OFF_ST = OFF_K;            // loaded over the K ring once every Q K^T has completed
    static constexpr int OFF_V = OFF_K + NK * KV_BYTES;
    static constexpr int SMEM_BYTES = OFF_V + NV * KV_BYTES + 1024;   // + alignment slack: 97 KB at D = 128
    static constexpr int THREADS = 384;
    // TMEM columns: two score buffers of 64 (P overwrites the first 32 columns of the buffer its
    // scores came from), then the output accumulator
    static constexpr uint32_t COL_SP = 0, SP_STRIDE = 64, COL_O = 128;
    static constexpr uint32_t TMEM_COLS = 256;
};
static_assert(FusedCfg<128>::ST_BYTES == FusedCfg<128>::NK * FusedCfg<128>::KV_BYTES, "the state tile fills the K ring");
static_assert(FusedCfg<64>::ST_BYTES <= FusedCfg<64>::NK * FusedCfg<64>::KV_BYTES, "the state tile fits in the K ring");

struct FusedBarriers {
    uint64_t q_full, st_full, k_full[2], v_full[2];
    uint64_t s_full[2], p_ready[2], pv_done[2], o_final, lin_ready, lin_done, out_staged, z_full;
};

template <int D>
__global__ void __launch_bounds__(384, 2)
salad_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                   const __grid_constant__ CUtensorMap map_st, const __grid_constant__ CUtensorMap map_q4,
                   const __grid_constant__ CUtensorMap map_k4, const __grid_constant__ CUtensorMap map_v4,
                   const __grid_constant__ CUtensorMap map_o4, const FusedParams p)
{
    using C = FusedCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ FusedBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float z_s[D];          // linear normaliser state of this head

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t s_base = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The work order comes from the first kernel of the call.  Without a linear branch that is the kernel
    // before this one.  With one, the state kernels lie between, and this kernel does not wait for them
    // here: it runs beside them (each of their CTAs has passed its own wait for the first kernel before
    // a CTA of this one is placed) and waits only where it first touches the state, in the epilogue.
    if ((p.mode & MODE_LINEAR) == 0 || p.wait_at_top) grid_dependency_wait();
    grid_launch_dependents();

    // work item: head by head (K/V of one head stay hot in L2: ordering the cheapest items of all
    // heads last instead was measured to shorten the launch by 0.3 % and to raise its DRAM traffic by
    // half), within a head the query blocks from the most to the least expensive, so that the
    // kernel ends on short items
    const int rank = blockIdx.x % p.nQb, bh = blockIdx.x / p.nQb;
    const int h = bh % p.H, b = bh / p.H;
    const int hm = (p.Hm == 1) ? 0 : (p.Hm == p.H ? h : bh);   // one mask, one per head, or one per (batch, head)
    const int qb = p.order ? __ldg(p.order + size_t(hm) * p.nQb + rank) : rank;
    // temporal head: blocks of spatial positions, fetched through the 4-D maps
    const bool perm = p.th.T > 0 && ((p.th.flags[h >> 5] >> (h & 31)) & 1u);
    const int q_rows = perm ? p.th.kq * p.th.T : p.Bq;          // rows of the 128-row tile that hold queries
    const int k_rows = perm ? p.th.ks * p.th.T : C::BK;         // rows of a 64-row tile that hold keys
    if (qb >= (perm ? p.th.nQb : p.nQb_tok)) return;            // (a list row beyond this head's blocks: whole CTA)
    const bool sparse = (p.mode & MODE_SPARSE) != 0;
    // post-tuning branch dropping (Sec. 4.3): no linear work at all for a dropped batch item
    const bool linear = (p.mode & MODE_LINEAR) != 0 &&
                        !(p.dyn_scale != nullptr && __ldg(p.dyn_scale + b) < p.drop_tau);
    // kept list of the query block
    int ls = 0, le = 0;
    if (sparse) {
        ls = __ldg(p.row_ptr + size_t(hm) * p.nQb + qb);
        le = __ldg(p.row_ptr + size_t(hm) * p.nQb + qb + 1);
    }

    // ------------------------------------------------------------------ set-up
    if (tid == 0) {
        // 2: an earlier kernel of this call has already reported a failure (a rejected mask, an expired wait):
        // this CTA starts nothing and reports nothing; 1 (set by a bounded wait of this CTA): a time-out
        abort_flag = (*reinterpret_cast<volatile int32_t*>(p.ws_status) != 0) ? 2 : 0;
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.st_full), 1);
        mbar_init(smem_u32(&bars.o_final), 1);
        mbar_init(smem_u32(&bars.lin_ready), 256);
        mbar_init(smem_u32(&bars.lin_done), 1);
        mbar_init(smem_u32(&bars.out_staged), 256);
        mbar_init(smem_u32(&bars.z_full), 32);
        for (int j = 0; j < 2; ++j) {
            mbar_init(smem_u32(&bars.s_full[j]), 1);
            mbar_init(smem_u32(&bars.p_ready[j]), 8);          // one arrival per softmax warp
            mbar_init(smem_u32(&bars.pv_done[j]), 1);
            mbar_init(smem_u32(&bars.k_full[j]), 1);
            mbar_init(smem_u32(&bars.v_full[j]), 1);
        }
        fence_mbar_init();
    }
    if (q_rows < 128 || k_rows < C::BK) {
        // rows [q_rows, 128) of the Q tile and [k_rows, 64) of the K and V tiles are never written by TMA:
        // zero them so that the unused part of an MMA tile holds finite numbers (zero keys are masked, zero
        // value rows meet zero probabilities)
        for (int i = tid; i < C::CH * (128 - q_rows) * 8; i += C::THREADS) {
            const int chunk = i / ((128 - q_rows) * 8), rest = i % ((128 - q_rows) * 8);
            *reinterpret_cast<uint4*>(smem + C::OFF_Q + chunk * C::Q_CHUNK + q_rows * 128 + rest * 16) =
                make_uint4(0, 0, 0, 0);
        }
        const int per_tile = (C::BK - k_rows) * 8;                // 16-byte vectors per 64-row chunk of a K or V tile
        for (int i = tid; i < (C::NK + C::NV) * C::CH * per_tile; i += C::THREADS) {
            const int tile = i / per_tile, rest = i % per_tile;  // K: [chunk][stage], V: [stage][chunk]: all 8 KB apart
            *reinterpret_cast<uint4*>(smem + C::OFF_K + tile * C::KV_CHUNK + k_rows * 128 + rest * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async_smem();
    }
    if (warp == 2) { tmem_alloc(smem_u32(&tmem_base_slot), C::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int len = le - ls;
    const bool inherited_abort = abort_flag != 0;      // uniform: read after the barrier above, before any wait

    // a bounded wait taken by a whole warp: warp-uniform outcome
    auto wait_warp = [&](uint64_t* bar, uint32_t parity) -> bool {
        return __all_sync(0xffffffffu, mbar_wait(smem_u32(bar), parity, abortp));
    };

    if (!inherited_abort) {
    if (warp < 4) {
    // the four producer / issuer warps (one warpgroup) give registers up, the eight softmax warps take them
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    if (warp == 0) {
        // ============================================================== TMA producer: Q, the K ring, the state tile
        bool ok = true;
        if (lane == 0) {
            prefetch_tmap(&map_q); prefetch_tmap(&map_k);
            // A block with no kept key block and no linear branch never reads Q: its epilogue
            // stages zeros in the Q tile without waiting for q_full, so nothing may land there.
            if (len > 0 || linear) {
                const uint32_t bar = smem_u32(&bars.q_full);
                mbar_arrive_expect_tx(bar, uint32_t(q_rows) * D * 2);
                for (int ch = 0; ch < C::CH; ++ch) {
                    if (perm) tma_load_4d(s_base + C::OFF_Q + ch * C::Q_CHUNK, &map_q4, bar, ch * 64, 0, qb * p.th.kq, bh);
                    else tma_load_3d(s_base + C::OFF_Q + ch * C::Q_CHUNK, &map_q, bar, ch * 64, qb * p.Bq, bh);
                }
            }
            for (int t = 0; t < len; ++t) {
                const int s = t % C::NK;
                // stage s = t & 1 is free once Q K^T of block t - 2 has completed: the barrier that hands its
                // scores to the softmax warps says so (one commit serves both)
                if (t >= C::NK) ok = mbar_wait(smem_u32(&bars.s_full[s]), ((t >> 1) - 1) & 1, abortp);
                if (!ok) break;
                const int col = __ldg(p.col_idx + ls + t);
                const uint32_t bar = smem_u32(&bars.k_full[s]);
                mbar_arrive_expect_tx(bar, uint32_t(k_rows) * D * 2);
                for (int ch = 0; ch < C::CH; ++ch) {     // chunk-major: the two stages of a chunk are adjacent
                    const uint32_t dst = s_base + C::OFF_K + ch * (C::NK * C::KV_CHUNK) + s * C::KV_CHUNK;
                    if (perm) tma_load_4d(dst, &map_k4, bar, ch * 64, 0, col * p.th.ks, bh);
                    else tma_load_3d(dst, &map_k, bar, ch * 64, col * C::BK, bh);
                }
            }
        }
        if (linear) {
            // From here on the linear state is needed: wait for the kernels that make it (whole warp: the
            // other lanes fetch the normaliser Z of this head for the softmax warps meanwhile).
            __syncwarp();
            grid_dependency_wait();
            if (*reinterpret_cast<volatile int32_t*>(p.ws_status) != 0 && *abortp == 0) *abortp = 2;   // the state kernel gave up (and said so)
            for (int a = lane; a < D; a += 32) z_s[a] = __ldcg(p.z + size_t(bh) * D + a);
            mbar_arrive(smem_u32(&bars.z_full));
            if (lane == 0 && ok) {
                // the state tile goes over the K ring: every Q K^T must have read its K block.  The products
                // complete in order, so the last one (signalled on its score buffer's barrier) covers all.
                if (len > 0) ok = mbar_wait(smem_u32(&bars.s_full[(len - 1) & 1]), ((len - 1) >> 1) & 1, abortp);
                if (ok) {
                    prefetch_tmap(&map_st);
                    const uint32_t bar = smem_u32(&bars.st_full);
                    mbar_arrive_expect_tx(bar, C::ST_BYTES);
                    for (int ch = 0; ch < C::CH; ++ch)
                        tma_load_3d(s_base + C::OFF_ST + ch * C::ST_CHUNK, &map_st, bar, ch * 64, 0, bh);
                }
            }
        }
    } else if (warp == 1) {
        // ============================================================== TMA producer of the V ring
        if (lane == 0) {
            prefetch_tmap(&map_v);
            for (int t = 0; t < len; ++t) {
                const int s = t % C::NV;
                // stage s = t & 1 is free once P V of block t - 2 has completed
                if (t >= C::NV && !mbar_wait(smem_u32(&bars.pv_done[s]), ((t >> 1) - 1) & 1, abortp)) break;
                const int col = __ldg(p.col_idx + ls + t);
                const uint32_t bar = smem_u32(&bars.v_full[s]);
                mbar_arrive_expect_tx(bar, uint32_t(k_rows) * D * 2);
                for (int ch = 0; ch < C::CH; ++ch) {
                    const uint32_t dst = s_base + C::OFF_V + s * C::KV_BYTES + ch * C::KV_CHUNK;
                    if (perm) tma_load_4d(dst, &map_v4, bar, ch * 64, 0, col * p.th.ks, bh);
                    else tma_load_3d(dst, &map_v, bar, ch * 64, col * C::BK, bh);
                }
            }
        }
    } else if (warp == 2) {
        // ============================================================== issuer of S = Q K^T
        // The whole warp walks the loop (every lane polls the barriers) and one elected lane issues: the
        // operands of the products are then warp-uniform values, which is what keeps the cost of issuing
        // a product low (measured: 27 against 45 cycles per instruction when one lane runs the loop alone).
        const uint32_t idesc_qk = make_idesc_bf16(128, C::BK, 0, 0);
        constexpr uint32_t HI = sdesc_hi_sw128(1024);   // the high descriptor word is one constant here
        const uint32_t q_lo = sdesc_lo(s_base + C::OFF_Q, 16);
        const uint32_t k_lo0 = sdesc_lo(s_base + C::OFF_K, 16);
        bool ok = true;
        {
            if (len > 0) ok = wait_warp(&bars.q_full, 0);
            for (int t = 0; t < len && ok; ++t) {
                const int s = t % C::NK;
                ok = wait_warp(&bars.k_full[s], (t / C::NK) & 1);
                // score buffer t & 1 held P of block t - 2: its P V product must have read it
                if (ok && t >= 2) ok = wait_warp(&bars.pv_done[t & 1], ((t >> 1) - 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint32_t kb_lo = k_lo0 + s * (C::KV_CHUNK >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)   // 16 channels: 32 bytes of each Q and K row, chunk k/4
                        mma_ss_lohi(tmem + C::COL_SP + (t & 1) * C::SP_STRIDE,
                                    q_lo + (((k / 4) * C::Q_CHUNK + (k % 4) * 32) >> 4), HI,
                                    kb_lo + (((k / 4) * (C::NK * C::KV_CHUNK) + (k % 4) * 32) >> 4), HI, idesc_qk, k > 0);
                    tc_commit(smem_u32(&bars.s_full[t & 1]));
                }
                __syncwarp();
            }
        }
    } else if (warp == 3) {
        // ============================================================== issuer of O += P V and of the linear numerator
        const uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
        const uint32_t idesc_lin = make_idesc_bf16(128, D, 0, 0);
        constexpr uint32_t HI = sdesc_hi_sw128(1024);
        const uint32_t q_lo = sdesc_lo(s_base + C::OFF_Q, 16);
        const uint32_t v_lo0 = sdesc_lo(s_base + C::OFF_V, C::KV_CHUNK);
        bool ok = true;
        for (int t = 0; t < len && ok; ++t) {
            const int s = t % C::NV;
            ok = wait_warp(&bars.v_full[s], (t / C::NV) & 1);
            if (ok) ok = wait_warp(&bars.p_ready[t & 1], (t >> 1) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t vb_lo = v_lo0 + s * (C::KV_BYTES >> 4);
                const uint32_t p_col = tmem + C::COL_SP + (t & 1) * C::SP_STRIDE;
#pragma unroll
                for (int k = 0; k < C::BK / 16; ++k)      // 16 keys = 16 rows of 128 bytes
                    mma_ts_lohi(tmem + C::COL_O, p_col + k * 8, vb_lo + ((k * 2048) >> 4), HI, idesc_pv,
                                (t > 0 || k > 0) ? 1u : 0u);
                tc_commit(smem_u32(&bars.pv_done[t & 1]));
                if (t + 1 == len) tc_commit(smem_u32(&bars.o_final));
            }
            __syncwarp();
        }
        if (ok && linear) {
            ok = wait_warp(&bars.st_full, 0);
            if (ok) ok = wait_warp(&bars.lin_ready, 0);
            if (ok) {
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint32_t st_lo = sdesc_lo(s_base + C::OFF_ST, 16);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        mma_ss_lohi(tmem, q_lo + (((k / 4) * C::Q_CHUNK + (k % 4) * 32) >> 4), HI,
                                    st_lo + (((k / 4) * C::ST_CHUNK + (k % 4) * 32) >> 4), HI, idesc_lin, k > 0);
                    tc_commit(smem_u32(&bars.lin_done));
                }
                __syncwarp();
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 96;");
        // ============================================================== softmax + epilogue
        // Eight warps.  A warp works on 16 TMEM lanes (query rows) with the 16-lane
        // load/store shapes: four threads share a row, each holding a quarter of its columns,
        // and every thread serves two rows (a and a + 8).  Row maxima and sums are combined
        // with two shuffles inside the group of four.
        const int sw = warp - 4;
        const int q4 = lane & 3;                                // position in the group of four
        const int lane0 = (warp & 3) * 32 + (sw >> 2) * 16;          // first TMEM lane of this warp
        const int ra = lane0 + (lane >> 2), rb = ra + 8;        // the thread's two query rows
        const uint32_t t_tile = tmem + (uint32_t(lane0) << 16);
        const int len = le - ls;
        uint8_t* qtile = smem + C::OFF_Q;
        float m_a = -INFINITY, m_b = -INFINITY;                 // running maxima (log2 domain)
        float l_a = 0.f, l_b = 0.f;                             // this thread's share of the row sums
        bool ok = true;
        // every lane of a warp must take the same path around the warp-collective tcgen05
        // loads/stores, so the outcome of a bounded wait is made warp-uniform
        auto wait_uniform = [&](uint64_t* bar, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(smem_u32(bar), parity, abortp));
        };
        auto quad_max = [](float v) -> float {
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
            return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
        };
        auto quad_sum = [](float v) -> float {
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            return v + __shfl_xor_sync(0xffffffffu, v, 2);
        };

        // Only the last key block of the sequence can be short (N not a multiple of 64), and in an ascending
        // list it can only be the last entry: one look at that entry, before the loop, settles which block
        // needs its missing keys masked.
        // (A temporal head: every block holds ks * T keys, the last one those of the positions that exist.)
        int valid_last = k_rows;
        if (len > 0) {
            if (perm) {
                if (__ldg(p.col_idx + le - 1) == p.th.nKb - 1) valid_last = (p.th.S - (p.th.nKb - 1) * p.th.ks) * p.th.T;
            } else if ((p.N % C::BK) != 0 && __ldg(p.col_idx + le - 1) == p.nKb - 1) {
                valid_last = p.N - (p.nKb - 1) * C::BK;
            }
        }
        for (int t = 0; t < len && ok; ++t) {
            ok = wait_uniform(&bars.s_full[t & 1], (t >> 1) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            // x[4n], x[4n+1] = S(row a, keys 8n + 2 q4, + 1);  x[4n+2], x[4n+3] = the same keys of row b
            uint32_t xr[32];
            tmem_ld_16x256b_x8(t_tile + C::COL_SP + (t & 1) * C::SP_STRIDE, xr);
            tmem_wait_ld();
            float* x = reinterpret_cast<float*>(xr);
            const int valid = (t + 1 == len) ? valid_last : k_rows;      // keys of this block that exist
            if (valid < C::BK) {
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    const int key = 8 * n + 2 * q4;
                    if (key >= valid) { x[4 * n] = -INFINITY; x[4 * n + 2] = -INFINITY; }
                    if (key + 1 >= valid) { x[4 * n + 1] = -INFINITY; x[4 * n + 3] = -INFINITY; }
                }
            }
            // block maxima of the two rows
            float mxa = fmaxf(x[0], x[1]), mxb = fmaxf(x[2], x[3]);
#pragma unroll
            for (int n = 1; n < 8; ++n) {
                mxa = fmaxf(mxa, fmaxf(x[4 * n], x[4 * n + 1]));
                mxb = fmaxf(mxb, fmaxf(x[4 * n + 2], x[4 * n + 3]));
            }
            // The running max only moves when it grows by more than 2^8 (checked on the threads' own
            // columns first: the shuffles that form the row maxima are needed only then).  The accumulator
            // of this warp's rows is then brought to the new max, once the previous P V product has
            // landed in it.  pv_done[b] completes a phase for every second block; the product of block t
            // cannot be issued before this warp hands over P of block t, so the barrier is at most one
            // phase past the one tested here and the parity test is exact.
            if (t == 0) {
                m_a = quad_max(mxa) * p.scale_log2; m_b = quad_max(mxb) * p.scale_log2;
            } else if (__any_sync(0xffffffffu, mxa * p.scale_log2 > m_a + 8.0f || mxb * p.scale_log2 > m_b + 8.0f)) {
                const float msa = quad_max(mxa) * p.scale_log2, msb = quad_max(mxb) * p.scale_log2;
                ok = wait_uniform(&bars.pv_done[(t - 1) & 1], ((t - 1) >> 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                const float na = fmaxf(m_a, msa), nb = fmaxf(m_b, msb);
                const float al_a = ex2_approx(m_a - na), al_b = ex2_approx(m_b - nb);
                l_a *= al_a; l_b *= al_b;
                m_a = na; m_b = nb;
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) {
                    uint32_t orr[16];
                    tmem_ld_16x256b_x4(t_tile + C::COL_O + cc * 32, orr);
                    tmem_wait_ld();
#pragma unroll
                    for (int n = 0; n < 4; ++n) {
                        orr[4 * n] = __float_as_uint(__uint_as_float(orr[4 * n]) * al_a);
                        orr[4 * n + 1] = __float_as_uint(__uint_as_float(orr[4 * n + 1]) * al_a);
                        orr[4 * n + 2] = __float_as_uint(__uint_as_float(orr[4 * n + 2]) * al_b);
                        orr[4 * n + 3] = __float_as_uint(__uint_as_float(orr[4 * n + 3]) * al_b);
                    }
                    tmem_st_16x256b_x4(t_tile + C::COL_O + cc * 32, orr);
                }
                tmem_wait_st();
            }
            // P = exp2(x * scale - m), packed bf16: word 2n = row a, keys (8n + 2 q4, + 1) = packed
            // column 4n + q4 of the P tile, word 2n + 1 the same of row b -- the 16x128b layout
            uint32_t pk[16];
            {
                const uint64_t sc2 = pack_f32x2(p.scale_log2, p.scale_log2);
                const uint64_t nma = pack_f32x2(-m_a, -m_a), nmb = pack_f32x2(-m_b, -m_b);
                uint64_t acc_a = pack_f32x2(0.f, 0.f), acc_b = acc_a;
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    float a0, a1, b0, b1;
                    unpack_f32x2(fma_f32x2(pack_f32x2(x[4 * n], x[4 * n + 1]), sc2, nma), a0, a1);
                    unpack_f32x2(fma_f32x2(pack_f32x2(x[4 * n + 2], x[4 * n + 3]), sc2, nmb), b0, b1);
                    const float pa0 = ex2_approx(a0), pa1 = ex2_approx(a1), pb0 = ex2_approx(b0), pb1 = ex2_approx(b1);
                    acc_a = add_f32x2(acc_a, pack_f32x2(pa0, pa1));
                    acc_b = add_f32x2(acc_b, pack_f32x2(pb0, pb1));
                    pk[2 * n] = pack_bf16x2(pa0, pa1);
                    pk[2 * n + 1] = pack_bf16x2(pb0, pb1);
                }
                float s0, s1;
                unpack_f32x2(acc_a, s0, s1); l_a += s0 + s1;
                unpack_f32x2(acc_b, s0, s1); l_b += s0 + s1;
            }
            // P goes over the scores it was computed from (this warp's own lanes, already in registers)
            tmem_st_16x128b_x8(t_tile + C::COL_SP + (t & 1) * C::SP_STRIDE, pk);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.p_ready[t & 1]));   // one arrival per warp
        }
        float coef_a = 0.f, coef_b = 0.f;
        if (ok && linear) {
            // ReLU of the Q rows in place, and the denominators ReLU(Q_n) . Z: the four threads of a
            // row take two 16-byte groups of every 64 channels each.  Every Q K^T of this tile has
            // completed (its scores were consumed above), so Q is no longer read; the last P V
            // product may still be running meanwhile.
            // Rotary variant (Sec. 4.1): the numerator takes ReLU(Q) rotated pair by pair, the denominator
            // the un-rotated values.  A thread meets CH * 4 vectors of 8 channels; the (cos, sin) values of
            // each (16 bytes of the table, from L2) are fetched two vectors ahead, the first before the waits.
            constexpr int NIT = C::CH * 4;
            const bool rotary = p.rope != nullptr;
            auto rot_ptr = [&](int it) {
                const int row = (it & 1) ? rb : ra;
                const int tok = min(qb * p.Bq + row, p.N - 1);           // rows past the block or N hold zeros
                return reinterpret_cast<const uint4*>(p.rope + size_t(tok) * D + (it >> 2) * 64 +
                                                      (q4 + 4 * ((it >> 1) & 1)) * 8);
            };
            uint4 tw[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                tw[u] = make_uint4(0, 0, 0, 0);
                if (rotary) tw[u] = __ldg(rot_ptr(u));
            }
            ok = wait_uniform(&bars.q_full, 0);
            if (ok) ok = wait_uniform(&bars.z_full, 0);
            if (ok) {
                float den_a = 0.f, den_b = 0.f;
#pragma unroll
                for (int it = 0; it < NIT; ++it) {
                    const int ch = it >> 2, c16 = q4 + 4 * ((it >> 1) & 1), e2 = it & 1;
                    const int row = e2 ? rb : ra;
                    uint4* ptr = reinterpret_cast<uint4*>(qtile + ch * C::Q_CHUNK + row * 128 +
                                                          ((c16 ^ (row & 7)) << 4));
                    uint4 v = *ptr;
                    __nv_bfloat162* hv = reinterpret_cast<__nv_bfloat162*>(&v);
                    const uint4 tv = tw[it & 1];
                    if (rotary && it + 2 < NIT) tw[it & 1] = __ldg(rot_ptr(it + 2));
                    const __half2* th = reinterpret_cast<const __half2*>(&tv);      // (cos, sin) of four pairs
                    float den = 0.f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        hv[e] = __hmax2(hv[e], __float2bfloat162_rn(0.f));
                        const float2 f = __bfloat1622float2(hv[e]);
                        const int a = ch * 64 + c16 * 8 + e * 2;
                        den = fmaf(f.x, z_s[a], den);
                        den = fmaf(f.y, z_s[a + 1], den);
                        if (rotary) {
                            const float2 cs = __half22float2(th[e]);
                            hv[e] = __floats2bfloat162_rn(cs.x * f.x - cs.y * f.y, cs.y * f.x + cs.x * f.y);
                        }
                    }
                    *ptr = v;
                    if (e2) den_b += den; else den_a += den;
                }
                den_a = quad_sum(den_a); den_b = quad_sum(den_b);
                float c_scale = 1.f;
                if (p.static_scale) c_scale *= __ldg(p.static_scale + h);
                if (p.dyn_scale) c_scale *= __ldg(p.dyn_scale + b);
                // a row with ReLU(Q_n) = 0 and eps = 0 is 0/0: defined as 0 (the numerator is 0 as well)
                const float da = den_a + p.eps, db = den_b + p.eps;
                coef_a = da > 0.f ? c_scale / da : 0.f;
                coef_b = db > 0.f ? c_scale / db : 0.f;
                fence_proxy_async_smem();
                mbar_arrive(smem_u32(&bars.lin_ready));
            }
        }
        if (ok && len > 0) {
            ok = wait_uniform(&bars.o_final, 0);
            tc_fence_after_sync();
        }
        if (ok && linear) {
            ok = wait_uniform(&bars.lin_done, 0);
            tc_fence_after_sync();
        }

        if (ok) {
            // O = O_acc / l + coef * num, rounded once to bf16, staged in the Q tile
            const float lt_a = quad_sum(l_a), lt_b = quad_sum(l_b);
            const float inv_a = (len > 0) ? 1.0f / lt_a : 0.f, inv_b = (len > 0) ? 1.0f / lt_b : 0.f;
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t orr[16], nr[16];
                if (len > 0) tmem_ld_16x256b_x4(t_tile + C::COL_O + cc * 32, orr);
                if (linear) tmem_ld_16x256b_x4(t_tile + cc * 32, nr);
                tmem_wait_ld();
#pragma unroll
                for (int n = 0; n < 4; ++n) {
                    float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
                    if (len > 0) {
                        a0 = __uint_as_float(orr[4 * n]) * inv_a;     a1 = __uint_as_float(orr[4 * n + 1]) * inv_a;
                        b0 = __uint_as_float(orr[4 * n + 2]) * inv_b; b1 = __uint_as_float(orr[4 * n + 3]) * inv_b;
                    }
                    if (linear) {
                        a0 = fmaf(coef_a, __uint_as_float(nr[4 * n]), a0);     a1 = fmaf(coef_a, __uint_as_float(nr[4 * n + 1]), a1);
                        b0 = fmaf(coef_b, __uint_as_float(nr[4 * n + 2]), b0); b1 = fmaf(coef_b, __uint_as_float(nr[4 * n + 3]), b1);
                    }
                    const int col16 = cc * 4 + n;                  // 16-byte group (8 columns) within the row
                    const int ch = col16 / 8, c16 = col16 % 8;
                    *reinterpret_cast<uint32_t*>(qtile + ch * C::Q_CHUNK + ra * 128 + ((c16 ^ (ra & 7)) << 4) + q4 * 4) =
                        pack_bf16x2(a0, a1);
                    *reinterpret_cast<uint32_t*>(qtile + ch * C::Q_CHUNK + rb * 128 + ((c16 ^ (rb & 7)) << 4) + q4 * 4) =
                        pack_bf16x2(b0, b1);
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(smem_u32(&bars.out_staged));
            if (ra == 0 && q4 == 0 && mbar_wait(smem_u32(&bars.out_staged), 0, abortp)) {
                for (int ch = 0; ch < C::CH; ++ch) {
                    if (perm) tma_store_4d(&map_o4, s_base + C::OFF_Q + ch * C::Q_CHUNK, ch * 64, 0, qb * p.th.kq, bh);
                    else tma_store_3d(&map_o, s_base + C::OFF_Q + ch * C::Q_CHUNK, ch * 64, qb * p.Bq, bh);
                }
                tma_store_commit();
                // only the shared-memory source must have been read before the CTA may exit; the
                // writes are complete, like all of the kernel's, when the grid is
                tma_store_wait_read_all();
            }
            if (p.lse != nullptr && q4 == 0) {
#pragma unroll
                for (int e2 = 0; e2 < 2; ++e2) {
                    const int row = e2 ? rb : ra;
                    int n = qb * p.Bq + row;
                    if (perm) {                      // row = position within the block * T + frame
                        const int sp = qb * p.th.kq + row / p.th.T;
                        n = (sp < p.th.S) ? (row % p.th.T) * p.th.S + sp : p.N;
                    }
                    if (row < q_rows && n < p.N)
                        p.lse[size_t(bh) * p.N + n] =
                            (len > 0) ? ((e2 ? m_b : m_a) + log2f(e2 ? lt_b : lt_a)) * 0.6931471805599453f : -INFINITY;
                }
            }
        }
    }
    }  // !inherited_abort

    // ------------------------------------------------------------------ tear-down
    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0 && !inherited_abort) {
        // a bounded wait expired somewhere (1: in this CTA, reported here; 2: in the state kernels, which
        // reported it themselves): give copies in flight time to land, leave
        if (tid == 0 && abort_flag == 1) {
            atomicExch(p.ws_status, SALAD_ERR_TIMEOUT);
            if (p.user_status) atomicExch(p.user_status, SALAD_ERR_TIMEOUT);
        }
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) { __nanosleep(1000); }
        __syncthreads();
    }
    if (warp == 2) tmem_dealloc(tmem, C::TMEM_COLS);
}

}  // namespace salad
