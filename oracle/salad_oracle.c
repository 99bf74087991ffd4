/*
 * CPU oracle for the SALAD attention forward pass.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain, slow definition of what the GPU library must compute.  It is
 * called from the tests, from the smoke check and from the CPU-baseline leg of the
 * benchmark, never from the product path, and it shares no code with the CUDA kernels.
 *
 * Everything is evaluated in fp64 on inputs that were already rounded to bf16 and
 * widened to fp32 by the caller, so the oracle and the GPU see identical operands.
 * The only "optimisation" is an OpenMP parallel-for over independent outputs; there is
 * no blocking, no online softmax, no reordering of the sums beyond what the equations
 * themselves state.
 *
 * Layout: Q, K, V are [B, H, N, d] row-major (d fastest).  Tokens of the latent grid
 * are numbered n = (t*Hs + h)*Ws + w, time slowest (Appendix A.1, token flattening).
 *
 * Mask representation: block-granular.  Query block i covers tokens [i*Bq, min(N,(i+1)*Bq)),
 * key block j covers [j*Bk, min(N,(j+1)*Bk)).  A CSR list per (mask head, query block)
 * names the kept key blocks; token pair (n, m) is allowed iff block(m) is in the list of
 * block(n).  This is the matrix M of Eq. 2 with entries 0 on kept blocks, -inf elsewhere.
 *
 * Pins (see tests): dense masked softmax written as an N x N matrix (Eq. 2 literally),
 * the library routine torch SDPA, the un-reordered N x N form of Eq. 3, closed forms
 * (constant V, zero K, homogeneity in K), hand-counted window masks; for the rotary linear branch a
 * two-token example worked by hand, the N x N form with explicit rotation matrices, zero angles
 * (plain Eq. 3), invariance under a common shift of all positions.
 *
 * Every function of this file has at least one such pin; none is left unpinned.  What no pin can
 * settle is whether a READING of the paper is the authors' (the paper prints no worked numeric
 * example and no code): the 3-D window reading of the ST-SWA mask, the per-head scalar reading of the
 * static projection, and the place of the rotary embedding in the linear branch (numerator only), for
 * which the paper has no formula.  Those readings are listed where the build documents its design.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

#ifdef _OPENMP
#include <omp.h>
#endif

/* Threads of the parallel-for loops below: a launcher may have set OMP_NUM_THREADS=1 for the process. */
ORACLE_API void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

ORACLE_API int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int iabs(int x) { return x < 0 ? -x : x; }

/* Does any (query token in block i, key token in block j) pair lie inside the 3-D window?
 * Direct enumeration of all token pairs; the block mask is the "any" over the token mask
 * (static sliding-window mask of Sec. 3 on the un-permuted t,h,w token order). */
static int block_pair_kept(int i, int j, int N, int Hs, int Ws, int Bq, int Bk,
                           int wt, int wh, int ww)
{
    int q0 = i * Bq, q1 = q0 + Bq; if (q1 > N) q1 = N;
    int k0 = j * Bk, k1 = k0 + Bk; if (k1 > N) k1 = N;
    for (int n = q0; n < q1; ++n) {
        int tq = n / (Hs * Ws), hq = (n / Ws) % Hs, wq = n % Ws;
        for (int m = k0; m < k1; ++m) {
            int tk = m / (Hs * Ws), hk = (m / Ws) % Hs, wk = m % Ws;
            if (iabs(tq - tk) <= wt && iabs(hq - hk) <= wh && iabs(wq - wk) <= ww) return 1;
        }
    }
    return 0;
}

/*
 * oracle_mask_build: CSR lists of kept key blocks for a 3-D sliding-window block mask.
 *   windows  [Hm][3] = (wt, wh, ww) per mask head.
 *   row_ptr  [Hm*nQb + 1] out, global offsets; row of (hm, i) is hm*nQb + i.
 *   col_idx  [capacity] out, ascending key-block ids per row; may be NULL to count only.
 * Returns nnz (even when capacity is too small; then col_idx holds only the first
 * `capacity` entries).
 */
ORACLE_API int64_t oracle_mask_build(int T, int Hs, int Ws, int Bq, int Bk, int Hm,
                                     const int32_t* windows, int32_t* row_ptr,
                                     int32_t* col_idx, int64_t capacity)
{
    int N = T * Hs * Ws;
    int nQb = (N + Bq - 1) / Bq, nKb = (N + Bk - 1) / Bk;
    int64_t rows = (int64_t)Hm * nQb;
    unsigned char* keep = (unsigned char*)malloc((size_t)rows * nKb);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
        int hm = (int)(r / nQb), i = (int)(r % nQb);
        for (int j = 0; j < nKb; ++j)
            keep[r * nKb + j] = (unsigned char)block_pair_kept(
                i, j, N, Hs, Ws, Bq, Bk, windows[3 * hm], windows[3 * hm + 1], windows[3 * hm + 2]);
    }
    int64_t nnz = 0;
    for (int64_t r = 0; r < rows; ++r) {
        row_ptr[r] = (int32_t)nnz;
        for (int j = 0; j < nKb; ++j)
            if (keep[r * nKb + j]) {
                if (col_idx && nnz < capacity) col_idx[nnz] = j;
                ++nnz;
            }
    }
    row_ptr[rows] = (int32_t)nnz;
    free(keep);
    return nnz;
}

/* Decode a selected output row.  sel == NULL means "all rows", identity order. */
static void decode_row(const int64_t* sel, int64_t s, int N, int64_t* bh, int* n)
{
    int64_t flat = sel ? sel[s] : s;
    *bh = flat / N;
    *n = (int)(flat % N);
}

/*
 * oracle_sparse_attn: Eq. 2 with the block-granular mask.
 * For each selected query row n of head (b,h):
 *     x_m = scale * <Q_n, K_m>   for every key token m < N in every kept key block
 *     O_s[n] = sum_m softmax(x)_m V_m ,   lse[n] = log sum_m exp(x_m)
 * A row whose list is empty gives O_s = 0 and lse = -inf.
 *   sel   [nsel] flat indices (b*H + h)*N + n, or NULL for all B*H*N rows.
 *   o     [nsel][d] out (fp64).   lse [nsel] out, may be NULL.
 */
ORACLE_API void oracle_sparse_attn(const float* q, const float* k, const float* v,
                                   int B, int H, int N, int d, int Bq, int Bk,
                                   const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                   double scale, const int64_t* sel, int64_t nsel,
                                   double* o, double* lse)
{
    int nQb = (N + Bq - 1) / Bq;
    if (!sel) nsel = (int64_t)B * H * N;
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)N);
        int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
#pragma omp for schedule(dynamic, 16)
        for (int64_t s = 0; s < nsel; ++s) {
            int64_t bh; int n;
            decode_row(sel, s, N, &bh, &n);
            int h = (int)(bh % H);
            /* one mask for all heads (Hm = 1), one per head (Hm = H), or one per batch item
             * and head (Hm = B*H: input-dependent masks such as the Top-K selection) */
            int64_t hm = (Hm == 1) ? 0 : (Hm == H ? h : bh);
            int64_t r = hm * nQb + n / Bq;
            const float* qn = q + (bh * N + n) * (int64_t)d;
            const float* kb = k + bh * (int64_t)N * d;
            const float* vb = v + bh * (int64_t)N * d;
            /* scores over all kept key tokens */
            int64_t cnt = 0;
            double mx = -INFINITY;
            for (int32_t e = row_ptr[r]; e < row_ptr[r + 1]; ++e) {
                int j = col_idx[e];
                int m1 = (j + 1) * Bk; if (m1 > N) m1 = N;
                for (int m = j * Bk; m < m1; ++m) {
                    double acc = 0.0;
                    const float* km = kb + (int64_t)m * d;
                    for (int c = 0; c < d; ++c) acc += (double)qn[c] * (double)km[c];
                    acc *= scale;
                    x[cnt] = acc; idx[cnt] = m; ++cnt;
                    if (acc > mx) mx = acc;
                }
            }
            double* on = o + s * (int64_t)d;
            for (int c = 0; c < d; ++c) on[c] = 0.0;
            if (cnt == 0) { if (lse) lse[s] = -INFINITY; continue; }
            double l = 0.0;
            for (int64_t e = 0; e < cnt; ++e) { x[e] = exp(x[e] - mx); l += x[e]; }
            for (int64_t e = 0; e < cnt; ++e) {
                double p = x[e] / l;
                const float* vm = vb + (int64_t)idx[e] * d;
                for (int c = 0; c < d; ++c) on[c] += p * (double)vm[c];
            }
            if (lse) lse[s] = mx + log(l);
        }
        free(x); free(idx);
    }
}

static double relu(double a) { return a > 0.0 ? a : 0.0; }

/*
 * oracle_linear_state: the two reductions of Eq. 3,
 *     KV[b,h] = sum_j ReLU(K_j)^T V_j   (d x d, row = key channel, column = value channel)
 *     Z[b,h]  = sum_j ReLU(K_j)         (d)
 */
ORACLE_API void oracle_linear_state(const float* k, const float* v, int B, int H, int N, int d,
                                    double* kv, double* z)
{
    int64_t BH = (int64_t)B * H;
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
    for (int64_t bh = 0; bh < BH; ++bh) {
        for (int a = 0; a < d; ++a) {
            const float* kb = k + bh * (int64_t)N * d;
            const float* vb = v + bh * (int64_t)N * d;
            double* row = kv + (bh * d + a) * (int64_t)d;
            for (int c = 0; c < d; ++c) row[c] = 0.0;
            double zs = 0.0;
            for (int j = 0; j < N; ++j) {
                double f = relu((double)kb[(int64_t)j * d + a]);
                zs += f;
                const float* vj = vb + (int64_t)j * d;
                for (int c = 0; c < d; ++c) row[c] += f * (double)vj[c];
            }
            z[bh * d + a] = zs;
        }
    }
}

/*
 * oracle_linear_attn: Eq. 3 for selected rows, from the state,
 *     O_l[n] = ReLU(Q_n) KV / (ReLU(Q_n) . Z + eps).
 * The paper's denominator has no eps; eps only defines the 0/0 case: a row whose ReLU(Q_n) . Z is
 * zero (then the numerator is zero too: Z bounds every column of KV's weights) gives O_l = 0, also
 * with eps = 0, where the quotient would be 0/0.
 */
ORACLE_API void oracle_linear_attn(const float* q, const double* kv, const double* z,
                                   int B, int H, int N, int d, double eps,
                                   const int64_t* sel, int64_t nsel, double* o_l)
{
    if (!sel) nsel = (int64_t)B * H * N;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        int64_t bh; int n;
        decode_row(sel, s, N, &bh, &n);
        const float* qn = q + (bh * N + n) * (int64_t)d;
        const double* kvb = kv + bh * (int64_t)d * d;
        const double* zb = z + bh * (int64_t)d;
        double den = 0.0;
        for (int a = 0; a < d; ++a) den += relu((double)qn[a]) * zb[a];
        double* on = o_l + s * (int64_t)d;
        for (int c = 0; c < d; ++c) {
            double num = 0.0;
            for (int a = 0; a < d; ++a) num += relu((double)qn[a]) * kvb[(int64_t)a * d + c];
            on[c] = (den + eps > 0.0) ? num / (den + eps) : 0.0;   /* 0/0 (eps = 0, ReLU(Q_n) . Z = 0) is taken as 0 */
        }
    }
}

/*
 * oracle_salad_fused: Algorithm 1, residual integration, with the static projection read
 * as one scalar per head (lambda of Eq. 5 folded in) and the dynamic scale s one scalar
 * per batch item:
 *     O[b,h,n] = O_s[b,h,n] + s[b] * lambda[h] * O_l[b,h,n].
 */
ORACLE_API void oracle_salad_fused(const float* q, const float* k, const float* v,
                                   int B, int H, int N, int d, int Bq, int Bk,
                                   const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                   const double* lambda_h, const double* s_b,
                                   double scale, double eps,
                                   const int64_t* sel, int64_t nsel, double* o)
{
    if (!sel) nsel = (int64_t)B * H * N;
    int64_t BH = (int64_t)B * H;
    double* kv = (double*)malloc(sizeof(double) * (size_t)(BH * d * d));
    double* z = (double*)malloc(sizeof(double) * (size_t)(BH * d));
    double* ol = (double*)malloc(sizeof(double) * (size_t)(nsel * d));
    oracle_sparse_attn(q, k, v, B, H, N, d, Bq, Bk, row_ptr, col_idx, Hm, scale, sel, nsel, o, NULL);
    oracle_linear_state(k, v, B, H, N, d, kv, z);
    oracle_linear_attn(q, kv, z, B, H, N, d, eps, sel, nsel, ol);
    for (int64_t s = 0; s < nsel; ++s) {
        int64_t bh; int n;
        decode_row(sel, s, N, &bh, &n);
        double c = s_b[bh / H] * lambda_h[bh % H];
        for (int a = 0; a < d; ++a) o[s * d + a] += c * ol[s * d + a];
    }
    free(kv); free(z); free(ol);
}

/*
 * oracle_dynamic_scale: the input- and timestep-aware scaling factor of Algorithm 1, Level 2,
 *     s[b] = Mean_n sigmoid( <X_t[b,n,:], w> + bias ),
 * one scalar per batch item (a token average of a sigmoid of a D -> 1 linear layer, Sec. 4.2).
 * The paper counts D x 1 weights and does not mention a bias; bias is an argument (0 = none).
 *   x  [B, N, D] (bf16-representable values widened to fp32),  w [D],  s [B] out.
 */
ORACLE_API void oracle_dynamic_scale(const float* x, const float* w, double bias, int B, int N, int D,
                                     double* s)
{
    for (int b = 0; b < B; ++b) {
        double total = 0.0;
#pragma omp parallel for reduction(+ : total) schedule(static)
        for (int n = 0; n < N; ++n) {
            const float* xn = x + ((int64_t)b * N + n) * (int64_t)D;
            double z = bias;
            for (int c = 0; c < D; ++c) z += (double)xn[c] * (double)w[c];
            total += 1.0 / (1.0 + exp(-z));
        }
        s[b] = total / (double)N;
    }
}

/*
 * oracle_salad_fused_drop: Algorithm 1 with post-tuning branch dropping (Sec. 4.3, Appendix
 * A.3): the linear branch of a batch item is skipped when its scaling factor is below the
 * threshold,
 *     O[b,h,n] = O_s[b,h,n] + [s[b] >= tau] * s[b] * lambda[h] * O_l[b,h,n].
 */
ORACLE_API void oracle_salad_fused_drop(const float* q, const float* k, const float* v,
                                        int B, int H, int N, int d, int Bq, int Bk,
                                        const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                        const double* lambda_h, const double* s_b, double tau,
                                        double scale, double eps,
                                        const int64_t* sel, int64_t nsel, double* o)
{
    double* s_eff = (double*)malloc(sizeof(double) * (size_t)B);
    for (int b = 0; b < B; ++b) s_eff[b] = (s_b[b] >= tau) ? s_b[b] : 0.0;
    oracle_salad_fused(q, k, v, B, H, N, d, Bq, Bk, row_ptr, col_idx, Hm, lambda_h, s_eff, scale, eps,
                       sel, nsel, o);
    free(s_eff);
}

/*
 * oracle_topk_mask: the dynamic Top-K block mask (Sec. 3, Appendix A.1), per batch item and head:
 *   Step 1  tokens are partitioned into blocks; the mean of every key block is formed,
 *               kbar_j = mean_{m in key block j} K_m          (the last block may be short);
 *   Step 2  similarity of the queries with the key-block means, top k blocks kept.  The attention
 *           kernel is block-granular on the query side as well, so a query block scores a key
 *           block with the average of its tokens' similarities,
 *               s[i][j] = mean_{n in query block i} <Q_n, kbar_j>  ( = <qbar_i, kbar_j> ),
 *           and keeps the k key blocks with the largest s (a tie goes to the lower block index);
 *   Step 3  is the block-sparse attention itself (oracle_sparse_attn on the lists built here).
 * Every row keeps kk = min(topk, nKb) blocks, so row_ptr[r] = r * kk; col_idx
 * [B*H*nQb][kk] holds each row's blocks in ascending order.  scores (may be NULL) receives
 * s as [B*H][nQb][nKb] for the tests.
 */
ORACLE_API void oracle_topk_mask(const float* q, const float* k, int B, int H, int N, int d,
                                 int Bq, int Bk, int topk, int32_t* col_idx, double* scores)
{
    int nQb = (N + Bq - 1) / Bq, nKb = (N + Bk - 1) / Bk;
    int kk = topk < nKb ? topk : nKb;
    int64_t BH = (int64_t)B * H;
#pragma omp parallel for schedule(static)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const float* qb = q + bh * (int64_t)N * d;
        const float* kb = k + bh * (int64_t)N * d;
        double* kbar = (double*)calloc((size_t)nKb * d, sizeof(double));
        double* s = (double*)malloc(sizeof(double) * (size_t)nKb);
        char* taken = (char*)malloc((size_t)nKb);
        for (int j = 0; j < nKb; ++j) {                                  /* Step 1 */
            int m1 = (j + 1) * Bk; if (m1 > N) m1 = N;
            for (int m = j * Bk; m < m1; ++m)
                for (int c = 0; c < d; ++c) kbar[(int64_t)j * d + c] += (double)kb[(int64_t)m * d + c];
            for (int c = 0; c < d; ++c) kbar[(int64_t)j * d + c] /= (double)(m1 - j * Bk);
        }
        for (int i = 0; i < nQb; ++i) {                                  /* Step 2 */
            int n1 = (i + 1) * Bq; if (n1 > N) n1 = N;
            for (int j = 0; j < nKb; ++j) {
                double acc = 0.0;
                for (int n = i * Bq; n < n1; ++n) {
                    double dot = 0.0;
                    for (int c = 0; c < d; ++c) dot += (double)qb[(int64_t)n * d + c] * kbar[(int64_t)j * d + c];
                    acc += dot;
                }
                s[j] = acc / (double)(n1 - i * Bq);
                if (scores) scores[(bh * nQb + i) * (int64_t)nKb + j] = s[j];
            }
            memset(taken, 0, (size_t)nKb);
            for (int t = 0; t < kk; ++t) {                               /* k times: the largest left */
                int best = -1;
                for (int j = 0; j < nKb; ++j)
                    if (!taken[j] && (best < 0 || s[j] > s[best])) best = j;
                taken[best] = 1;
            }
            int32_t* out = col_idx + (bh * nQb + i) * (int64_t)kk;
            int w = 0;
            for (int j = 0; j < nKb; ++j) if (taken[j]) out[w++] = j;    /* ascending */
        }
        free(kbar); free(s); free(taken);
    }
}

/*
 * oracle_proj_combine: Algorithm 1, Level 1 and the residual integration, with the full projection:
 *     O'_l = Proj(O_l)        a linear layer on the head-concatenated linear-branch output
 *                             (D = H*d channels in, D out; zero-initialised before tuning, Sec. 4.2),
 *     O~   = O_s + s * O'_l   (s the dynamic scale of the batch item; Eq. 5's lambda is a further
 *                             scalar on the same term and can be folded into s).
 * Layouts: o_s, o_l, out [B, H, N, d]; channel j = h*d + c of the concatenation.
 *   w     [D][D], w[j_out][j_in]      (y = x W^T, the usual linear-layer storage)
 *   bias  [D] or NULL
 *   s_b   [B]
 */
ORACLE_API void oracle_proj_combine(const float* o_s, const float* o_l, const float* w, const float* bias,
                                    const double* s_b, int B, int H, int N, int d, double* out)
{
    int D = H * d;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int n = 0; n < N; ++n) {
            for (int jo = 0; jo < D; ++jo) {
                double acc = bias ? (double)bias[jo] : 0.0;
                for (int h = 0; h < H; ++h) {
                    const float* x = o_l + (((int64_t)b * H + h) * N + n) * (int64_t)d;
                    const float* wr = w + (int64_t)jo * D + (int64_t)h * d;
                    for (int c = 0; c < d; ++c) acc += (double)x[c] * (double)wr[c];
                }
                int64_t idx = (((int64_t)b * H + jo / d) * N + n) * (int64_t)d + jo % d;
                out[idx] = (double)o_s[idx] + s_b[b] * acc;
            }
        }
    }
}

/*
 * oracle_salad_fused_blockproj: Algorithm 1 with a block-diagonal Level-1 projection (Sec. 4.2): the
 * projection layer of the linear branch restricted to one d x d block per head, no mixing between heads,
 *     O'_l[b,h,n,:] = W_h O_l[b,h,n,:]         (W_h[c_out][a_in], the diagonal block h of Proj's weight)
 *     O~[b,h,n,:]   = O_s[b,h,n,:] + [s_b >= tau] * s_b * O'_l[b,h,n,:].
 * W_h = lambda_h I gives oracle_salad_fused; a full weight matrix that is zero off the diagonal blocks
 * gives oracle_proj_combine.
 *   w_blocks [H][d][d]
 */
ORACLE_API void oracle_salad_fused_blockproj(const float* q, const float* k, const float* v,
                                             int B, int H, int N, int d, int Bq, int Bk,
                                             const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                             const float* w_blocks, const double* s_b, double tau,
                                             double scale, double eps,
                                             const int64_t* sel, int64_t nsel, double* o)
{
    if (!sel) nsel = (int64_t)B * H * N;
    int64_t BH = (int64_t)B * H;
    double* kv = (double*)malloc(sizeof(double) * (size_t)(BH * d * d));
    double* z = (double*)malloc(sizeof(double) * (size_t)(BH * d));
    double* ol = (double*)malloc(sizeof(double) * (size_t)(nsel * d));
    oracle_sparse_attn(q, k, v, B, H, N, d, Bq, Bk, row_ptr, col_idx, Hm, scale, sel, nsel, o, NULL);
    oracle_linear_state(k, v, B, H, N, d, kv, z);
    oracle_linear_attn(q, kv, z, B, H, N, d, eps, sel, nsel, ol);
    for (int64_t s = 0; s < nsel; ++s) {
        int64_t bh; int n;
        decode_row(sel, s, N, &bh, &n);
        double sb = s_b[bh / H];
        if (!(sb >= tau)) continue;                      /* dropped branch: the sparse output alone */
        const float* wh = w_blocks + (bh % H) * (int64_t)d * d;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int a = 0; a < d; ++a) acc += (double)wh[(int64_t)c * d + a] * ol[s * d + a];
            o[s * d + c] += sb * acc;
        }
    }
    free(kv); free(z); free(ol);
}

/*
 * Linear branch with rotary position embedding.  Sec. 4.1 states that the linear branch carries a
 * 3-D rotary embedding and gives no formula; the form taken here is the one the rotary-embedding
 * paper it cites defines for linear attention: the rotation enters the numerator only,
 *     O_l[n] = sum_j < R_n ReLU(Q_n), R_j ReLU(K_j) > V_j  /  ( sum_j < ReLU(Q_n), ReLU(K_j) > + eps ),
 * so that the normaliser keeps its sign.  R_n rotates the channel pair (2i, 2i+1) of token n by an
 * angle given through its cosine and sine, rope[n][i][0] and rope[n][i][1] (fp32, an input: for a 3-D
 * embedding the pairs are shared out among the t, h and w axes of the latent grid).
 *
 * rotate_pairs:  y[2i] = c x[2i] - s x[2i+1],   y[2i+1] = s x[2i] + c x[2i+1].
 */
static void rotate_pairs(const double* x, const float* cs, int d, double* y)
{
    for (int i = 0; i < d / 2; ++i) {
        double c = (double)cs[2 * i], s = (double)cs[2 * i + 1];
        y[2 * i] = c * x[2 * i] - s * x[2 * i + 1];
        y[2 * i + 1] = s * x[2 * i] + c * x[2 * i + 1];
    }
}

/*
 * oracle_linear_state_rope: the two reductions of Eq. 3 with rotated keys in the first,
 *     KV[b,h] = sum_j (R_j ReLU(K_j))^T V_j,     Z[b,h] = sum_j ReLU(K_j)   (not rotated).
 */
ORACLE_API void oracle_linear_state_rope(const float* k, const float* v, const float* rope,
                                         int B, int H, int N, int d, double* kv, double* z)
{
    int64_t BH = (int64_t)B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < BH; ++bh) {
        const float* kb = k + bh * (int64_t)N * d;
        const float* vb = v + bh * (int64_t)N * d;
        double* kvb = kv + bh * (int64_t)d * d;
        double* zb = z + bh * (int64_t)d;
        double* f = (double*)malloc(sizeof(double) * (size_t)d);
        double* fr = (double*)malloc(sizeof(double) * (size_t)d);
        for (int64_t i = 0; i < (int64_t)d * d; ++i) kvb[i] = 0.0;
        for (int a = 0; a < d; ++a) zb[a] = 0.0;
        for (int j = 0; j < N; ++j) {
            for (int a = 0; a < d; ++a) f[a] = relu((double)kb[(int64_t)j * d + a]);
            rotate_pairs(f, rope + (int64_t)j * d, d, fr);
            const float* vj = vb + (int64_t)j * d;
            for (int a = 0; a < d; ++a) {
                zb[a] += f[a];
                for (int c = 0; c < d; ++c) kvb[(int64_t)a * d + c] += fr[a] * (double)vj[c];
            }
        }
        free(f); free(fr);
    }
}

/*
 * oracle_linear_attn_rope: for selected rows, from that state,
 *     O_l[n] = (R_n ReLU(Q_n)) KV / (ReLU(Q_n) . Z + eps).
 */
ORACLE_API void oracle_linear_attn_rope(const float* q, const float* rope, const double* kv, const double* z,
                                        int B, int H, int N, int d, double eps,
                                        const int64_t* sel, int64_t nsel, double* o_l)
{
    if (!sel) nsel = (int64_t)B * H * N;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s) {
        int64_t bh; int n;
        decode_row(sel, s, N, &bh, &n);
        const float* qn = q + (bh * N + n) * (int64_t)d;
        const double* kvb = kv + bh * (int64_t)d * d;
        const double* zb = z + bh * (int64_t)d;
        double* f = (double*)malloc(sizeof(double) * (size_t)d);
        double* fr = (double*)malloc(sizeof(double) * (size_t)d);
        double den = 0.0;
        for (int a = 0; a < d; ++a) { f[a] = relu((double)qn[a]); den += f[a] * zb[a]; }
        rotate_pairs(f, rope + (int64_t)n * d, d, fr);
        double* on = o_l + s * (int64_t)d;
        for (int c = 0; c < d; ++c) {
            double num = 0.0;
            for (int a = 0; a < d; ++a) num += fr[a] * kvb[(int64_t)a * d + c];
            on[c] = (den + eps > 0.0) ? num / (den + eps) : 0.0;   /* 0/0 (eps = 0, ReLU(Q_n) . Z = 0) is taken as 0 */
        }
        free(f); free(fr);
    }
}

/*
 * oracle_salad_fused_rope: Algorithm 1 with that linear branch and the drop threshold of Sec. 4.3,
 *     O[b,h,n] = O_s[b,h,n] + [s[b] >= tau] * s[b] * lambda[h] * O_l[b,h,n]      (tau = -inf: never dropped).
 */
ORACLE_API void oracle_salad_fused_rope(const float* q, const float* k, const float* v, const float* rope,
                                        int B, int H, int N, int d, int Bq, int Bk,
                                        const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                        const double* lambda_h, const double* s_b, double tau,
                                        double scale, double eps,
                                        const int64_t* sel, int64_t nsel, double* o)
{
    if (!sel) nsel = (int64_t)B * H * N;
    int64_t BH = (int64_t)B * H;
    double* kv = (double*)malloc(sizeof(double) * (size_t)(BH * d * d));
    double* z = (double*)malloc(sizeof(double) * (size_t)(BH * d));
    double* ol = (double*)malloc(sizeof(double) * (size_t)(nsel * d));
    oracle_sparse_attn(q, k, v, B, H, N, d, Bq, Bk, row_ptr, col_idx, Hm, scale, sel, nsel, o, NULL);
    oracle_linear_state_rope(k, v, rope, B, H, N, d, kv, z);
    oracle_linear_attn_rope(q, rope, kv, z, B, H, N, d, eps, sel, nsel, ol);
    for (int64_t s = 0; s < nsel; ++s) {
        int64_t bh; int n;
        decode_row(sel, s, N, &bh, &n);
        double sb = s_b[bh / H];
        double c = (sb >= tau) ? sb * lambda_h[bh % H] : 0.0;
        for (int a = 0; a < d; ++a) o[s * d + a] += c * ol[s * d + a];
    }
    free(kv); free(z); free(ol);
}
