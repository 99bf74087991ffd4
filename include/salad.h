/*
 * libsalad -- SALAD sparse-linear attention forward for NVIDIA B200 (sm_100a).
 *
 * The library computes the attention core of Algorithm 1 ("SALAD Attention with
 * Multi-level Scaling"):
 *
 *     O_s = SparseAttn(Q, K, V)                 Eq. 2, block-granular mask
 *     O_l = LinearAttn(Q, K, V)                 Eq. 3, ReLU feature map
 *     O   = O_s + s_b * lambda_h * O_l          Alg. 1 residual integration, Eq. 5
 *
 * Conventions shared by every entry point
 *   - Q, K, V, O are bf16 tensors [B, H, N, d], contiguous, d fastest, base address 16-byte
 *     aligned.  Tokens are the row-major flattening of a T x Hs x Ws latent grid, time
 *     slowest (Appendix A.1).  N need not be a multiple of the block sizes: the last blocks
 *     are short, keys >= N take no part, queries >= N are never written.
 *   - The sparsity mask is block granular: query block i covers tokens [i*Bq, (i+1)*Bq),
 *     key block j covers [j*Bk, (j+1)*Bk).  It is passed as CSR lists: row r = hm*nQb + i
 *     (nQb = ceil(N/Bq)) owns col_idx[row_ptr[r] .. row_ptr[r+1]), the kept key blocks,
 *     ascending and unique, each in [0, ceil(N/Bk)).  Hm is 1 (one mask for all heads), H
 *     (one per head, shared by the batch items; hm = h) or B*H (one per batch item and head,
 *     hm = b*H + h: input-dependent masks such as salad_topk_mask_build's).  An empty row is
 *     legal: its O_s is zero.
 *   - Every pointer is DEVICE memory owned by the caller unless its name starts with h_
 *     (host).  Nothing is allocated or freed by the library; scratch comes from a caller
 *     workspace of at least salad_workspace_bytes() bytes, 256-byte aligned, which must
 *     not be shared by calls that may overlap on the GPU.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work is enqueued
 *     asynchronously on it; only salad_mask_build synchronises (to return nnz).
 *   - Return value: SALAD_OK or a negative code.  Argument errors are detected on the host
 *     before anything is launched.  There is no CPU fallback: without a usable CUDA device
 *     the compute entry points return SALAD_ERR_CUDA.
 *   - d_status (optional, device int32): set to 0 by a successful launch and to a non-zero
 *     code by a kernel whose bounded internal wait expired (SALAD_ERR_TIMEOUT; the kernel then
 *     returns early instead of hanging) or by the mask checks (SALAD_ERR_BAD_MASK, below); the
 *     remaining kernels of the call then return at once and the outputs are undefined.  Read it
 *     after synchronising the stream.
 *   - Mask checks.  The lists are device data, so the host cannot check them before the launch.
 *     Every call with a sparse branch checks, in its first kernel, that the row offsets are
 *     non-negative and non-decreasing (it reads them anyway).  The full contract (offsets
 *     start at 0 and end within col_idx, block ids strictly ascending and in range) is checked
 *     by salad_csr_validate, on request; salad_set_mask_validation makes the attention entry
 *     points run it first.  Without that opt-in, offsets that point past the end of col_idx
 *     make the attention kernel read outside the caller's array.
 *   - SALAD_LOG=1 in the environment prints one line per kernel launch on stderr.
 *   - Supported shapes: d in {64, 128}; Bq in {64, 128}; Bk = 64; softmax_scale > 0.
 */
#ifndef SALAD_H_
#define SALAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SALAD_OK 0
#define SALAD_ERR_INVALID_ARG (-1) /* null pointer, non-positive size, bad Hm, misalignment  */
#define SALAD_ERR_UNSUPPORTED (-2) /* d, Bq or Bk outside the supported set                  */
#define SALAD_ERR_WORKSPACE (-3)   /* workspace missing, misaligned or too small             */
#define SALAD_ERR_CAPACITY (-4)    /* col_idx capacity smaller than nnz (nnz still returned) */
#define SALAD_ERR_CUDA (-5)        /* a CUDA runtime/driver call or a launch failed          */
#define SALAD_ERR_TIMEOUT (-6)     /* value written to d_status by a kernel that gave up     */
#define SALAD_ERR_BAD_MASK (-7)    /* value written to d_status: the CSR lists break the contract */

/* Human-readable name of a status code (static string, never NULL). */
const char* salad_status_string(int status);

/* Bytes of workspace the *_fwd calls need for this problem size (0 if the shape is
 * unsupported).  Depends only on the arguments, never on the device. */
size_t salad_workspace_bytes(int B, int H, int N, int d, int Bq, int Bk);

/*
 * salad_mask_build -- static spatio-temporal sliding-window block mask (Sec. 3 "static
 * sparse attention", Appendix A.1), 3-D window form on the un-permuted t,h,w token order.
 * Key block j is kept for query block i of mask head hm iff some query token (t,h,w) of
 * block i and some key token (t',h',w') of block j satisfy |t-t'| <= wt, |h-h'| <= wh,
 * |w-w'| <= ww with (wt,wh,ww) = h_windows[hm].
 *   T, Hs, Ws      latent grid; N = T*Hs*Ws.
 *   Bq, Bk         block sizes (any positive values).
 *   Hm             number of mask heads; h_windows is a HOST array [Hm][3].
 *   d_row_ptr      device int32 [Hm*nQb + 1], written.
 *   d_col_idx      device int32 [col_capacity], written ascending per row; may be NULL with
 *                  col_capacity 0 to obtain only row_ptr and nnz.
 *   h_nnz          HOST int64, written with the total number of kept blocks (optional).
 * Synchronises `stream` (once to return nnz, once more after the fill when d_col_idx is given; the
 * count pass runs in both of the usual two calls, "size, then fill": the mask is built once per
 * model, so this costs a fraction of a millisecond in total).  Returns SALAD_ERR_CAPACITY (row_ptr and *h_nnz valid, col_idx
 * untouched) if col_capacity < nnz and d_col_idx != NULL.
 */
int salad_mask_build(int T, int Hs, int Ws, int Bq, int Bk, int Hm, const int32_t* h_windows,
                     int32_t* d_row_ptr, int32_t* d_col_idx, int64_t col_capacity,
                     int64_t* h_nnz, void* stream);

/*
 * salad_csr_validate -- checks block lists against the contract above (the mask M of Eq. 2 in its
 * block-granular CSR form):  row_ptr[0] == 0;  row_ptr non-decreasing;  row_ptr[rows] <=
 * col_capacity;  inside every row the block ids strictly ascending (sorted, unique) and in [0, nKb).
 *   row_ptr        device int32 [rows + 1];   col_idx  device int32 [col_capacity] (may be NULL
 *                  with capacity 0);   rows = Hm * nQb;   nKb = ceil(N / Bk).
 *   d_status       device int32, required: 0 if the lists are valid, SALAD_ERR_BAD_MASK if not.
 * Reads nothing outside row_ptr[0..rows] and col_idx[0..col_capacity), whatever the lists hold, so
 * it is safe on corrupted input.  Asynchronous on `stream` (a memset and one small kernel).
 *
 * salad_set_mask_validation -- col_capacity > 0: every later call of salad_sparse_attn_fwd and the
 * salad_fused_* entry points made by this host thread first runs the check above on its lists, with
 * col_idx holding col_capacity entries; a failure is reported as SALAD_ERR_BAD_MASK in d_status,
 * and the attention kernels of that call do nothing.  0 switches it off (the default).  A debugging
 * aid: it adds a memset and a kernel to every call.
 */
int salad_csr_validate(const int32_t* row_ptr, const int32_t* col_idx, int64_t col_capacity,
                       int64_t rows, int nKb, int32_t* d_status, void* stream);
int salad_set_mask_validation(int64_t col_capacity);

/*
 * salad_sparse_attn_fwd -- block-sparse softmax attention, Eq. 2:
 *     O_s[n] = sum_m softmax_m(softmax_scale * <Q_n, K_m>) V_m   over keys m of kept blocks.
 *   o              bf16 [B,H,N,d], written.
 *   lse            optional fp32 [B,H,N]: log-sum-exp (natural log) of the scaled scores of
 *                  each row; -inf for rows with an empty list.
 *   softmax_scale  0 selects 1/sqrt(d).
 */
int salad_sparse_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                          int B, int H, int N, int d, int Bq, int Bk,
                          const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                          float softmax_scale, void* workspace, size_t workspace_bytes,
                          int32_t* d_status, void* stream);

/*
 * salad_linear_attn_fwd -- ReLU linear attention, Eq. 3:
 *     KV = sum_j ReLU(K_j)^T V_j  (d x d),   Z = sum_j ReLU(K_j)  (d),
 *     O_l[n] = ReLU(Q_n) KV / (ReLU(Q_n) . Z + eps).
 *   o_l            bf16 [B,H,N,d], written.
 *   kv_out         optional fp32 [B,H,d,d] (row = key channel, column = value channel).
 *   z_out          optional fp32 [B,H,d].
 *   eps            >= 0; only defines the 0/0 case: a row with ReLU(Q_n) = 0 gives 0, also
 *                  with eps = 0 (the quotient 0/0 is taken as 0, never NaN).
 */
int salad_linear_attn_fwd(const void* q, const void* k, const void* v, void* o_l,
                          float* kv_out, float* z_out, int B, int H, int N, int d, float eps,
                          void* workspace, size_t workspace_bytes, int32_t* d_status,
                          void* stream);

/*
 * salad_fused_fwd -- both branches and the scaled residual sum of Algorithm 1 with a single
 * bf16 write of O:
 *     O[b,h,n] = O_s[b,h,n] + d_dyn_scale[b] * d_static_scale[h] * O_l[b,h,n].
 *   d_static_scale fp32 [H]: the layer-wise static scaling read as one scalar per head
 *                  (block-diagonal projection; lambda of Eq. 5 multiplied in by the caller).
 *   d_dyn_scale    fp32 [B]: the input- and timestep-aware factor s of Alg. 1, produced
 *                  upstream on the device; any finite value is accepted.
 * A zero product of the scales reproduces salad_sparse_attn_fwd bit for bit.
 */
int salad_fused_fwd(const void* q, const void* k, const void* v, void* o,
                    int B, int H, int N, int d, int Bq, int Bk,
                    const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                    const float* d_static_scale, const float* d_dyn_scale,
                    float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                    int32_t* d_status, void* stream);

/*
 * salad_fused_drop_fwd -- salad_fused_fwd with post-tuning branch dropping (Sec. 4.3, Appendix
 * A.3): the linear branch of batch item b is skipped when its scaling factor is below the
 * threshold,
 *     O[b,h,n] = O_s[b,h,n] + [d_dyn_scale[b] >= drop_tau] * d_dyn_scale[b] * d_static_scale[h] * O_l[b,h,n].
 * The comparison happens on the device (the scale is produced there), so there is no host
 * synchronisation: the linear-state kernels of a dropped batch item return at once and the
 * attention kernel does no linear work for it; its output equals salad_sparse_attn_fwd bit
 * for bit.  drop_tau is the calibrated per-timestep threshold tau_t (a host float).
 */
int salad_fused_drop_fwd(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int N, int d, int Bq, int Bk,
                         const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                         const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                         float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                         int32_t* d_status, void* stream);

/*
 * salad_linear_state_fwd / salad_fused_prepared_fwd -- salad_fused_drop_fwd in two calls, for callers who
 * have K and V before Q (or a free stream): the two reductions of Eq. 3,
 *     KV = sum_j ReLU(K_j)^T V_j ,   Z = sum_j ReLU(K_j) ,
 * are one pass over K and V that needs nothing else, so it can run early or beside other work; the
 * attention call then finds the state in the workspace and runs without the reduction kernels.
 *   salad_linear_state_fwd(k, v, ...)     leaves the state in `workspace`; kv_out (fp32 [B,H,d,d]) and
 *                                         z_out (fp32 [B,H,d]) receive copies when not NULL.
 *   salad_fused_prepared_fwd(q, k, v, ..) arguments as salad_fused_drop_fwd; `workspace` must be the one a
 *                                         completed salad_linear_state_fwd call on the same K, V, B, H, N, d
 *                                         wrote (order the two calls with the stream or an event).  The result
 *                                         equals salad_fused_drop_fwd bit for bit.
 * Branch dropping happens in the second call (the state is computed for every batch item).
 */
int salad_linear_state_fwd(const void* k, const void* v, float* kv_out, float* z_out, int B, int H, int N, int d,
                           void* workspace, size_t workspace_bytes, int32_t* d_status, void* stream);
int salad_fused_prepared_fwd(const void* q, const void* k, const void* v, void* o,
                             int B, int H, int N, int d, int Bq, int Bk,
                             const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                             const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                             float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                             int32_t* d_status, void* stream);

/*
 * salad_fused_proj_fwd -- salad_fused_drop_fwd with a block-diagonal Level-1 projection (Algorithm 1,
 * "Level 1: layer-wise static scaling"; Sec. 4.2, the zero-initialised projection of the linear branch)
 * in place of the per-head scalar: one d x d block per head, no mixing between heads,
 *     O[b,h,n,:] = O_s[b,h,n,:] + [d_dyn_scale[b] >= drop_tau] * d_dyn_scale[b] * W_h O_l[b,h,n,:].
 * The block folds into the linear state, W_h (ReLU(Q_n) KV)^T = (KV W_h^T)^T ReLU(Q_n)^T: the state of
 * every head is multiplied with its block once (a d x d x d product in fp32, rounded once to bf16) and
 * the attention kernel runs unchanged, so the call still reads Q, K, V once and writes O once.  The
 * normaliser Z is applied before the projection, as in Algorithm 1.
 *   d_proj_blocks  device bf16 [H, d, d], 16-byte aligned: W_h[c_out][a_in], i.e. the diagonal blocks of
 *                  the weight matrix salad_proj_combine_fwd takes; lambda of Eq. 5 multiplied in by the
 *                  caller.  W_h = lambda_h I reproduces salad_fused_fwd; zero blocks (the layer before
 *                  tuning) reproduce salad_sparse_attn_fwd.
 *   drop_tau       -INFINITY: no branch is dropped.
 * A projection that mixes heads cannot be folded in this way: see salad_proj_combine_fwd.
 */
int salad_fused_proj_fwd(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int N, int d, int Bq, int Bk,
                         const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                         const void* d_proj_blocks, const float* d_dyn_scale, float drop_tau,
                         float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                         int32_t* d_status, void* stream);

/*
 * salad_fused_rope_fwd / salad_linear_attn_rope_fwd -- the same two calls with a rotary position
 * embedding in the linear branch (Sec. 4.1 states that the linear branch carries a 3-D rotary embedding
 * and gives no formula; the rotation enters the numerator only, as the rotary-embedding paper it cites
 * defines for linear attention, so the normaliser keeps its sign):
 *     O_l[n] = sum_j < R_n ReLU(Q_n), R_j ReLU(K_j) > V_j / ( sum_j < ReLU(Q_n), ReLU(K_j) > + eps ),
 * R_n rotating the channel pair (2i, 2i+1) of token n:  y[2i] = c x[2i] - s x[2i+1],  y[2i+1] = s x[2i] + c x[2i+1].
 *   d_rope  device fp16 (IEEE half) [N, d/2, 2], 16-byte aligned: (c, s) = cosine and sine of the angle of
 *           token n and pair i; shared by every batch item and head; read-only; a 3-D embedding shares the
 *           pairs out among the t, h, w axes of the latent grid (the caller's table decides).  Half precision
 *           (11 significant bits for values in [-1, 1]) halves the traffic of the table, which every tile
 *           of every head re-reads from L2; it is finer than the bf16 activations it multiplies.
 * The rotation is applied in fp32 to the bf16 ReLU values and rounded to bf16 for the tensor cores; the
 * state KV = sum_j (R_j ReLU(K_j))^T V_j is what kv_out receives, Z stays the plain sum.
 * salad_fused_rope_fwd takes drop_tau like salad_fused_drop_fwd (-INFINITY: no branch is dropped).
 * Errors as for the calls without the table; a null d_rope is SALAD_ERR_INVALID_ARG.
 */
int salad_fused_rope_fwd(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int N, int d, int Bq, int Bk,
                         const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                         const float* d_static_scale, const float* d_dyn_scale, const void* d_rope,
                         float drop_tau, float softmax_scale, float eps, void* workspace,
                         size_t workspace_bytes, int32_t* d_status, void* stream);

int salad_linear_attn_rope_fwd(const void* q, const void* k, const void* v, void* o_l,
                               float* kv_out, float* z_out, int B, int H, int N, int d,
                               const void* d_rope, float eps, void* workspace, size_t workspace_bytes,
                               int32_t* d_status, void* stream);

/*
 * salad_rope3d_table_build -- the rotation table of a 3-D rotary position embedding for the tokens of a
 * T x Hs x Ws latent grid, n = (t*Hs + h)*Ws + w (Sec. 4.1 says the embedding is 3-D and gives no layout;
 * this one follows video DiTs of the Wan family).  The d/2 channel pairs are shared out among the axes:
 * floor(d/6) pairs each for h and w (in that order, after the t pairs), the rest for t; pair j of an axis
 * with P pairs turns by  position * base^(-j / P).
 *   d_rope  out, device fp16 [T*Hs*Ws, d/2, 2] = (cos, sin), 16-byte aligned, caller-owned; the table
 *           argument of the two calls above.  Built once per grid; angles in double precision, so every
 *           entry is the correctly rounded fp16 value.
 * base > 1 (10000 is customary); d even.  Errors: SALAD_ERR_INVALID_ARG, SALAD_ERR_UNSUPPORTED (more
 * than 2^31 - 1 tokens), SALAD_ERR_CUDA.  Asynchronous on `stream`.
 */
int salad_rope3d_table_build(int T, int Hs, int Ws, int d, float base, void* d_rope, void* stream);

/*
 * salad_dynamic_scale -- the input- and timestep-aware scaling factor of Algorithm 1, Level 2
 * (Sec. 4.2): a D -> 1 linear layer on the modulated hidden states, a sigmoid, a token average:
 *     s[b] = (1/N) sum_n sigmoid( <x[b,n,:], w> + bias ),   s in (0, 1).
 *   x          bf16 [B, N, D], contiguous, 16-byte aligned; D a multiple of 8, D <= 8192.
 *   w          fp32 [D] (device).   bias: the paper counts D x 1 weights only; pass 0 for none.
 *   s_out      fp32 [B] (device), written; it can be passed on as d_dyn_scale.
 *   workspace  at least SALAD_DYN_SCALE_WS_BYTES bytes of device memory, 256-byte aligned.
 * HBM-bound (x is read once); the result is deterministic.  B <= 2048.
 */
#define SALAD_DYN_SCALE_WS_BYTES 8192
int salad_dynamic_scale(const void* x, const float* w, float bias, int B, int N, int D,
                        float* s_out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * salad_topk_mask_build -- the dynamic Top-K block mask (Sec. 3; Appendix A.1, Steps 1-2), as
 * CSR lists for the attention entry points (Hm = B*H).  Per batch item and head:
 *     kbar_j = mean of the key tokens of block j,   qbar_i = mean of the query tokens of block i,
 *     s[i][j] = <qbar_i, kbar_j>   (= the block's average of its tokens' similarity with kbar_j),
 *     row i keeps the kk = min(topk, nKb) key blocks with the largest s, a tie going to the
 *     lower block index; the kept blocks are written in ascending order.
 * Arithmetic: fp32 sums and FMAs in a fixed order (deterministic).  Scores are assumed finite.
 *   q, k           bf16 [B, H, N, d], d in {64, 128}; Bq, Bk <= 1024.
 *   d_row_ptr      device int32 [B*H*nQb + 1], written (row r starts at r*kk).
 *   d_col_idx      device int32, capacity col_capacity entries; B*H*nQb*kk are written,
 *                  SALAD_ERR_CAPACITY if it is smaller (nothing is launched).
 *   workspace      at least salad_topk_workspace_bytes() bytes, 256-byte aligned (block means and
 *                  the B*H*nQb*nKb scores).
 * Asynchronous on `stream`; no host synchronisation (the list sizes are known in advance).
 */
size_t salad_topk_workspace_bytes(int B, int H, int N, int d, int Bq, int Bk);
int salad_topk_mask_build(const void* q, const void* k, int B, int H, int N, int d, int Bq, int Bk,
                          int topk, int32_t* d_row_ptr, int32_t* d_col_idx, int64_t col_capacity,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * salad_permute_tokens -- the token re-ordering of Appendix A.1 for heads with temporal locality.
 * Tokens arrive flattened with time slowest, n = t*(Hs*Ws) + s; a flagged head is re-ordered to
 * m = s*T + t (tokens grouped by spatial location, temporal neighbours adjacent), so that a 1-D
 * sliding-window mask (salad_mask_build on the grid 1 x 1 x N) captures temporal locality:
 *     inverse == 0:  y[b,h,m,:] = x[b,h,n,:]        inverse != 0:  y[b,h,n,:] = x[b,h,m,:]
 * Heads whose flag is 0 are copied unchanged.  Use: permute Q, K, V, run an attention entry
 * point with per-head 1-D windows, permute O back with inverse = 1.
 *   x, y           bf16 [B, H, N, d], N == T*Hs*Ws, d in {64, 128}; y must not alias x.
 *   h_head_flags   HOST int32 [H]; H <= 1024.
 * HBM-bound (one read and one write of the tensor); asynchronous on `stream`.
 */
int salad_permute_tokens(const void* x, void* y, int B, int H, int N, int d, int T, int Hs, int Ws,
                         const int32_t* h_head_flags, int inverse, void* stream);

/*
 * salad_fused_stswa_fwd -- the paper's own ST-SWA (Appendix A.1) in one call, without re-ordering passes:
 * every head gets a 1-D sliding-window mask on ITS token order, which for heads with temporal locality
 * (h_head_flags[h] != 0) is the order that groups tokens by spatial position, m = s*T + t for token
 * n = t*(Hs*Ws) + s.  Such a head reads Q, K, V and writes O through 4-D tensor maps over the unchanged
 * [B,H,N,d] tensors, in which the T tokens of a spatial position are one box row; nothing is permuted in
 * memory, and the output arrives in the original token order.  Both branches are equivariant under the
 * re-ordering, so the result equals salad_permute_tokens -> salad_fused_drop_fwd -> salad_permute_tokens
 * (inverse) with the block sizes below.
 *   Blocks.  Heads in token order: 128 query x 64 key tokens, as everywhere.  Temporal heads: a key block is
 *   the T tokens of ks = floor(64 / T) consecutive spatial positions, a query block those of kq =
 *   floor(128 / T) positions (T = 21: 63 and 126 tokens; the rest of the 64- / 128-row tiles is masked), so
 *   that a block is a run of consecutive tokens of the re-ordered sequence.  T <= 64.
 *   Lists.  Hm = H.  Every head owns `rows` = max(ceil(N/128), ceil(Hs*Ws/kq)) list rows (salad_stswa_blocks
 *   returns rows, kq, ks and the number of key blocks of a temporal head); row h*rows + i is query block i of
 *   head h, rows beyond a head's own blocks are empty; block ids refer to the head's own key blocks.
 *   salad_stswa_mask_build makes the lists of the 1-D windows: h_windows[h] is the half-width of head h's
 *   window in tokens of its own order (a block pair is kept iff some token pair lies within it).
 *   Workspace: salad_stswa_workspace_bytes.  Other arguments as salad_fused_drop_fwd; d in {64, 128},
 *   H <= 256.  The rotary variant is not available with re-ordered heads (SALAD_ERR_UNSUPPORTED).
 */
int salad_stswa_blocks(int T, int Hs, int Ws, int32_t* h_list_rows, int32_t* h_q_positions,
                       int32_t* h_k_positions, int32_t* h_key_blocks);
size_t salad_stswa_workspace_bytes(int B, int H, int T, int Hs, int Ws, int d);
int salad_stswa_mask_build(int T, int Hs, int Ws, int H, const int32_t* h_head_flags,
                           const int32_t* h_windows, int32_t* d_row_ptr, int32_t* d_col_idx,
                           int64_t col_capacity, int64_t* h_nnz, void* stream);
int salad_fused_stswa_fwd(const void* q, const void* k, const void* v, void* o,
                          int B, int H, int N, int d, int T, int Hs, int Ws,
                          const int32_t* h_head_flags, const int32_t* row_ptr, const int32_t* col_idx,
                          const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                          float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                          int32_t* d_status, void* stream);

/*
 * salad_proj_combine_fwd -- Algorithm 1 with the full Level-1 projection (Sec. 4.2): a linear layer
 * on the head-concatenated output of the linear branch (zero-initialised before tuning), scaled by
 * the dynamic factor and added to the sparse branch,
 *     out[b, :, n, :] = O_s[b, :, n, :] + d_dyn_scale[b] * ( concat_h O_l[b, h, n, :] . W^T + bias ).
 * salad_fused_fwd covers the case W = blockdiag(lambda_h I) in one pass over Q, K, V; a projection
 * that mixes heads needs the two branch outputs first: salad_sparse_attn_fwd -> O_s,
 * salad_linear_attn_fwd -> O_l, then this call (a [B*N x D] x [D x D] tensor-core GEMM, D = H*d,
 * with the sum fused into its epilogue).
 *   o_s, o_l, out  bf16 [B, H, N, d], d in {64, 128}.  out may alias o_s, not o_l.
 *   w              bf16 [D][D], w[j_out][j_in], channel j = h*d + c (device).
 *   d_bias         fp32 [D] or NULL;   d_dyn_scale fp32 [B] or NULL (= 1).
 * Allocates nothing, needs no workspace.  fp32 accumulation, one rounding to bf16.
 */
int salad_proj_combine_fwd(const void* o_s, const void* o_l, const void* w, const float* d_bias,
                           const float* d_dyn_scale, void* out, int B, int H, int N, int d,
                           int32_t* d_status, void* stream);

/*
 * salad_selftest_bounded_wait -- diagnostic (no counterpart in the paper).  Every wait inside the
 * kernels is bounded: when one expires, the kernel records SALAD_ERR_TIMEOUT in the status word,
 * lets copies in flight land, frees its tensor memory and returns, so the context stays usable.
 * This entry point runs that mechanism on its own: a one-thread kernel waits 2 ms on a barrier
 * that nothing arrives on and then writes SALAD_ERR_TIMEOUT (-6) to *d_status; *d_waited_ns
 * (optional, device) receives the time it waited.  Nothing faults and nothing hangs.
 */
int salad_selftest_bounded_wait(int32_t* d_status, unsigned long long* d_waited_ns, void* stream);

/*
 * salad_linear_attn_fwd_noalloc -- salad_linear_attn_fwd for callers that cannot provide
 * scratch memory (the paper has no counterpart; this is a deployment convenience).
 * Some hosts of this library may not call cudaMalloc at the point where attention runs: a
 * plugin inside an inference server whose memory pool is fixed at start-up, code running
 * while a CUDA graph is being captured or replayed, a real-time loop that must not touch the
 * driver's allocator.  For them this entry point takes no workspace: its scratch (status
 * word, partial and final linear states) lives in a fixed array inside the library image,
 * SALAD_NOALLOC_SCRATCH_BYTES bytes of device memory that every GPU which loads the library
 * holds until the process exits.
 *   Arguments as salad_linear_attn_fwd, without workspace / workspace_bytes.
 *   Limits: B*H <= SALAD_NOALLOC_MAX_HEADS and d in {64, 128}; anything larger returns
 *   SALAD_ERR_UNSUPPORTED before any launch (use salad_linear_attn_fwd with a workspace).
 *   The first call on each device looks up the device address of the array (one runtime
 *   query, no allocation, with that device current); make that first call outside of any
 *   stream capture.  Later calls only enqueue work.
 *   All calls on a device share the one array: calls that may overlap on the GPU (different
 *   streams, different host threads) race on it and must be serialised by the caller.  The
 *   array keeps the previous call's contents; the call itself re-initialises everything it
 *   reads (the status word is cleared, every partial it sums is rewritten first).
 *   No cudaMalloc, cudaFree or other allocating routine is called.
 *   The looked-up address (like the library's other once-per-device set-up) is kept for the life of
 *   the process: after cudaDeviceReset on a device, do not call the library on that device again.
 */
#define SALAD_NOALLOC_MAX_HEADS 16
#define SALAD_NOALLOC_SCRATCH_BYTES 4759808
int salad_linear_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* o_l,
                                  float* kv_out, float* z_out, int B, int H, int N, int d,
                                  float eps, int32_t* d_status, void* stream);

/*
 * salad_set_profile_events -- optional instrumentation for benchmarks (no counterpart in
 * the paper).  h_events is a HOST array of four cudaEvent_t handles (as void*), or NULL to
 * switch the instrumentation off.  While set, every *_fwd call made by the calling host
 * thread records
 *     h_events[0], h_events[1]   around the linear-state kernels (Eq. 3 reductions), and
 *     h_events[2], h_events[3]   around the attention kernel (Eq. 2 + apply + combine)
 * on the call's stream; entries may individually be NULL.  The events stay owned by the
 * caller.  The setting is per host thread and changes nothing else about the calls.
 */
int salad_set_profile_events(void* const* h_events);

#ifdef __cplusplus
}
#endif
#endif /* SALAD_H_ */
