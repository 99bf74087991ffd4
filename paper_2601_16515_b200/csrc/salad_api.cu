// C ABI of libsalad (see include/salad.h): argument validation, workspace carving, TMA
// tensor maps and kernel launches.  No allocation, no global state beyond per-device
// "attributes already set" flags, no CPU fallback.
#include "../../include/salad.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include <mutex>

#include "dynamic_scale_kernel.cuh"
#include "fused_kernel.cuh"
#include "linear_apply_kernel.cuh"
#include "linear_state_kernel.cuh"
#include "mask_kernels.cuh"
#include "permute_kernel.cuh"
#include "proj_gemm_kernel.cuh"
#include "rope_table_kernel.cuh"
#include "selftest_kernel.cuh"
#include "tmap.cuh"
#include "topk_mask_kernels.cuh"
#include "work_order_kernel.cuh"

using namespace salad;

#define SALAD_EXPORT extern "C" __attribute__((visibility("default")))

namespace {

constexpr size_t kAlign = 256;
constexpr int kPartialSlots = 512;     // upper bound on (batch*heads) x chunks partial states
constexpr int kMaxMaskHeads = 256;

thread_local cudaEvent_t g_profile_events[4] = {nullptr, nullptr, nullptr, nullptr};
// > 0: the attention entry points called by this host thread validate their lists first, col_idx holding
// this many entries (salad_set_mask_validation)
thread_local int64_t g_validate_capacity = 0;

// SALAD_LOG=1 in the environment: one line per launch on stderr (host side only; read once).
bool log_enabled() {
    static const bool on = [] { const char* e = getenv("SALAD_LOG"); return e && e[0] && e[0] != '0'; }();
    return on;
}
#define SALAD_LOGF(...) do { if (log_enabled()) { fprintf(stderr, "[salad] " __VA_ARGS__); fputc('\n', stderr); } } while (0)

inline void record_profile(int idx, cudaStream_t st) {
    if (g_profile_events[idx]) cudaEventRecord(g_profile_events[idx], st);
}

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Workspace {
    size_t off_status, off_kvt, off_z, off_kvp, off_zp, off_order, total;
    int slots;
};

Workspace carve(int B, int H, int N, int d, int Bq, int list_rows = 0) {
    Workspace w;
    const size_t BH = size_t(B) * H;
    // work items of the attention kernel: query blocks (list rows per head, when a caller's lists have more)
    const size_t nItems = list_rows > 0 ? size_t(list_rows) : size_t(N + Bq - 1) / Bq;
    w.slots = int(BH > size_t(kPartialSlots) ? BH : size_t(kPartialSlots));
    w.off_status = 0;
    w.off_kvt = kAlign;
    w.off_z = w.off_kvt + align_up(BH * d * d * 2);
    w.off_kvp = w.off_z + align_up(BH * d * 4);
    w.off_zp = w.off_kvp + align_up(size_t(w.slots) * d * d * 4);
    w.off_order = w.off_zp + align_up(size_t(w.slots) * d * 4);
    w.total = w.off_order + align_up(BH * nItems * 4);              // launch order, per mask (at most B*H)
    return w;
}

bool shape_supported(int d, int Bq, int Bk) {
    return (d == 64 || d == 128) && (Bq == 64 || Bq == 128) && Bk == 64;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceInfo { int sms; bool ok; };

// Guards the once-per-device initialisation below (the entry points may be called from several host threads).
std::mutex g_init_mutex;

// sm_100 check and shared-memory opt-in of every kernel, once per device.
int prepare_device(DeviceInfo* info) {
    static bool attr_set[64] = {};
    static int sm_count[64] = {};
    std::lock_guard<std::mutex> lock(g_init_mutex);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SALAD_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return SALAD_ERR_CUDA;
    if (!attr_set[dev]) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return SALAD_ERR_CUDA;
        }
        if (major != 10) return SALAD_ERR_CUDA;   // kernels exist for sm_100a only
        cudaError_t e = cudaSuccess;
        e = cudaFuncSetAttribute(salad_fused_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 FusedCfg<128>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_fused_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     FusedCfg<64>::SMEM_BYTES);
        if (e == cudaSuccess)      // two CTAs of the attention kernel share an SM: ask for the largest shared-memory carve-out
            e = cudaFuncSetAttribute(salad_fused_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_fused_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<128, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<128, false, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<64, false, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<128, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<128, true, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<64, true, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<128, false, true>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     StateCfg<64, false, true>::SMEM_BYTES);
        if (e == cudaSuccess)      // beside a CTA of the attention kernel
            e = cudaFuncSetAttribute(salad_linear_state_kernel<128, true, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_state_kernel<64, true, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_apply_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     ApplyCfg<128, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_apply_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     ApplyCfg<64, false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_apply_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     ApplyCfg<128, true>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_linear_apply_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     ApplyCfg<64, true>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(topk_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kScoreSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_proj_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     ProjCfg::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(salad_proj_gemm_pair_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Proj2Cfg<256>::SMEM_BYTES);
        if (e != cudaSuccess) { cudaGetLastError(); return SALAD_ERR_CUDA; }
        sm_count[dev] = sms;
        attr_set[dev] = true;
    }
    info->sms = sm_count[dev];
    info->ok = true;
    return SALAD_OK;
}

// Launch with the programmatic-stream-serialization attribute: the kernel may be set up and its CTAs
// placed while the kernel before it in the stream drains.  Every kernel launched this way starts with
// grid_dependency_wait(), so stream order is kept; only the launch latency between the kernels of a
// call goes away.
template <typename... KArgs, typename... Args>
void launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                      Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);     // errors are read by check_launch()
}

int check_launch() {
    return cudaGetLastError() == cudaSuccess ? SALAD_OK : SALAD_ERR_CUDA;
}

// The temporal-head block geometry of a T x Hs x Ws grid: blocks of whole spatial positions.
struct StswaGeom { int S, kq, ks, nQb_p, nKb_p, nQb_tok, nKb_tok, rows; };
bool stswa_geometry(int T, int Hs, int Ws, StswaGeom* o) {
    if (T <= 0 || Hs <= 0 || Ws <= 0 || T > 64) return false;
    const int64_t S = int64_t(Hs) * Ws, N = S * T;
    if (N > 2147483647ll / 2) return false;
    o->S = int(S); o->kq = 128 / T; o->ks = 64 / T;
    o->nQb_p = int((S + o->kq - 1) / o->kq); o->nKb_p = int((S + o->ks - 1) / o->ks);
    o->nQb_tok = int((N + 127) / 128); o->nKb_tok = int((N + 63) / 64);
    o->rows = o->nQb_p > o->nQb_tok ? o->nQb_p : o->nQb_tok;
    return true;
}

struct Problem {
    const void *q, *k, *v; void* o; float* lse;
    int B, H, N, d, Bq, Bk, Hm, mode;
    const int32_t *row_ptr, *col_idx;
    const float *static_scale, *dyn_scale;
    float softmax_scale, eps, drop_tau;
    float *kv_out, *z_out;
    const void* rope;             // fp16 [N, d/2, 2] cosine and sine per token and channel pair, or null
    const void* proj_blocks;      // bf16 [H, d, d]: one projection block per head on the linear branch, or null
    int st_T, st_Hs, st_Ws;       // salad_fused_stswa_fwd: the latent grid (st_T == 0 otherwise) ...
    const int32_t* st_flags;      // ... and the host flags of the heads with temporal locality
    bool state_only;              // salad_linear_state_fwd: the two reductions of Eq. 3 and nothing else
    bool prepared;                // salad_fused_prepared_fwd: the workspace already holds the linear state
    void* ws; size_t ws_bytes; int32_t* d_status; cudaStream_t stream;
};

int validate(const Problem& P) {
    if (P.state_only) {
        if (!P.k || !P.v || !aligned16(P.k) || !aligned16(P.v)) return SALAD_ERR_INVALID_ARG;
    } else if (!P.q || !P.k || !P.v || !P.o) {
        return SALAD_ERR_INVALID_ARG;
    }
    if (P.B <= 0 || P.H <= 0 || P.N <= 0 || P.d <= 0 || P.Bq <= 0 || P.Bk <= 0) return SALAD_ERR_INVALID_ARG;
    if (!shape_supported(P.d, P.Bq, P.Bk)) return SALAD_ERR_UNSUPPORTED;
    if (!P.state_only && (!aligned16(P.q) || !aligned16(P.k) || !aligned16(P.v) || !aligned16(P.o)))
        return SALAD_ERR_INVALID_ARG;
    if (int64_t(P.B) * P.H > 65535) return SALAD_ERR_UNSUPPORTED;
    if (P.mode & MODE_SPARSE) {
        if (!P.row_ptr || !P.col_idx) return SALAD_ERR_INVALID_ARG;
        if (P.Hm != 1 && P.Hm != P.H && P.Hm != P.B * P.H) return SALAD_ERR_INVALID_ARG;
        if (!(P.softmax_scale >= 0.f) || !isfinite(P.softmax_scale)) return SALAD_ERR_INVALID_ARG;
    }
    if (P.mode & MODE_LINEAR) {
        if (!(P.eps >= 0.f) || !isfinite(P.eps)) return SALAD_ERR_INVALID_ARG;
        if (P.rope && !aligned16(P.rope)) return SALAD_ERR_INVALID_ARG;
    }
    if (P.mode == MODE_FUSED && ((!P.static_scale && !P.proj_blocks) || !P.dyn_scale)) return SALAD_ERR_INVALID_ARG;
    if (P.proj_blocks && !aligned16(P.proj_blocks)) return SALAD_ERR_INVALID_ARG;
    int list_rows = 0;
    if (P.st_T > 0) {
        StswaGeom sg;
        if (!P.st_flags || int64_t(P.st_T) * P.st_Hs * P.st_Ws != P.N) return SALAD_ERR_INVALID_ARG;
        if (!stswa_geometry(P.st_T, P.st_Hs, P.st_Ws, &sg) || P.H > 256 || P.Bq != 128 || P.rope) return SALAD_ERR_UNSUPPORTED;
        if (P.Hm != P.H) return SALAD_ERR_INVALID_ARG;
        list_rows = sg.rows;
    }
    const Workspace w = carve(P.B, P.H, P.N, P.d, P.Bq, list_rows);
    if (!P.ws || (reinterpret_cast<uintptr_t>(P.ws) % kAlign) != 0 || P.ws_bytes < w.total)
        return SALAD_ERR_WORKSPACE;
    return SALAD_OK;
}

int list_rows_of(const Problem& P) {
    StswaGeom sg;
    return (P.st_T > 0 && stswa_geometry(P.st_T, P.st_Hs, P.st_Ws, &sg)) ? sg.rows : 0;
}

template <int D>
int launch_state(const Problem& P, const Workspace& w, const DeviceInfo& dev) {
    const int BH = P.B * P.H;
    const int nKb = (P.N + 63) / 64;
    int chunks = dev.sms / BH;          // one CTA per SM (its stage ring takes most of the shared memory)
    if (chunks < 1) chunks = 1;
    if (chunks > nKb) chunks = nKb;
    if (int64_t(chunks) * BH > w.slots) chunks = w.slots / BH;
    const int bpc = (nKb + chunks - 1) / chunks;
    uint8_t* ws = static_cast<uint8_t*>(P.ws);
    CUtensorMap mk, mv;
    if (!make_tmap_bf16_3d(&mk, P.k, D, P.N, BH, 64) || !make_tmap_bf16_3d(&mv, P.v, D, P.N, BH, 64))
        return SALAD_ERR_CUDA;
    CUtensorMap mr = mk;          // unused without a rotation table
    if (P.rope && !make_tmap_f16_rows(&mr, P.rope, D, P.N, 64)) return SALAD_ERR_CUDA;
    StateParams sp;
    sp.N = P.N; sp.nKb = nKb; sp.chunks = chunks; sp.blocks_per_chunk = bpc;
    sp.kv_part = reinterpret_cast<float*>(ws + w.off_kvp);
    sp.z_part = reinterpret_cast<float*>(ws + w.off_zp);
    sp.ws_status = reinterpret_cast<int32_t*>(ws + w.off_status);
    sp.user_status = P.d_status;
    sp.dyn_scale = P.dyn_scale; sp.drop_tau = P.drop_tau; sp.H = P.H;
    record_profile(0, P.stream);
    // Fused calls: the short-ring variant, which shares its SM with a CTA of the attention kernel.  With a
    // rotation table the state pass keeps the SM to itself (full ring, eight ReLU warps): sharing the SM with
    // the attention kernel was measured no faster.
    // In a linear-only call this is the first kernel: an ordinary launch (it must not start before the call
    // before it has ended), which clears the status words itself.
    sp.clear_status = (P.mode & MODE_SPARSE) ? 0 : 1;
    auto launch = [&](auto kernel, int threads, int smem) {
        if (sp.clear_status)
            kernel<<<dim3(chunks, BH), dim3(threads), size_t(smem), P.stream>>>(mk, mv, mr, sp);
        else
            launch_dependent(kernel, dim3(chunks, BH), dim3(threads), size_t(smem), P.stream, mk, mv, mr, sp);
    };
    if (P.rope)
        launch(salad_linear_state_kernel<D, false, true>, StateCfg<D, false, true>::THREADS,
               StateCfg<D, false, true>::SMEM_BYTES);
    else if (P.mode & MODE_SPARSE)
        launch(salad_linear_state_kernel<D, true, false>, StateCfg<D, true, false>::THREADS,
               StateCfg<D, true, false>::SMEM_BYTES);
    else
        launch(salad_linear_state_kernel<D, false, false>, StateCfg<D, false, false>::THREADS,
               StateCfg<D, false, false>::SMEM_BYTES);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    float* z_ws = reinterpret_cast<float*>(ws + w.off_z);
    __nv_bfloat16* kvt = reinterpret_cast<__nv_bfloat16*>(ws + w.off_kvt);
    if (P.proj_blocks)      // block-diagonal projection folded into the state: the attention kernel multiplies with KV W_h^T
        launch_dependent(salad_linear_finalize_proj_kernel<D>, dim3(D / 8, BH), dim3(256), 0, P.stream,
                         sp.kv_part, sp.z_part, chunks, static_cast<const __nv_bfloat16*>(P.proj_blocks), P.kv_out, z_ws,
                         P.z_out, kvt, P.dyn_scale, P.drop_tau, P.H);
    else if ((P.mode & MODE_SPARSE) && !P.rope)
        launch_dependent(salad_linear_finalize_kernel<D, 8>, dim3(D / 32, D / 32, BH), dim3(32, 8), 0, P.stream,
                         sp.kv_part, sp.z_part, chunks, P.kv_out, z_ws, P.z_out, kvt, P.dyn_scale, P.drop_tau, P.H);
    else
        launch_dependent(salad_linear_finalize_kernel<D, 32>, dim3(D / 32, D / 32, BH), dim3(32, 32), 0, P.stream,
                         sp.kv_part, sp.z_part, chunks, P.kv_out, z_ws, P.z_out, kvt, P.dyn_scale, P.drop_tau, P.H);
    record_profile(1, P.stream);
    return check_launch();
}

template <int D>
int launch_fused(const Problem& P, const Workspace& w, const DeviceInfo& dev) {
    const int BH = P.B * P.H;
    uint8_t* ws = static_cast<uint8_t*>(P.ws);
    CUtensorMap mq, mk, mv, mo, ms;
    if (!make_tmap_bf16_3d(&mq, P.q, D, P.N, BH, P.Bq) || !make_tmap_bf16_3d(&mk, P.k, D, P.N, BH, 64) ||
        !make_tmap_bf16_3d(&mv, P.v, D, P.N, BH, 64) || !make_tmap_bf16_3d(&mo, P.o, D, P.N, BH, P.Bq) ||
        !make_tmap_bf16_3d(&ms, ws + w.off_kvt, D, D, BH, D))
        return SALAD_ERR_CUDA;
    FusedParams fp;
    fp.N = P.N; fp.H = P.H; fp.Bq = P.Bq; fp.Hm = P.Hm; fp.mode = P.mode;
    fp.nQb = (P.N + P.Bq - 1) / P.Bq;
    fp.nKb = (P.N + 63) / 64;
    fp.nQb_tok = fp.nQb;
    fp.th = TemporalHeads{};
    CUtensorMap mq4 = mq, mk4 = mk, mv4 = mv, mo4 = mo;        // unused without temporal heads
    if (P.st_T > 0) {
        // heads with temporal locality read and write their tokens grouped by spatial position through 4-D maps
        StswaGeom sg;
        stswa_geometry(P.st_T, P.st_Hs, P.st_Ws, &sg);
        fp.th.T = P.st_T; fp.th.S = sg.S; fp.th.kq = sg.kq; fp.th.ks = sg.ks; fp.th.nQb = sg.nQb_p; fp.th.nKb = sg.nKb_p;
        for (int h = 0; h < P.H; ++h)
            if (P.st_flags[h]) fp.th.flags[h >> 5] |= 1u << (h & 31);
        fp.nQb = sg.rows;
        if (!make_tmap_bf16_4d_by_position(&mq4, P.q, D, P.st_T, sg.S, BH, sg.kq) ||
            !make_tmap_bf16_4d_by_position(&mk4, P.k, D, P.st_T, sg.S, BH, sg.ks) ||
            !make_tmap_bf16_4d_by_position(&mv4, P.v, D, P.st_T, sg.S, BH, sg.ks) ||
            !make_tmap_bf16_4d_by_position(&mo4, P.o, D, P.st_T, sg.S, BH, sg.kq))
            return SALAD_ERR_CUDA;
    }
    fp.row_ptr = P.row_ptr; fp.col_idx = P.col_idx;
    fp.BH = BH;
    fp.order = nullptr;
    if (P.mode & MODE_SPARSE) fp.order = reinterpret_cast<const int32_t*>(ws + w.off_order);   // written by run()
    fp.static_scale = P.static_scale; fp.dyn_scale = P.dyn_scale;
    fp.z = reinterpret_cast<const float*>(ws + w.off_z);
    fp.lse = P.lse;
    const float sc = (P.softmax_scale > 0.f) ? P.softmax_scale : 1.0f / sqrtf(float(D));
    fp.scale_log2 = sc * 1.4426950408889634f;
    fp.eps = P.eps;
    fp.drop_tau = P.drop_tau;
    fp.rope = static_cast<const __half*>(P.rope);
    fp.ws_status = reinterpret_cast<int32_t*>(ws + w.off_status);
    fp.user_status = P.d_status;
    fp.wait_at_top = P.prepared ? 1 : 0;      // no state kernels in this call: the kernel before is the first one
    const int64_t grid = int64_t(fp.nQb) * BH;
    if (grid > 2147483647ll) return SALAD_ERR_UNSUPPORTED;
    record_profile(2, P.stream);
    SALAD_LOGF("salad_fused_kernel<%d> grid %lld block %d smem %d (mode %d)", D, (long long)grid, FusedCfg<D>::THREADS,
               FusedCfg<D>::SMEM_BYTES, P.mode);
    launch_dependent(salad_fused_kernel<D>, dim3(unsigned(grid)), dim3(FusedCfg<D>::THREADS),
                     FusedCfg<D>::SMEM_BYTES, P.stream, mq, mk, mv, mo, ms, mq4, mk4, mv4, mo4, fp);
    record_profile(3, P.stream);
    return check_launch();
}

// Linear-only calls: the stand-alone apply kernel, one persistent CTA per SM.
template <int D>
int launch_apply(const Problem& P, const Workspace& w, const DeviceInfo& dev) {
    const int BH = P.B * P.H;
    uint8_t* ws = static_cast<uint8_t*>(P.ws);
    CUtensorMap mq, mo, ms, mr;
    if (!make_tmap_bf16_3d(&mq, P.q, D, P.N, BH, 128) || !make_tmap_bf16_3d(&mo, P.o, D, P.N, BH, 128) ||
        !make_tmap_bf16_3d(&ms, ws + w.off_kvt, D, D, BH, D))
        return SALAD_ERR_CUDA;
    mr = mq;                      // unused without a rotation table
    // the fp16 table [N, D] is tiled exactly like a Q tile of one (batch, head): 16-bit elements, 128-byte swizzle
    if (P.rope && !make_tmap_bf16_3d(&mr, P.rope, D, P.N, 1, 128)) return SALAD_ERR_CUDA;
    ApplyParams ap;
    ap.N = P.N; ap.H = P.H;
    ap.nQb = (P.N + 127) / 128;
    ap.tiles = (long long)ap.nQb * BH;
    ap.z = reinterpret_cast<const float*>(ws + w.off_z);
    ap.static_scale = P.static_scale; ap.dyn_scale = P.dyn_scale;
    ap.eps = P.eps;
    ap.ws_status = reinterpret_cast<int32_t*>(ws + w.off_status);
    ap.user_status = P.d_status;
    const unsigned grid = unsigned(ap.tiles < dev.sms ? ap.tiles : dev.sms);
    record_profile(2, P.stream);
    if (P.rope)
        launch_dependent(salad_linear_apply_kernel<D, true>, dim3(grid), dim3(ApplyCfg<D, true>::THREADS),
                         ApplyCfg<D, true>::SMEM_BYTES, P.stream, mq, ms, mo, mr, ap);
    else
        launch_dependent(salad_linear_apply_kernel<D, false>, dim3(grid), dim3(ApplyCfg<D, false>::THREADS),
                         ApplyCfg<D, false>::SMEM_BYTES, P.stream, mq, ms, mo, mr, ap);
    record_profile(3, P.stream);
    return check_launch();
}

// Clears the status words in stream order, then checks the lists (see work_order_kernel.cuh).
int launch_csr_validate(const int32_t* row_ptr, const int32_t* col_idx, int64_t col_capacity, int64_t rows, int nKb,
                        int32_t* status_a, int32_t* status_b, cudaStream_t st) {
    if (rows <= 0 || rows > (1ll << 26)) return SALAD_ERR_UNSUPPORTED;
    if ((status_a && cudaMemsetAsync(status_a, 0, sizeof(int32_t), st) != cudaSuccess) ||
        (status_b && cudaMemsetAsync(status_b, 0, sizeof(int32_t), st) != cudaSuccess)) {
        cudaGetLastError();
        return SALAD_ERR_CUDA;
    }
    const unsigned blocks = unsigned((rows * 32 + 255) / 256);
    SALAD_LOGF("csr_validate_kernel grid %u block 256 (rows %lld, capacity %lld)", blocks, (long long)rows,
               (long long)col_capacity);
    csr_validate_kernel<<<blocks, 256, 0, st>>>(row_ptr, col_idx, (long long)col_capacity, int(rows), nKb, status_a,
                                                status_b);
    return check_launch();
}

int run(const Problem& P) {
    int rc = validate(P);
    if (rc != SALAD_OK) return rc;
    DeviceInfo dev{};
    rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    const Workspace w = carve(P.B, P.H, P.N, P.d, P.Bq, list_rows_of(P));
    uint8_t* ws = static_cast<uint8_t*>(P.ws);
    if (P.mode & MODE_SPARSE) {
        // first kernel of the call: longest work items first (the mask is an input of every call,
        // so is its order); it also clears the status words
        const int nQb = list_rows_of(P) > 0 ? list_rows_of(P) : (P.N + P.Bq - 1) / P.Bq;
        int32_t* ws_status = reinterpret_cast<int32_t*>(ws + w.off_status);
        int clear_status = 1;
        if (g_validate_capacity > 0) {
            // opt-in check of the lists (salad_set_mask_validation): it owns the status words of this call
            int nkb_bound = (P.N + 63) / 64;
            StswaGeom sg;                      // temporal heads have their own key-block count: the larger bounds both
            if (P.st_T > 0 && stswa_geometry(P.st_T, P.st_Hs, P.st_Ws, &sg) && sg.nKb_p > nkb_bound) nkb_bound = sg.nKb_p;
            rc = launch_csr_validate(P.row_ptr, P.col_idx, g_validate_capacity, int64_t(P.Hm) * nQb, nkb_bound,
                                     ws_status, P.d_status, P.stream);
            if (rc != SALAD_OK) return rc;
            clear_status = 0;
        }
        SALAD_LOGF("work_order_kernel grid %d block 1024 (nQb %d)%s", P.Hm, nQb, clear_status ? "" : " after csr_validate_kernel");
        work_order_kernel<<<P.Hm, 1024, 0, P.stream>>>(P.row_ptr, nQb, P.Hm,
                                                      reinterpret_cast<int32_t*>(ws + w.off_order), ws_status,
                                                      P.d_status, clear_status);
        if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    }
    if ((P.mode & MODE_LINEAR) && !P.prepared) {
        rc = (P.d == 128) ? launch_state<128>(P, w, dev) : launch_state<64>(P, w, dev);
        if (rc != SALAD_OK) return rc;
    }
    if (P.state_only) return SALAD_OK;
    // linear-only calls: the stand-alone apply kernel
    if (P.mode == MODE_LINEAR)
        return (P.d == 128) ? launch_apply<128>(P, w, dev) : launch_apply<64>(P, w, dev);
    return (P.d == 128) ? launch_fused<128>(P, w, dev) : launch_fused<64>(P, w, dev);
}

// ---------------------------------------------------------------------------------------
// Scratch for salad_linear_attn_fwd_noalloc: a fixed array in the library image instead of a
// caller workspace.  In host code the symbol below is only a handle; the device address is
// obtained once per device with cudaGetSymbolAddress and cached.
constexpr int kNoAllocSlots = 64;      // partial-state slots (batch*heads x chunks)

constexpr size_t noalloc_align(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
constexpr size_t kNoAllocBytes =
    kAlign +                                                              // status word
    noalloc_align(size_t(SALAD_NOALLOC_MAX_HEADS) * 128 * 128 * 2) +      // bf16 transposed state
    noalloc_align(size_t(SALAD_NOALLOC_MAX_HEADS) * 128 * 4) +            // Z
    noalloc_align(size_t(kNoAllocSlots) * 128 * 128 * 4) +                // partial KV
    noalloc_align(size_t(kNoAllocSlots) * 128 * 4);                       // partial Z
static_assert(kNoAllocBytes == SALAD_NOALLOC_SCRATCH_BYTES, "header constant out of date");

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Layout of the fixed scratch for this (B, H, d): the same regions as a caller workspace,
// with fewer partial slots.
Workspace carve_noalloc(int B, int H, int d) {
    Workspace w;
    const size_t BH = size_t(B) * H;
    w.slots = kNoAllocSlots;
    w.off_status = 0;
    w.off_kvt = kAlign;
    w.off_z = w.off_kvt + align_up(BH * d * d * 2);
    w.off_kvp = w.off_z + align_up(BH * d * 4);
    w.off_zp = w.off_kvp + align_up(size_t(w.slots) * d * d * 4);
    w.off_order = 0;                                  // linear attention has no kept lists to order
    w.total = w.off_zp + align_up(size_t(w.slots) * d * 4);
    return w;
}

// Device address of g_noalloc_scratch on the current device (looked up on first use).
int noalloc_scratch_ptr(void** out) {
    static void* cached[64] = {};
    std::lock_guard<std::mutex> lock(g_init_mutex);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return SALAD_ERR_CUDA; }
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return SALAD_ERR_CUDA;
        }
        cached[dev] = ptr;
    }
    *out = cached[dev];
    return SALAD_OK;
}

}  // namespace

SALAD_EXPORT const char* salad_status_string(int status) {
    switch (status) {
        case SALAD_OK: return "SALAD_OK";
        case SALAD_ERR_INVALID_ARG: return "SALAD_ERR_INVALID_ARG";
        case SALAD_ERR_UNSUPPORTED: return "SALAD_ERR_UNSUPPORTED";
        case SALAD_ERR_WORKSPACE: return "SALAD_ERR_WORKSPACE";
        case SALAD_ERR_CAPACITY: return "SALAD_ERR_CAPACITY";
        case SALAD_ERR_CUDA: return "SALAD_ERR_CUDA";
        case SALAD_ERR_TIMEOUT: return "SALAD_ERR_TIMEOUT";
        case SALAD_ERR_BAD_MASK: return "SALAD_ERR_BAD_MASK";
        default: return "SALAD_ERR_UNKNOWN";
    }
}

SALAD_EXPORT int salad_set_profile_events(void* const* h_events) {
    for (int i = 0; i < 4; ++i)
        g_profile_events[i] = h_events ? static_cast<cudaEvent_t>(h_events[i]) : nullptr;
    return SALAD_OK;
}

SALAD_EXPORT int salad_set_mask_validation(int64_t col_capacity) {
    if (col_capacity < 0) return SALAD_ERR_INVALID_ARG;
    g_validate_capacity = col_capacity;
    return SALAD_OK;
}

SALAD_EXPORT int salad_csr_validate(const int32_t* row_ptr, const int32_t* col_idx, int64_t col_capacity,
                                    int64_t rows, int nKb, int32_t* d_status, void* stream) {
    if (!row_ptr || !d_status || rows <= 0 || nKb <= 0 || col_capacity < 0 || (!col_idx && col_capacity > 0))
        return SALAD_ERR_INVALID_ARG;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    return launch_csr_validate(row_ptr, col_idx, col_capacity, rows, nKb, d_status, nullptr,
                               static_cast<cudaStream_t>(stream));
}

SALAD_EXPORT size_t salad_workspace_bytes(int B, int H, int N, int d, int Bq, int Bk) {
    if (B <= 0 || H <= 0 || N <= 0 || !shape_supported(d, Bq, Bk)) return 0;
    return carve(B, H, N, d, Bq).total;
}

int build_mask_lists(MaskGeom g, const int32_t* h_windows, const uint32_t* alt_bits, int32_t* d_row_ptr,
                     int32_t* d_col_idx, int64_t col_capacity, int64_t* h_nnz, void* stream);

SALAD_EXPORT int salad_mask_build(int T, int Hs, int Ws, int Bq, int Bk, int Hm, const int32_t* h_windows,
                                  int32_t* d_row_ptr, int32_t* d_col_idx, int64_t col_capacity,
                                  int64_t* h_nnz, void* stream) {
    if (T <= 0 || Hs <= 0 || Ws <= 0 || Bq <= 0 || Bk <= 0 || Hm <= 0 || !h_windows || !d_row_ptr)
        return SALAD_ERR_INVALID_ARG;
    if (col_capacity < 0 || (d_col_idx == nullptr && col_capacity != 0)) return SALAD_ERR_INVALID_ARG;
    if (Hm > kMaxMaskHeads) return SALAD_ERR_UNSUPPORTED;
    const int64_t N64 = int64_t(T) * Hs * Ws;
    if (N64 > 2147483647ll / 2) return SALAD_ERR_UNSUPPORTED;
    for (int i = 0; i < 3 * Hm; ++i) if (h_windows[i] < 0) return SALAD_ERR_INVALID_ARG;
    MaskGeom g;
    g.T = T; g.Hs = Hs; g.Ws = Ws; g.N = int(N64); g.Bq = Bq; g.Bk = Bk; g.Hm = Hm;
    g.nQb = (g.N + Bq - 1) / Bq; g.nKb = (g.N + Bk - 1) / Bk;
    g.Bq2 = Bq; g.Bk2 = Bk; g.nQb2 = g.nQb; g.nKb2 = g.nKb; g.nQb1 = g.nQb;      // one geometry for every mask head
    return build_mask_lists(g, h_windows, nullptr, d_row_ptr, d_col_idx, col_capacity, h_nnz, stream);
}


int build_mask_lists(MaskGeom g, const int32_t* h_windows, const uint32_t* alt_bits, int32_t* d_row_ptr,
                     int32_t* d_col_idx, int64_t col_capacity, int64_t* h_nnz, void* stream) {
    const int Hm = g.Hm;
    const int64_t rows64 = int64_t(Hm) * g.nQb;
    if (rows64 > (1 << 24)) return SALAD_ERR_UNSUPPORTED;
    const int rows = int(rows64);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // The windows travel as a kernel argument; the per-row counts are scanned in place in
    // row_ptr; row_ptr[rows] doubles as the overflow probe target before it is overwritten.
    MaskWindows win;
    for (int i = 0; i < 3 * kMaxMaskHeads; ++i) win.w[i] = (i < 3 * Hm) ? h_windows[i] : 0;
    for (int i = 0; i < 8; ++i) win.alt[i] = alt_bits ? alt_bits[i] : 0u;
    const int blocks = (rows * 32 + 255) / 256;
    mask_rows_kernel<false><<<blocks, 256, 0, st>>>(g, win, d_row_ptr, nullptr);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    mask_scan_kernel<<<1, 1024, 0, st>>>(d_row_ptr, rows);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    int32_t last = 0;
    if (cudaMemcpyAsync(&last, d_row_ptr + rows, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return SALAD_ERR_CUDA;
    }
    if (last < 0) return SALAD_ERR_UNSUPPORTED;     // more than 2^31 - 1 kept blocks
    if (h_nnz) *h_nnz = last;
    if (!d_col_idx) return SALAD_OK;
    if (col_capacity < last) return SALAD_ERR_CAPACITY;
    mask_rows_kernel<true><<<blocks, 256, 0, st>>>(g, win, d_row_ptr, d_col_idx);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return SALAD_ERR_CUDA; }
    return SALAD_OK;
}

SALAD_EXPORT int salad_sparse_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                                       int B, int H, int N, int d, int Bq, int Bk,
                                       const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                       float softmax_scale, void* workspace, size_t workspace_bytes,
                                       int32_t* d_status, void* stream) {
    Problem P{};
    P.drop_tau = -INFINITY;
    P.q = q; P.k = k; P.v = v; P.o = o; P.lse = lse;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = Bq; P.Bk = Bk; P.Hm = Hm; P.mode = MODE_SPARSE;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.softmax_scale = softmax_scale; P.eps = 0.f;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_linear_attn_fwd(const void* q, const void* k, const void* v, void* o_l,
                                       float* kv_out, float* z_out, int B, int H, int N, int d, float eps,
                                       void* workspace, size_t workspace_bytes, int32_t* d_status,
                                       void* stream) {
    Problem P{};
    P.drop_tau = -INFINITY;
    P.q = q; P.k = k; P.v = v; P.o = o_l;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = 128; P.Bk = 64; P.Hm = 1; P.mode = MODE_LINEAR;
    P.eps = eps; P.kv_out = kv_out; P.z_out = z_out;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_fused_drop_fwd(const void* q, const void* k, const void* v, void* o,
                                      int B, int H, int N, int d, int Bq, int Bk,
                                      const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                      const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                                      float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                                      int32_t* d_status, void* stream) {
    if (isnan(drop_tau)) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.q = q; P.k = k; P.v = v; P.o = o;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = Bq; P.Bk = Bk; P.Hm = Hm; P.mode = MODE_FUSED;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.static_scale = d_static_scale; P.dyn_scale = d_dyn_scale; P.drop_tau = drop_tau;
    P.softmax_scale = softmax_scale; P.eps = eps;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_fused_fwd(const void* q, const void* k, const void* v, void* o,
                                 int B, int H, int N, int d, int Bq, int Bk,
                                 const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                 const float* d_static_scale, const float* d_dyn_scale,
                                 float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                                 int32_t* d_status, void* stream) {
    // no threshold: every branch is kept, whatever the value of its scale
    return salad_fused_drop_fwd(q, k, v, o, B, H, N, d, Bq, Bk, row_ptr, col_idx, Hm, d_static_scale, d_dyn_scale,
                                -INFINITY, softmax_scale, eps, workspace, workspace_bytes, d_status, stream);
}

SALAD_EXPORT int salad_linear_state_fwd(const void* k, const void* v, float* kv_out, float* z_out, int B, int H, int N,
                                        int d, void* workspace, size_t workspace_bytes, int32_t* d_status,
                                        void* stream) {
    Problem P{};
    P.drop_tau = -INFINITY;
    P.k = k; P.v = v;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = 128; P.Bk = 64; P.Hm = 1; P.mode = MODE_LINEAR;
    P.state_only = true;
    P.kv_out = kv_out; P.z_out = z_out;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_fused_prepared_fwd(const void* q, const void* k, const void* v, void* o,
                                          int B, int H, int N, int d, int Bq, int Bk,
                                          const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                          const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                                          float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                                          int32_t* d_status, void* stream) {
    if (isnan(drop_tau)) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.q = q; P.k = k; P.v = v; P.o = o;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = Bq; P.Bk = Bk; P.Hm = Hm; P.mode = MODE_FUSED;
    P.prepared = true;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.static_scale = d_static_scale; P.dyn_scale = d_dyn_scale; P.drop_tau = drop_tau;
    P.softmax_scale = softmax_scale; P.eps = eps;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_stswa_blocks(int T, int Hs, int Ws, int32_t* h_list_rows, int32_t* h_q_positions,
                                    int32_t* h_k_positions, int32_t* h_key_blocks) {
    StswaGeom sg;
    if (T <= 0 || Hs <= 0 || Ws <= 0) return SALAD_ERR_INVALID_ARG;
    if (!stswa_geometry(T, Hs, Ws, &sg)) return SALAD_ERR_UNSUPPORTED;
    if (h_list_rows) *h_list_rows = sg.rows;
    if (h_q_positions) *h_q_positions = sg.kq;
    if (h_k_positions) *h_k_positions = sg.ks;
    if (h_key_blocks) *h_key_blocks = sg.nKb_p;
    return SALAD_OK;
}

SALAD_EXPORT size_t salad_stswa_workspace_bytes(int B, int H, int T, int Hs, int Ws, int d) {
    StswaGeom sg;
    if (B <= 0 || H <= 0 || (d != 64 && d != 128) || !stswa_geometry(T, Hs, Ws, &sg)) return 0;
    return carve(B, H, T * sg.S, d, 128, sg.rows).total;
}

SALAD_EXPORT int salad_stswa_mask_build(int T, int Hs, int Ws, int H, const int32_t* h_head_flags,
                                        const int32_t* h_windows, int32_t* d_row_ptr, int32_t* d_col_idx,
                                        int64_t col_capacity, int64_t* h_nnz, void* stream) {
    if (T <= 0 || Hs <= 0 || Ws <= 0 || H <= 0 || !h_head_flags || !h_windows || !d_row_ptr) return SALAD_ERR_INVALID_ARG;
    if (col_capacity < 0 || (d_col_idx == nullptr && col_capacity != 0)) return SALAD_ERR_INVALID_ARG;
    StswaGeom sg;
    if (H > kMaxMaskHeads || !stswa_geometry(T, Hs, Ws, &sg)) return SALAD_ERR_UNSUPPORTED;
    for (int h = 0; h < H; ++h) if (h_windows[h] < 0) return SALAD_ERR_INVALID_ARG;
    // a 1-D window on every head's own token order: the grid 1 x 1 x N, blocks of 128 x 64 tokens, or of the
    // tokens of kq x ks whole spatial positions for the heads that take their tokens grouped by position
    MaskGeom g;
    g.T = 1; g.Hs = 1; g.Ws = T * sg.S; g.N = T * sg.S; g.Hm = H;
    g.Bq = 128; g.Bk = 64; g.nQb1 = sg.nQb_tok; g.nKb = sg.nKb_tok;
    g.Bq2 = sg.kq * T; g.Bk2 = sg.ks * T; g.nQb2 = sg.nQb_p; g.nKb2 = sg.nKb_p;
    g.nQb = sg.rows;
    int32_t win[3 * kMaxMaskHeads];
    uint32_t alt[8] = {};
    for (int h = 0; h < H; ++h) {
        win[3 * h] = 0; win[3 * h + 1] = 0; win[3 * h + 2] = h_windows[h];
        if (h_head_flags[h]) alt[h >> 5] |= 1u << (h & 31);
    }
    return build_mask_lists(g, win, alt, d_row_ptr, d_col_idx, col_capacity, h_nnz, stream);
}

SALAD_EXPORT int salad_fused_stswa_fwd(const void* q, const void* k, const void* v, void* o,
                                       int B, int H, int N, int d, int T, int Hs, int Ws,
                                       const int32_t* h_head_flags, const int32_t* row_ptr, const int32_t* col_idx,
                                       const float* d_static_scale, const float* d_dyn_scale, float drop_tau,
                                       float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                                       int32_t* d_status, void* stream) {
    if (isnan(drop_tau) || !h_head_flags || T <= 0 || Hs <= 0 || Ws <= 0) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.q = q; P.k = k; P.v = v; P.o = o;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = 128; P.Bk = 64; P.Hm = H; P.mode = MODE_FUSED;
    P.st_T = T; P.st_Hs = Hs; P.st_Ws = Ws; P.st_flags = h_head_flags;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.static_scale = d_static_scale; P.dyn_scale = d_dyn_scale; P.drop_tau = drop_tau;
    P.softmax_scale = softmax_scale; P.eps = eps;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_fused_proj_fwd(const void* q, const void* k, const void* v, void* o,
                                      int B, int H, int N, int d, int Bq, int Bk,
                                      const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                      const void* d_proj_blocks, const float* d_dyn_scale, float drop_tau,
                                      float softmax_scale, float eps, void* workspace, size_t workspace_bytes,
                                      int32_t* d_status, void* stream) {
    if (isnan(drop_tau) || !d_proj_blocks) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.q = q; P.k = k; P.v = v; P.o = o;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = Bq; P.Bk = Bk; P.Hm = Hm; P.mode = MODE_FUSED;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.static_scale = nullptr; P.dyn_scale = d_dyn_scale; P.drop_tau = drop_tau;
    P.proj_blocks = d_proj_blocks;
    P.softmax_scale = softmax_scale; P.eps = eps;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_fused_rope_fwd(const void* q, const void* k, const void* v, void* o,
                                      int B, int H, int N, int d, int Bq, int Bk,
                                      const int32_t* row_ptr, const int32_t* col_idx, int Hm,
                                      const float* d_static_scale, const float* d_dyn_scale, const void* d_rope,
                                      float drop_tau, float softmax_scale, float eps, void* workspace,
                                      size_t workspace_bytes, int32_t* d_status, void* stream) {
    if (isnan(drop_tau) || !d_rope) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.q = q; P.k = k; P.v = v; P.o = o;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = Bq; P.Bk = Bk; P.Hm = Hm; P.mode = MODE_FUSED;
    P.row_ptr = row_ptr; P.col_idx = col_idx;
    P.static_scale = d_static_scale; P.dyn_scale = d_dyn_scale; P.drop_tau = drop_tau;
    P.rope = d_rope;
    P.softmax_scale = softmax_scale; P.eps = eps;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_linear_attn_rope_fwd(const void* q, const void* k, const void* v, void* o_l,
                                            float* kv_out, float* z_out, int B, int H, int N, int d,
                                            const void* d_rope, float eps, void* workspace,
                                            size_t workspace_bytes, int32_t* d_status, void* stream) {
    if (!d_rope) return SALAD_ERR_INVALID_ARG;
    Problem P{};
    P.drop_tau = -INFINITY;
    P.q = q; P.k = k; P.v = v; P.o = o_l;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = 128; P.Bk = 64; P.Hm = 1; P.mode = MODE_LINEAR;
    P.rope = d_rope;
    P.eps = eps; P.kv_out = kv_out; P.z_out = z_out;
    P.ws = workspace; P.ws_bytes = workspace_bytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    return run(P);
}

SALAD_EXPORT int salad_dynamic_scale(const void* x, const float* w, float bias, int B, int N, int D,
                                     float* s_out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!x || !w || !s_out || B <= 0 || N <= 0 || D <= 0 || !isfinite(bias)) return SALAD_ERR_INVALID_ARG;
    if (!aligned16(x)) return SALAD_ERR_INVALID_ARG;
    if (D % 8 != 0 || D > 8192 || B > 2048) return SALAD_ERR_UNSUPPORTED;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0 ||
        workspace_bytes < SALAD_DYN_SCALE_WS_BYTES)
        return SALAD_ERR_WORKSPACE;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int slots = SALAD_DYN_SCALE_WS_BYTES / 4;
    // one wave: as many CTAs as the device holds at once, split over the batch items
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dynamic_scale_partial_kernel, kDynScaleThreads,
                                                      size_t(D) * 4) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        return SALAD_ERR_CUDA;
    }
    int G = (per_sm * dev.sms) / B;
    if (G > slots / B) G = slots / B;
    if (G > (N + 7) / 8) G = (N + 7) / 8;            // at least one token per warp
    if (G < 1) G = 1;
    float* partial = static_cast<float*>(workspace);
    dynamic_scale_partial_kernel<<<dim3(G, B), kDynScaleThreads, size_t(D) * 4, st>>>(
        static_cast<const uint4*>(x), w, bias, N, D, partial);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    dynamic_scale_finalize_kernel<<<B, 32, 0, st>>>(partial, G, N, s_out);
    return check_launch();
}

SALAD_EXPORT size_t salad_topk_workspace_bytes(int B, int H, int N, int d, int Bq, int Bk) {
    if (B <= 0 || H <= 0 || N <= 0 || d <= 0 || Bq <= 0 || Bk <= 0) return 0;
    const size_t BH = size_t(B) * H;
    const size_t nQb = (size_t(N) + Bq - 1) / Bq, nKb = (size_t(N) + Bk - 1) / Bk;
    const size_t ldk = (nKb + kScoreTile - 1) / kScoreTile * kScoreTile;
    // query-block means | key-block means, channel-major, rows padded to whole tiles | scores
    return align_up(BH * nQb * d * 4) + align_up(BH * d * ldk * 4) + align_up(BH * nQb * nKb * 4);
}

SALAD_EXPORT int salad_topk_mask_build(const void* q, const void* k, int B, int H, int N, int d, int Bq, int Bk,
                                       int topk, int32_t* d_row_ptr, int32_t* d_col_idx, int64_t col_capacity,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!q || !k || !d_row_ptr || !d_col_idx || B <= 0 || H <= 0 || N <= 0 || d <= 0 || Bq <= 0 || Bk <= 0 ||
        topk <= 0)
        return SALAD_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k)) return SALAD_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || Bq > 1024 || Bk > 1024) return SALAD_ERR_UNSUPPORTED;
    const int64_t BH = int64_t(B) * H;
    const int64_t nQb = (int64_t(N) + Bq - 1) / Bq, nKb = (int64_t(N) + Bk - 1) / Bk;
    const int64_t kk = topk < nKb ? topk : nKb;
    const int64_t rows = BH * nQb;
    if (BH > 65535 || nQb > 65535 * int64_t(kScoreRows) || rows * kk > 2147483647ll) return SALAD_ERR_UNSUPPORTED;
    if (col_capacity < rows * kk) return SALAD_ERR_CAPACITY;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0 ||
        workspace_bytes < salad_topk_workspace_bytes(B, H, N, d, Bq, Bk))
        return SALAD_ERR_WORKSPACE;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int ldk = int((nKb + kScoreTile - 1) / kScoreTile * kScoreTile);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    float* qmean = reinterpret_cast<float*>(ws);
    float* kmeanT = reinterpret_cast<float*>(ws + align_up(size_t(BH) * nQb * d * 4));
    uint32_t* score = reinterpret_cast<uint32_t*>(ws + align_up(size_t(BH) * nQb * d * 4) +
                                                  align_up(size_t(BH) * d * ldk * 4));
    MeanJob jq{static_cast<const uint4*>(q), qmean, Bq, int(nQb), 0};
    MeanJob jk{static_cast<const uint4*>(k), kmeanT, Bk, int(nKb), ldk};
    block_mean_kernel<<<dim3(unsigned(nQb > nKb ? nQb : nKb), unsigned(BH), 2), kMeanThreads, 0, st>>>(jq, jk, N, d);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    const size_t smem = kScoreSmemBytes;
    launch_dependent(topk_score_kernel, dim3(unsigned(ldk / kScoreTile), unsigned((nQb + kScoreRows - 1) / kScoreRows),
                                             unsigned(BH)),
                     dim3(128), smem, st, qmean, kmeanT, int(nQb), int(nKb), ldk, d, score);
    if (check_launch() != SALAD_OK) return SALAD_ERR_CUDA;
    const dim3 pgrid(unsigned((rows + 7) / 8));
    // a CTA per row while the row fits the threads' registers; the warp-per-two-rows kernel beyond that
    if (nKb <= 512 && rows <= 2147483647ll)
        launch_dependent(topk_pick_row_kernel<4>, dim3(unsigned(rows)), dim3(128), 0, st, score, int(nKb), int(kk), d_row_ptr, d_col_idx, rows);
    else if (nKb <= 1024 && rows <= 2147483647ll)
        launch_dependent(topk_pick_row_kernel<8>, dim3(unsigned(rows)), dim3(128), 0, st, score, int(nKb), int(kk), d_row_ptr, d_col_idx, rows);
    else
        launch_dependent(topk_pick_kernel, pgrid, dim3(128), 0, st, score, int(nKb), int(kk), d_row_ptr, d_col_idx, rows);
    return check_launch();
}

SALAD_EXPORT int salad_permute_tokens(const void* x, void* y, int B, int H, int N, int d, int T, int Hs, int Ws,
                                      const int32_t* h_head_flags, int inverse, void* stream) {
    if (!x || !y || x == y || !h_head_flags || B <= 0 || H <= 0 || N <= 0 || T <= 0 || Hs <= 0 || Ws <= 0)
        return SALAD_ERR_INVALID_ARG;
    if (int64_t(T) * Hs * Ws != N) return SALAD_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return SALAD_ERR_INVALID_ARG;
    if ((d != 64 && d != 128) || H > kPermuteMaxHeads || int64_t(B) * H > 65535) return SALAD_ERR_UNSUPPORTED;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    PermuteParams pp{};
    pp.N = N; pp.T = T; pp.S = Hs * Ws; pp.H = H; pp.vec_per_row = d / 8; pp.inverse = inverse ? 1 : 0;
    for (int h = 0; h < H; ++h)
        if (h_head_flags[h]) pp.flag_bits[h >> 5] |= 1u << (h & 31);
    permute_tokens_kernel<<<dim3(unsigned((N + kPermuteRows - 1) / kPermuteRows), unsigned(B * H)), kPermuteThreads, 0,
                            static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4*>(x), static_cast<uint4*>(y), pp);
    return check_launch();
}

SALAD_EXPORT int salad_rope3d_table_build(int T, int Hs, int Ws, int d, float base, void* d_rope, void* stream) {
    if (!d_rope || T <= 0 || Hs <= 0 || Ws <= 0 || d <= 0 || (d & 1) || !(base > 1.f) || !isfinite(base))
        return SALAD_ERR_INVALID_ARG;
    if (!aligned16(d_rope)) return SALAD_ERR_INVALID_ARG;
    const int64_t N = int64_t(T) * Hs * Ws;
    if (N > 2147483647ll) return SALAD_ERR_UNSUPPORTED;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    RopeGeom g{};
    g.T = T; g.Hs = Hs; g.Ws = Ws; g.pairs = d / 2;
    g.p_hw = g.pairs / 3; g.p_t = g.pairs - 2 * g.p_hw;
    g.entries = N * g.pairs;
    g.log2_base = log2(double(base));
    const long long blocks = (g.entries + 255) / 256;
    if (blocks > 2147483647ll) return SALAD_ERR_UNSUPPORTED;
    rope3d_table_kernel<<<unsigned(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(g, static_cast<__half2*>(d_rope));
    return check_launch();
}

SALAD_EXPORT int salad_proj_combine_fwd(const void* o_s, const void* o_l, const void* w, const float* d_bias,
                                        const float* d_dyn_scale, void* out, int B, int H, int N, int d,
                                        int32_t* d_status, void* stream) {
    if (!o_s || !o_l || !w || !out || B <= 0 || H <= 0 || N <= 0 || d <= 0) return SALAD_ERR_INVALID_ARG;
    if (!aligned16(o_s) || !aligned16(o_l) || !aligned16(w) || !aligned16(out)) return SALAD_ERR_INVALID_ARG;
    if (out == o_l) return SALAD_ERR_INVALID_ARG;                 // the activation is re-read by other tiles
    if (d != 64 && d != 128) return SALAD_ERR_UNSUPPORTED;
    if (int64_t(B) * H > 65535 || int64_t(H) * d > 65536) return SALAD_ERR_UNSUPPORTED;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d_status && cudaMemsetAsync(d_status, 0, sizeof(int32_t), st) != cudaSuccess) { cudaGetLastError(); return SALAD_ERR_CUDA; }
    const int D = H * d;
    CUtensorMap ma, mw;
    if (!make_tmap_bf16_3d(&ma, o_l, d, N, int64_t(B) * H, ProjCfg::BM) || !make_tmap_bf16_3d(&mw, w, D, D, 1, ProjCfg::BN))
        return SALAD_ERR_CUDA;
    ProjParams pp;
    pp.B = B; pp.H = H; pp.N = N; pp.d = d; pp.D = D;
    pp.nMt = (N + ProjCfg::BM - 1) / ProjCfg::BM;
    pp.nNt = (D + ProjCfg::BN - 1) / ProjCfg::BN;
    pp.ksteps = D / ProjCfg::BK;
    pp.tiles = (long long)B * pp.nMt * pp.nNt;
    pp.o_s = static_cast<const __nv_bfloat16*>(o_s);
    pp.out = static_cast<__nv_bfloat16*>(out);
    pp.bias = d_bias; pp.s_b = d_dyn_scale; pp.status = d_status;
    // CTA pairs on 256 x 256 tiles (one pair per TPC) when the problem has at least a pair's worth of rows.
    // (192 output columns per tile would fill the last wave of tiles better at the 1.3B width: 13.8 waves instead
    // of 10.4; measured slower, 1048 against 1161 TFLOP/s: the narrower product costs more than the tail.)
    const char* force_single = getenv("SALAD_PROJ_SINGLE");
    if (dev.sms >= 2 && N > 128 && !(force_single && force_single[0] == '1')) {
        const long long pairs_dev = dev.sms / 2, mt2 = (long long)B * ((N + 255) / 256);
        constexpr int bn = 256;
        const long long tiles2 = mt2 * ((D + bn - 1) / bn);
        CUtensorMap ma2, mw2;
        if (!make_tmap_bf16_3d(&ma2, o_l, d, N, int64_t(B) * H, 128) || !make_tmap_bf16_3d(&mw2, w, D, D, 1, bn / 2))
            return SALAD_ERR_CUDA;
        const long long pairs = pairs_dev < tiles2 ? pairs_dev : tiles2;
        SALAD_LOGF("salad_proj_gemm_pair_kernel<%d> grid %lld (clusters of 2) block %d", bn, 2 * pairs, Proj2Cfg<256>::THREADS);
        salad_proj_gemm_pair_kernel<256><<<unsigned(2 * pairs), Proj2Cfg<256>::THREADS, Proj2Cfg<256>::SMEM_BYTES, st>>>(ma2, mw2, pp);
        return check_launch();
    }
    const unsigned grid = unsigned(pp.tiles < dev.sms ? pp.tiles : dev.sms);
    SALAD_LOGF("salad_proj_gemm_kernel grid %u block %d smem %d", grid, ProjCfg::THREADS, ProjCfg::SMEM_BYTES);
    salad_proj_gemm_kernel<<<grid, ProjCfg::THREADS, ProjCfg::SMEM_BYTES, st>>>(ma, mw, pp);
    return check_launch();
}

SALAD_EXPORT int salad_selftest_bounded_wait(int32_t* d_status, unsigned long long* d_waited_ns, void* stream) {
    if (!d_status) return SALAD_ERR_INVALID_ARG;
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(d_status, d_waited_ns);
    return check_launch();
}

SALAD_EXPORT int salad_linear_attn_fwd_noalloc(const void* q, const void* k, const void* v, void* o_l,
                                               float* kv_out, float* z_out, int B, int H, int N, int d,
                                               float eps, int32_t* d_status, void* stream) {
    if (!q || !k || !v || !o_l) return SALAD_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || d <= 0) return SALAD_ERR_INVALID_ARG;
    if (!(eps >= 0.f) || !isfinite(eps)) return SALAD_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o_l)) return SALAD_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return SALAD_ERR_UNSUPPORTED;
    if (int64_t(B) * H > SALAD_NOALLOC_MAX_HEADS) return SALAD_ERR_UNSUPPORTED;   // beyond the fixed scratch
    DeviceInfo dev{};
    int rc = prepare_device(&dev);
    if (rc != SALAD_OK) return rc;
    void* scratch = nullptr;
    rc = noalloc_scratch_ptr(&scratch);
    if (rc != SALAD_OK) return rc;
    const Workspace w = carve_noalloc(B, H, d);
    if (w.total > kNoAllocBytes) return SALAD_ERR_UNSUPPORTED;

    Problem P{};
    P.drop_tau = -INFINITY;
    P.q = q; P.k = k; P.v = v; P.o = o_l;
    P.B = B; P.H = H; P.N = N; P.d = d; P.Bq = 128; P.Bk = 64; P.Hm = 1; P.mode = MODE_LINEAR;
    P.eps = eps; P.kv_out = kv_out; P.z_out = z_out;
    P.ws = scratch; P.ws_bytes = kNoAllocBytes; P.d_status = d_status;
    P.stream = static_cast<cudaStream_t>(stream);
    // (the array keeps the last call's contents: the state kernel, first of the call, clears the status words)
    rc = (d == 128) ? launch_state<128>(P, w, dev) : launch_state<64>(P, w, dev);
    if (rc != SALAD_OK) return rc;
    return (d == 128) ? launch_apply<128>(P, w, dev) : launch_apply<64>(P, w, dev);
}
