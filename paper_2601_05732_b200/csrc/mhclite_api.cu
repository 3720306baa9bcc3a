// C ABI of the library: argument validation, workspace planning and kernel sequencing.
#include <stdarg.h>
#include <new>

#include "common.cuh"
#include "kernels.h"

namespace mhcl {

int fail(mhclite_ctx* ctx, int status, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return status;
}

int check_cuda(mhclite_ctx* ctx, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return MHCLITE_OK;
    return fail(ctx, MHCLITE_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

Workspace plan_workspace(int n, int C, int64_t T, int N, void* base, int sm_count) {
    Workspace w;
    w.Npad = round_up(N, 8);
    char* p = (char*)base;
    size_t off = 0;
    w.e = (float*)(p + off);     off += align256((size_t)T * w.Npad * sizeof(float));
    w.kappa = (float*)(p + off); off += align256((size_t)T * sizeof(float));
    w.G = (float*)(p + off);     off += align256((size_t)n * C * w.Npad * sizeof(float));
    w.dH_pre = (float*)(p + off); off += align256((size_t)T * n * sizeof(float));
    const ProjPlan pp = plan_proj(n, C, T, N, sm_count);     // sizes do not depend on the SM count
    w.Wp = p + off;              off += align256((size_t)pp.ksteps * pp.NT * 32 * 16);
    w.qpart = (float*)(p + off); off += align256((size_t)kMaxKSplit * T * pp.Npad * sizeof(float));
    w.ssq = (float*)(p + off);   off += align256((size_t)kMaxKSplit * T * sizeof(float));
    const TailPlan tp = plan_tail(n, C, T, N, sm_count);      // the token ranges (G partials) do
    const size_t erows = (size_t)round_up64(T, kEGranule);
    w.ehi = p + off;             off += align256(erows * tp.Kp * 2);
    w.elo = p + off;             off += align256(erows * tp.Kp * 2);
    int gparts = tp.supported ? tp.splits : (tp.tc ? tp.g_splits : 0);
    if (tp.ftc && tp.f_splits > gparts) gparts = tp.f_splits;
    w.Gpart = (float*)(p + off); off += align256((size_t)gparts * n * C * tp.Kp * sizeof(float));
    w.Wt = p + off;              off += align256((size_t)2 * proj_tc_nq(N) * pp.nchunks * 64 * 2);
    w.Wb = p + off;              off += align256((tp.tc || tp.ftc) ? tail_wb_bytes(n, C, tp.Kp) : 0);
    w.dpart = (float*)(p + off); off += align256((size_t)kMaxParts * kPartStride * sizeof(float));
    w.status = (int*)(p + off);  off += 256;
    w.bytes = off;
    return w;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Makes the context's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) { err = cudaSetDevice(dev); switched = (err == cudaSuccess); }
    }
    ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

}  // namespace mhcl

using namespace mhcl;

#define MHCL_REQUIRE_CTX(ctx)  do { if (!(ctx)) return MHCLITE_ERR_BAD_ARG; (ctx)->err[0] = 0; } while (0)
#define MHCL_REQUIRE_T(ctx, T) do { if ((T) < 0) return fail(ctx, MHCLITE_ERR_BAD_ARG, "T < 0"); } while (0)
#define MHCL_PTR(ctx, p)                                                                            \
    do {                                                                                            \
        if (!(p)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "null pointer: %s", #p);                    \
        if (!aligned16(p)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "pointer not 16-byte aligned: %s", #p); \
    } while (0)
#define MHCL_OPT_PTR(ctx, p)                                                                        \
    do {                                                                                            \
        if ((p) && !aligned16(p)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "pointer not 16-byte aligned: %s", #p); \
    } while (0)
// An output that aliases an input is refused: the kernels read activations through the read-only path and by TMA.
#define MHCL_NO_ALIAS(ctx, out, in)                                                                 \
    do {                                                                                            \
        if ((const void*)(out) == (const void*)(in))                                                \
            return fail(ctx, MHCLITE_ERR_BAD_ARG, "%s must not alias %s", #out, #in);               \
    } while (0)
#define MHCL_DEVICE(ctx)                                                                            \
    DeviceGuard guard_((ctx)->device);                                                              \
    if (guard_.err != cudaSuccess) return check_cuda(ctx, guard_.err, "cudaSetDevice")
#define MHCL_LAUNCH_CHECK(ctx, what) do { int rc_ = check_cuda(ctx, cudaGetLastError(), what); if (rc_) return rc_; } while (0)

static int need_workspace(mhclite_ctx* ctx, int64_t T, int kind, Workspace* w) {
    const size_t need = plan_workspace(ctx->n, ctx->C, T, ctx_cols(ctx, kind), nullptr, ctx->sm_count).bytes;
    if (!ctx->ws || ctx->ws_bytes < need)
        return fail(ctx, MHCLITE_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu attached", need, ctx->ws ? ctx->ws_bytes : (size_t)0);
    *w = plan_workspace(ctx->n, ctx->C, T, ctx_cols(ctx, kind), ctx->ws, ctx->sm_count);
    // status words of the workspace (status + four words describing the first report), at its very end,
    // cleared when first used
    w->status = (int*)((char*)ctx->ws + ((ctx->ws_bytes - 32) & ~(size_t)255));
    if (ctx->status_word != w->status) {
        DeviceGuard g(ctx->device);
        if (cudaMemset(w->status, 0, 32) != cudaSuccess) return fail(ctx, MHCLITE_ERR_CUDA, "clearing the status word");
        ctx->status_word = w->status;
    }
    return MHCLITE_OK;
}

// RMSNorm statistics + projection partials of every entry point's forward: tcgen05 / TMA kernel when the
// padded projection has at most 256 columns (hi and lo halves of W' side by side while they fit one instruction,
// as two instructions into one accumulator beyond that), the mma.sync kernel otherwise.
static int proj_forward(mhclite_ctx* ctx, int64_t T, int N, const Workspace& w, const ProjPlan& pp, const mhclite_bf16* x,
                        const float* W, const float* gain, cudaStream_t s) {
    if (proj_tc_supported(ctx->n, ctx->C, N)) {
        launch_pack_wt(ctx, pp, N, W, gain, w.Wt, s);
        MHCL_LAUNCH_CHECK(ctx, "pack_wt");
        if (launch_proj_fwd_tc(ctx, T, N, pp, x, w.Wt, w.qpart, w.ssq, w.status, s)) {
            MHCL_LAUNCH_CHECK(ctx, "proj_fwd_tc");
            return MHCLITE_OK;
        }
    }
    launch_pack_w(ctx, pp, N, W, gain, w.Wp, s);
    MHCL_LAUNCH_CHECK(ctx, "pack_w");
    launch_proj_fwd_mma(ctx, T, pp, x, w.Wp, w.qpart, w.ssq, s);
    MHCL_LAUNCH_CHECK(ctx, "proj_fwd_mma");
    return MHCLITE_OK;
}

// True when the activation backward must leave e as the tiled bf16 pair (a tensor-core kernel reads it).
static bool tail_pair(const TailPlan& tp) { return tp.supported || (tp.tc && tensor_maps_available()); }

// The part of the backward shared by every entry point, after the activation backward has produced e and
// kappa: projection / RMSNorm backward into dx (fused with H_res^T g + H_pre du when g is given) and the
// parameter gradients dW, dgain.  Tensor cores when the projection is narrow enough, CUDA cores otherwise.
static int proj_backward(mhclite_ctx* ctx, int64_t T, int N, const Workspace& w, const TailPlan& tp,
                         const mhclite_bf16* x, const mhclite_bf16* g, const mhclite_bf16* du, const float* H_res,
                         const float* H_pre, const float* W, const float* gain, bool wf_packed, mhclite_bf16* dx,
                         int accumulate_dx, float* dW, float* dgain, int accumulate_params, cudaStream_t s,
                         const float* dpart = nullptr, int nparts = 0, float* db = nullptr, float* dalpha = nullptr) {
    // dpart: db and dalpha were left as nparts per-block partials by the activation backward
    if (tp.ftc && launch_tail_ftc(ctx, T, N, tp, x, g, du, w.ehi, w.elo, w.kappa, H_res, H_pre, W, gain, w.Wb, wf_packed,
                                  dx, accumulate_dx, w.Gpart, w.status, s)) {
        MHCL_LAUNCH_CHECK(ctx, "tail_ftc");
        ctx->launches += 1;
        launch_tail_finish(ctx, N, tp.Kp, tp.f_splits, W, gain, w.Gpart, dW, dgain, accumulate_params, s, dpart, nparts, db,
                           dalpha);
        MHCL_LAUNCH_CHECK(ctx, "tail_finish");
        return MHCLITE_OK;
    }
    if (dpart) {
        launch_dpart_sum(ctx, N, dpart, nparts, db, dalpha, accumulate_params, s);
        MHCL_LAUNCH_CHECK(ctx, "dpart_sum");
    }
    if (tp.supported) {
        launch_tail_mma(ctx, T, N, tp, x, g, du, w.ehi, w.elo, w.kappa, H_res, H_pre, W, gain, dx, accumulate_dx,
                        w.Gpart, dW, dgain, accumulate_params, s);
        MHCL_LAUNCH_CHECK(ctx, "tail_mma");
        return MHCLITE_OK;
    }
    bool dx_done = false;
    if (tail_pair(tp)) {
        dx_done = launch_tail_dx_tc(ctx, T, N, tp, x, g, du, w.ehi, w.kappa, H_res, H_pre, W, gain, w.Wb, dx,
                                    accumulate_dx, w.status, s);
        if (dx_done) MHCL_LAUNCH_CHECK(ctx, "tail_dx_tc");
    }
    if (!dx_done && g) {
        launch_tail_mix(ctx, T, x, g, du, H_res, H_pre, nullptr, dx, s);
        MHCL_LAUNCH_CHECK(ctx, "tail_mix");
        accumulate_dx = 1;
    }
    if (!dx_done) {
        launch_proj_bwd_dx(ctx, T, N, w.Npad, x, W, gain, w.e, w.kappa, dx, accumulate_dx, s);
        MHCL_LAUNCH_CHECK(ctx, "proj_bwd_dx");
    }
    if (tail_pair(tp) && launch_tail_g_tc(ctx, T, tp, x, w.ehi, w.elo, w.Gpart, w.status, s)) {
        MHCL_LAUNCH_CHECK(ctx, "tail_g_tc");
        ctx->launches += 1;
        launch_tail_finish(ctx, N, tp.Kp, tp.g_splits, W, gain, w.Gpart, dW, dgain, accumulate_params, s);
        MHCL_LAUNCH_CHECK(ctx, "tail_finish");
        return MHCLITE_OK;
    }
    launch_proj_bwd_dw(ctx, T, N, w.Npad, x, W, gain, w.e, w.G, dW, dgain, accumulate_params, s);
    MHCL_LAUNCH_CHECK(ctx, "proj_bwd_dw");
    return MHCLITE_OK;
}

extern "C" {

const char* mhclite_status_string(int status) {
    switch (status) {
        case MHCLITE_OK: return "ok";
        case MHCLITE_ERR_BAD_ARG: return "bad argument";
        case MHCLITE_ERR_CUDA: return "CUDA error";
        case MHCLITE_ERR_WORKSPACE: return "workspace missing or too small";
        case MHCLITE_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

const char* mhclite_last_error(const mhclite_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int mhclite_create(mhclite_ctx** out, int n, int C, int device) {
    if (!out) return MHCLITE_ERR_BAD_ARG;
    *out = nullptr;
    if (n < 2 || n > kMaxN || C <= 0 || (C % 8) != 0 || device < 0) return MHCLITE_ERR_BAD_ARG;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device >= count) return MHCLITE_ERR_CUDA;
    mhclite_ctx* ctx = new (std::nothrow) mhclite_ctx();
    if (!ctx) return MHCLITE_ERR_CUDA;
    ctx->n = n; ctx->C = C; ctx->device = device; ctx->nfact = ipow_fact(n); ctx->table_dev = nullptr;
    ctx->pending_T = -1; ctx->pending_x = nullptr;
    ctx->ws = nullptr; ctx->ws_bytes = 0; ctx->err[0] = 0; ctx->launches = 0; ctx->timing = false; ctx->status_word = nullptr;
    for (int k = 0; k < MHCLITE_KERNEL_COUNT; ++k) { ctx->ev[k][0] = ctx->ev[k][1] = nullptr; ctx->ev_recorded[k] = false; }
    ctx->copy_in = ctx->copy_out = nullptr; ctx->ev_fork = ctx->ev_join = nullptr;
    for (int k = 0; k < MHCLITE_STEP_CHUNKS; ++k) ctx->ev_in[k] = ctx->ev_cmp[k] = nullptr;
    {
        DeviceGuard g(device);
        cudaError_t e = g.err;
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
        for (int k = 2; k <= kMaxN && e == cudaSuccess; ++k) e = upload_perm_tables(k);
        if (e != cudaSuccess) { delete ctx; return MHCLITE_ERR_CUDA; }
    }
    *out = ctx;
    return MHCLITE_OK;
}

int mhclite_destroy(mhclite_ctx* ctx) {
    if (!ctx) return MHCLITE_ERR_BAD_ARG;
    for (int k = 0; k < MHCLITE_KERNEL_COUNT; ++k)
        for (int e = 0; e < 2; ++e)
            if (ctx->ev[k][e]) cudaEventDestroy(ctx->ev[k][e]);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    for (int k = 0; k < MHCLITE_STEP_CHUNKS; ++k) {
        if (ctx->ev_in[k]) cudaEventDestroy(ctx->ev_in[k]);
        if (ctx->ev_cmp[k]) cudaEventDestroy(ctx->ev_cmp[k]);
    }
    delete ctx;
    return MHCLITE_OK;
}

int mhclite_perm_table(int n, uint8_t* sigma_host) {
    if (n < 2 || n > kMaxN || !sigma_host) return MHCLITE_ERR_BAD_ARG;
    PermTables t;
    host_perm_tables(n, &t);
    memcpy(sigma_host, t.sigma, (size_t)ipow_fact(n) * n);
    return MHCLITE_OK;
}

int mhclite_perm_table_device(mhclite_ctx* ctx, uint8_t* sigma_host) {
    MHCL_REQUIRE_CTX(ctx);
    if (!sigma_host) return fail(ctx, MHCLITE_ERR_BAD_ARG, "null pointer: sigma_host");
    MHCL_DEVICE(ctx);
    return check_cuda(ctx, download_perm_sigma(ctx->n, sigma_host), "read permutation table");
}

size_t mhclite_workspace_bytes(int n, int C, int64_t T, int kind) {
    if (n < 2 || n > kMaxN || C <= 0 || T < 0 || kind < 0 || kind > 1) return 0;
    return plan_workspace(n, C, T, n_cols(n, kind), nullptr).bytes;
}

size_t mhclite_workspace_bytes_subset(int n, int C, int64_t T, int K) {
    if (n < 2 || n > kMaxN || C <= 0 || T < 0 || K < 1 || K > ipow_fact(n)) return 0;
    return plan_workspace(n, C, T, K + 2 * n, nullptr).bytes;
}

int mhclite_set_perm_subset(mhclite_ctx* ctx, int K, const uint8_t* table) {
    MHCL_REQUIRE_CTX(ctx);
    if (K == 0 || !table) {                            // back to all n! permutations
        ctx->nfact = ipow_fact(ctx->n);
        ctx->table_dev = nullptr;
        return MHCLITE_OK;
    }
    const int n = ctx->n;
    if (K < 1 || K > ipow_fact(n) || K > kMaxFact) return fail(ctx, MHCLITE_ERR_BAD_ARG, "K must be in [1, n!]");
    MHCL_DEVICE(ctx);
    uint8_t h[kMaxFact * kMaxN];
    int rc = check_cuda(ctx, cudaMemcpy(h, table, (size_t)K * n, cudaMemcpyDeviceToHost), "read permutation subset");
    if (rc) return rc;
    for (int k = 0; k < K; ++k) {
        unsigned seen = 0;
        for (int i = 0; i < n; ++i) {
            const int v = h[k * n + i];
            if (v >= n || (seen >> v & 1u)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "row %d of the table is not a permutation of 0..%d", k, n - 1);
            seen |= 1u << v;
        }
        for (int k2 = 0; k2 < k; ++k2)
            if (memcmp(h + k * n, h + k2 * n, (size_t)n) == 0)
                return fail(ctx, MHCLITE_ERR_BAD_ARG, "row %d of the table repeats row %d", k, k2);
    }
    memcpy(ctx->table_host, h, (size_t)K * n);
    ctx->table_dev = table;
    ctx->nfact = K;
    return MHCLITE_OK;
}

int mhclite_set_workspace(mhclite_ctx* ctx, void* workspace, size_t bytes) {
    MHCL_REQUIRE_CTX(ctx);
    if (workspace && ((uintptr_t)workspace & 255)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "workspace not 256-byte aligned");
    ctx->ws = workspace;
    ctx->ws_bytes = workspace ? bytes : 0;
    ctx->status_word = nullptr;
    return MHCLITE_OK;
}

// ---- forward -------------------------------------------------------------------------------------
int mhclite_coeffs_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* b,
                       const float* alpha, const float* gain, float eps, float* H_res, float* H_pre, float* H_post,
                       float* a_saved, float* p_saved, float* rstd, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W); MHCL_PTR(ctx, b); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, a_saved);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd);
    if (!(eps >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps must be >= 0");
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    const ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    rc = proj_forward(ctx, T, N, w, pp, x, W, gain, s);
    if (rc) return rc;
    launch_lite_act_fwd(ctx, T, pp, w.qpart, w.ssq, eps, b, alpha, H_res, H_pre, H_post, a_saved, p_saved, rstd, s);
    MHCL_LAUNCH_CHECK(ctx, "lite_act_fwd");
    return MHCLITE_OK;
}

int mhclite_premix_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* H_pre, mhclite_bf16* u,
                       void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, u);
    MHCL_NO_ALIAS(ctx, u, x);
    MHCL_DEVICE(ctx);
    launch_premix_fwd(ctx, T, x, H_pre, u, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "premix_fwd");
    return MHCLITE_OK;
}

int mhclite_postres_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const mhclite_bf16* y, const float* H_res,
                        const float* H_post, mhclite_bf16* x_next, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, y); MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, x_next);
    MHCL_NO_ALIAS(ctx, x_next, x); MHCL_NO_ALIAS(ctx, x_next, y);
    MHCL_DEVICE(ctx);
    launch_postres_fwd(ctx, T, x, y, H_res, H_post, x_next, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "postres_fwd");
    return MHCLITE_OK;
}

static int pre_fwd_fused_impl(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* b,
                              const float* alpha, const float* gain, float eps, float* H_res, float* H_pre, float* H_post,
                              float* a_saved, float* p_saved, float* rstd, mhclite_bf16* u, float* u_rstd, float eps_u,
                              void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W); MHCL_PTR(ctx, b); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, a_saved);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, u);
    MHCL_NO_ALIAS(ctx, u, x);
    if (!(eps >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps must be >= 0");
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    const ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    rc = proj_forward(ctx, T, N, w, pp, x, W, gain, s);
    if (rc) return rc;
    launch_lite_act_premix(ctx, T, pp, w.qpart, w.ssq, eps, b, alpha, H_res, H_pre, H_post, a_saved, p_saved, rstd, x, u, s,
                           u_rstd, eps_u);
    MHCL_LAUNCH_CHECK(ctx, "lite_act_premix");
    return MHCLITE_OK;
}

int mhclite_pre_fwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* b,
                          const float* alpha, const float* gain, float eps, float* H_res, float* H_pre, float* H_post,
                          float* a_saved, float* p_saved, float* rstd, mhclite_bf16* u, void* stream) {
    return pre_fwd_fused_impl(ctx, T, x, W, b, alpha, gain, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd, u, nullptr,
                              0.f, stream);
}

int mhclite_pre_fwd_fused_ustat(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* b,
                                const float* alpha, const float* gain, float eps, float* H_res, float* H_pre,
                                float* H_post, float* a_saved, float* p_saved, float* rstd, mhclite_bf16* u,
                                float* u_rstd, float eps_u, void* stream) {
    if (!ctx) return MHCLITE_ERR_BAD_ARG;
    if (!u_rstd || ((uintptr_t)u_rstd & 15) != 0) return fail(ctx, MHCLITE_ERR_BAD_ARG, "u_rstd: null or not 16-byte aligned");
    if (!(eps_u >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps_u must be >= 0");
    return pre_fwd_fused_impl(ctx, T, x, W, b, alpha, gain, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd, u, u_rstd,
                              eps_u, stream);
}

// One K slice covering all of n*C: the plan of projection partials that a single kernel produced per token tile.
static ProjPlan whole_k_plan(const mhclite_ctx* ctx, int64_t T, int N) {
    ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    pp.ksplit = 1;
    pp.chunks_per_split = pp.nchunks;
    return pp;
}

int mhclite_postres_fwd_next_proj(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const mhclite_bf16* y,
                                  const float* H_res, const float* H_post, mhclite_bf16* x_next, const float* W_next,
                                  const float* gain_next, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    ctx->pending_T = -1;
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, y); MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, x_next);
    MHCL_PTR(ctx, W_next); MHCL_PTR(ctx, gain_next);
    if ((const void*)x_next == (const void*)x) return fail(ctx, MHCLITE_ERR_BAD_ARG, "x_next must not alias x");
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    if (postres_proj_supported(ctx->n, ctx->C, N)) {
        const ProjPlan pp = whole_k_plan(ctx, T, N);
        launch_pack_wt(ctx, pp, N, W_next, gain_next, w.Wt, s);
        MHCL_LAUNCH_CHECK(ctx, "pack_wt");
        if (launch_postres_proj(ctx, T, N, pp, x, y, H_res, H_post, x_next, w.Wt, w.qpart, w.ssq, w.status, s)) {
            MHCL_LAUNCH_CHECK(ctx, "postres_proj");
            ctx->pending_T = T; ctx->pending_x = x_next; ctx->pending_ksplit = 1;
            return MHCLITE_OK;
        }
    }
    // shapes the fused kernel does not take: the merge, then the projection of the next layer as usual
    launch_postres_fwd(ctx, T, x, y, H_res, H_post, x_next, s);
    MHCL_LAUNCH_CHECK(ctx, "postres_fwd");
    const ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    rc = proj_forward(ctx, T, N, w, pp, x_next, W_next, gain_next, s);
    if (rc) return rc;
    ctx->pending_T = T; ctx->pending_x = x_next; ctx->pending_ksplit = pp.ksplit;
    return MHCLITE_OK;
}

int mhclite_pre_fwd_resume(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* b, const float* alpha,
                           float eps, float* H_res, float* H_pre, float* H_post, float* a_saved, float* p_saved,
                           float* rstd, mhclite_bf16* u, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, b); MHCL_PTR(ctx, alpha);
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, a_saved);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, u);
    if (!(eps >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps must be >= 0");
    if (ctx->pending_T != T || ctx->pending_x != (const void*)x)
        return fail(ctx, MHCLITE_ERR_BAD_ARG, "no projection partials of this x are pending: call "
                                              "mhclite_postres_fwd_next_proj(..., x_next = x, ...) on this context first");
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    if (ctx->pending_ksplit == 1) pp = whole_k_plan(ctx, T, N);
    ctx->pending_T = -1;
    launch_lite_act_premix(ctx, T, pp, w.qpart, w.ssq, eps, b, alpha, H_res, H_pre, H_post, a_saved, p_saved, rstd, x, u, s);
    MHCL_LAUNCH_CHECK(ctx, "lite_act_premix");
    return MHCLITE_OK;
}

// ---- backward ------------------------------------------------------------------------------------
int mhclite_postres_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const mhclite_bf16* y, const float* H_res,
                        const float* H_post, const mhclite_bf16* g, mhclite_bf16* dy, float* dH_res, float* dH_post,
                        mhclite_bf16* dx, int accumulate_dx, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, y); MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, g);
    MHCL_PTR(ctx, dy); MHCL_PTR(ctx, dH_res); MHCL_PTR(ctx, dH_post); MHCL_OPT_PTR(ctx, dx);
    MHCL_NO_ALIAS(ctx, dy, y); MHCL_NO_ALIAS(ctx, dy, g); MHCL_NO_ALIAS(ctx, dy, x);
    if (dx) { MHCL_NO_ALIAS(ctx, dx, x); MHCL_NO_ALIAS(ctx, dx, g); }
    MHCL_DEVICE(ctx);
    launch_postres_bwd(ctx, T, x, y, H_res, H_post, g, dy, dH_res, dH_post, dx, accumulate_dx, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "postres_bwd");
    return MHCLITE_OK;
}

int mhclite_premix_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* H_pre, const mhclite_bf16* du,
                       float* dH_pre, mhclite_bf16* dx, int accumulate_dx, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, du); MHCL_PTR(ctx, dH_pre); MHCL_OPT_PTR(ctx, dx);
    if (dx) MHCL_NO_ALIAS(ctx, dx, x);
    MHCL_DEVICE(ctx);
    launch_premix_bwd(ctx, T, x, H_pre, du, dH_pre, dx, accumulate_dx, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "premix_bwd");
    return MHCLITE_OK;
}

// The fused backward tails that end in tail_ftc_k leave db and dalpha as per-block partials in their first kernel
// (dH_pre + activation backward); tail_finish_k adds them up in a fixed order.  Nothing has to be cleared first,
// and the sums do not depend on the order in which blocks finish.  True when that route is open: W' has then been
// packed for tail_ftc_k.  (Packing on a second stream while the first kernel runs was measured: no gain.)
static bool part_pack(mhclite_ctx* ctx, int N, const TailPlan& tp, const Workspace& w, const float* W, const float* gain,
                      cudaStream_t s) {
    if (!tp.ftc || !tensor_maps_available() || ctx->sm_count * 16 > kMaxParts) return false;
    return launch_tail_ftc_prep(ctx, N, tp, W, gain, w.Wb, nullptr, nullptr, s);
}

// Zeroes the parameter-gradient accumulators that the kernels add into, unless the caller accumulates.  When
// the backward ends in the fused tcgen05 tail, the kernel that packs W' for it does the zeroing as well
// (*wf_packed tells proj_backward that W' is ready).
static int prep_param_grads(mhclite_ctx* ctx, int N, const TailPlan& tp, const Workspace& w, const float* W,
                            const float* gain, float* db, float* dalpha, int accumulate, cudaStream_t s,
                            bool* wf_packed) {
    *wf_packed = launch_tail_ftc_prep(ctx, N, tp, W, gain, w.Wb, accumulate ? nullptr : db, accumulate ? nullptr : dalpha, s);
    if (*wf_packed) return check_cuda(ctx, cudaGetLastError(), "pack_wf");
    if (accumulate) return MHCLITE_OK;
    int rc = check_cuda(ctx, cudaMemsetAsync(db, 0, (size_t)N * sizeof(float), s), "memset db");
    if (rc) return rc;
    return check_cuda(ctx, cudaMemsetAsync(dalpha, 0, 3 * sizeof(float), s), "memset dalpha");
}

int mhclite_coeffs_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* alpha,
                       const float* gain, float eps, const float* a_saved, const float* p_saved, const float* rstd,
                       const float* H_pre, const float* H_post, const float* dH_res, const float* dH_pre,
                       const float* dH_post, mhclite_bf16* dx, int accumulate_dx, float* dW, float* db, float* dalpha,
                       float* dgain, int accumulate_params, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    (void)eps;
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain); MHCL_PTR(ctx, a_saved);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, dH_res);
    MHCL_PTR(ctx, dH_pre); MHCL_PTR(ctx, dH_post); MHCL_PTR(ctx, dx); MHCL_PTR(ctx, dW); MHCL_PTR(ctx, db);
    MHCL_PTR(ctx, dalpha); MHCL_PTR(ctx, dgain);
    MHCL_NO_ALIAS(ctx, dx, x); MHCL_NO_ALIAS(ctx, dW, W);
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    const TailPlan tp = plan_tail(ctx->n, ctx->C, T, N, ctx->sm_count);
    bool wf_packed = false;
    rc = prep_param_grads(ctx, N, tp, w, W, gain, db, dalpha, accumulate_params, s, &wf_packed);
    if (rc) return rc;
    launch_lite_act_bwd(ctx, T, w.Npad, a_saved, p_saved, rstd, alpha, H_pre, H_post, dH_res, dH_pre, dH_post,
                        tp.supported ? nullptr : w.e, tail_pair(tp) ? w.ehi : nullptr, w.elo, tp.Kp, w.kappa, db, dalpha, s);
    MHCL_LAUNCH_CHECK(ctx, "lite_act_bwd");
    return proj_backward(ctx, T, N, w, tp, x, nullptr, nullptr, nullptr, nullptr, W, gain, wf_packed, dx, accumulate_dx, dW, dgain,
                         accumulate_params, s);
}

int mhclite_tail_bwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* alpha,
                           const float* gain, float eps, const float* a_saved, const float* p_saved, const float* rstd,
                           const float* H_res, const float* H_pre, const float* H_post, const mhclite_bf16* g,
                           const mhclite_bf16* du, const float* dH_res, const float* dH_post, mhclite_bf16* dx,
                           float* dW, float* db, float* dalpha, float* dgain, int accumulate_params, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    (void)eps; (void)H_post;
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain); MHCL_PTR(ctx, a_saved);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post);
    MHCL_PTR(ctx, g); MHCL_PTR(ctx, du); MHCL_PTR(ctx, dH_res); MHCL_PTR(ctx, dH_post); MHCL_PTR(ctx, dx);
    MHCL_PTR(ctx, dW); MHCL_PTR(ctx, db); MHCL_PTR(ctx, dalpha); MHCL_PTR(ctx, dgain);
    MHCL_NO_ALIAS(ctx, dx, x); MHCL_NO_ALIAS(ctx, dx, g); MHCL_NO_ALIAS(ctx, dW, W);
    Workspace w;
    int rc = need_workspace(ctx, T, 0, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 0);
    const TailPlan tp = plan_tail(ctx->n, ctx->C, T, N, ctx->sm_count);
    bool wf_packed = false;
    // (the partials are written by the n <= 4 kernel of a context without a permutation subset)
    const bool part = ctx->n <= 4 && !ctx->table_dev && part_pack(ctx, N, tp, w, W, gain, s);
    if (part) {
        wf_packed = true;
    } else {
        rc = prep_param_grads(ctx, N, tp, w, W, gain, db, dalpha, accumulate_params, s, &wf_packed);
        if (rc) return rc;
    }
    const int nparts = launch_lite_tailpre(ctx, T, x, du, a_saved, p_saved, rstd, alpha, H_pre, H_post, dH_res, dH_post,
                                           w.dH_pre, tp.supported ? nullptr : w.e, w.Npad, tail_pair(tp) ? w.ehi : nullptr,
                                           w.elo, tp.Kp, w.kappa, part ? w.dpart : db, part ? nullptr : dalpha, s);
    MHCL_LAUNCH_CHECK(ctx, "lite_tailpre");
    return proj_backward(ctx, T, N, w, tp, x, g, du, H_res, H_pre, W, gain, wf_packed, dx, 0, dW, dgain, accumulate_params, s,
                         part ? w.dpart : nullptr, nparts, db, dalpha);
}

// ---- SK comparison path --------------------------------------------------------------------------
int mhc_sk20_coeffs_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W_sk, const float* b_sk,
                        const float* alpha, const float* gain, float eps, int iters, float* H_res, float* H_pre,
                        float* H_post, float* p_saved, float* rstd, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (iters < 1 || iters > 64) return fail(ctx, MHCLITE_ERR_BAD_ARG, "iters must be in [1,64]");
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W_sk); MHCL_PTR(ctx, b_sk); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd);
    if (!(eps >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps must be >= 0");
    Workspace w;
    int rc = need_workspace(ctx, T, 1, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 1);
    const ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    rc = proj_forward(ctx, T, N, w, pp, x, W_sk, gain, s);
    if (rc) return rc;
    launch_sk_act_fwd(ctx, T, iters, pp, w.qpart, w.ssq, eps, b_sk, alpha, H_res, H_pre, H_post, p_saved, rstd, s);
    MHCL_LAUNCH_CHECK(ctx, "sk_act_fwd");
    return MHCLITE_OK;
}

int mhc_sk20_pre_fwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W_sk, const float* b_sk,
                           const float* alpha, const float* gain, float eps, int iters, float* H_res, float* H_pre,
                           float* H_post, float* p_saved, float* rstd, mhclite_bf16* u, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (iters < 1 || iters > 64) return fail(ctx, MHCLITE_ERR_BAD_ARG, "iters must be in [1,64]");
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W_sk); MHCL_PTR(ctx, b_sk); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd);
    MHCL_PTR(ctx, u);
    if (!(eps >= 0.f)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "eps must be >= 0");
    Workspace w;
    int rc = need_workspace(ctx, T, 1, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 1);
    const ProjPlan pp = plan_proj(ctx->n, ctx->C, T, N, ctx->sm_count);
    rc = proj_forward(ctx, T, N, w, pp, x, W_sk, gain, s);
    if (rc) return rc;
    launch_sk_act_premix(ctx, T, iters, pp, w.qpart, w.ssq, eps, b_sk, alpha, H_res, H_pre, H_post, p_saved, rstd, x, u, s);
    MHCL_LAUNCH_CHECK(ctx, "sk_act_premix");
    return MHCLITE_OK;
}

int mhc_sk20_coeffs_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W_sk, const float* b_sk,
                        const float* alpha, const float* gain, float eps, int iters, const float* p_saved,
                        const float* rstd, const float* H_pre, const float* H_post, const float* dH_res,
                        const float* dH_pre, const float* dH_post, mhclite_bf16* dx, int accumulate_dx, float* dW,
                        float* db, float* dalpha, float* dgain, int accumulate_params, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    (void)eps;
    if (iters < 1 || iters > 64) return fail(ctx, MHCLITE_ERR_BAD_ARG, "iters must be in [1,64]");
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W_sk); MHCL_PTR(ctx, b_sk); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post); MHCL_PTR(ctx, dH_res);
    MHCL_PTR(ctx, dH_pre); MHCL_PTR(ctx, dH_post); MHCL_PTR(ctx, dx); MHCL_PTR(ctx, dW); MHCL_PTR(ctx, db);
    MHCL_PTR(ctx, dalpha); MHCL_PTR(ctx, dgain);
    Workspace w;
    int rc = need_workspace(ctx, T, 1, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 1);
    const TailPlan tp = plan_tail(ctx->n, ctx->C, T, N, ctx->sm_count);
    bool wf_packed = false;
    rc = prep_param_grads(ctx, N, tp, w, W_sk, gain, db, dalpha, accumulate_params, s, &wf_packed);
    if (rc) return rc;
    launch_sk_act_bwd(ctx, T, w.Npad, iters, p_saved, b_sk, rstd, alpha, H_pre, H_post, dH_res, dH_pre, dH_post,
                      tp.supported ? nullptr : w.e, tail_pair(tp) ? w.ehi : nullptr, w.elo, tp.Kp, w.kappa, db, dalpha, s);
    MHCL_LAUNCH_CHECK(ctx, "sk_act_bwd");
    return proj_backward(ctx, T, N, w, tp, x, nullptr, nullptr, nullptr, nullptr, W_sk, gain, wf_packed, dx, accumulate_dx, dW,
                         dgain, accumulate_params, s);
}

int mhc_sk20_tail_bwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W_sk, const float* b_sk,
                            const float* alpha, const float* gain, float eps, int iters, const float* p_saved,
                            const float* rstd, const float* H_res, const float* H_pre, const float* H_post,
                            const mhclite_bf16* g, const mhclite_bf16* du, const float* dH_res, const float* dH_post,
                            mhclite_bf16* dx, float* dW, float* db, float* dalpha, float* dgain,
                            int accumulate_params, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    (void)eps;
    if (iters < 1 || iters > 64) return fail(ctx, MHCLITE_ERR_BAD_ARG, "iters must be in [1,64]");
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, x); MHCL_PTR(ctx, W_sk); MHCL_PTR(ctx, b_sk); MHCL_PTR(ctx, alpha); MHCL_PTR(ctx, gain);
    MHCL_PTR(ctx, p_saved); MHCL_PTR(ctx, rstd); MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, H_pre); MHCL_PTR(ctx, H_post);
    MHCL_PTR(ctx, g); MHCL_PTR(ctx, du); MHCL_PTR(ctx, dH_res); MHCL_PTR(ctx, dH_post); MHCL_PTR(ctx, dx);
    MHCL_PTR(ctx, dW); MHCL_PTR(ctx, db); MHCL_PTR(ctx, dalpha); MHCL_PTR(ctx, dgain);
    Workspace w;
    int rc = need_workspace(ctx, T, 1, &w);
    if (rc) return rc;
    MHCL_DEVICE(ctx);
    cudaStream_t s = (cudaStream_t)stream;
    const int N = ctx_cols(ctx, 1);
    const TailPlan tp = plan_tail(ctx->n, ctx->C, T, N, ctx->sm_count);
    bool wf_packed = false;
    const bool part = part_pack(ctx, N, tp, w, W_sk, gain, s);
    if (part) {
        wf_packed = true;
    } else {
        rc = prep_param_grads(ctx, N, tp, w, W_sk, gain, db, dalpha, accumulate_params, s, &wf_packed);
        if (rc) return rc;
    }
    const int nparts = launch_sk_tailpre(ctx, T, iters, x, du, p_saved, b_sk, rstd, alpha, H_pre, H_post, dH_res, dH_post,
                                         tp.supported ? nullptr : w.e, w.Npad, tail_pair(tp) ? w.ehi : nullptr, w.elo, tp.Kp,
                                         w.kappa, part ? w.dpart : db, part ? nullptr : dalpha, s);
    MHCL_LAUNCH_CHECK(ctx, "sk_tailpre");
    return proj_backward(ctx, T, N, w, tp, x, g, du, H_res, H_pre, W_sk, gain, wf_packed, dx, 0, dW, dgain, accumulate_params, s,
                         part ? w.dpart : nullptr, nparts, db, dalpha);
}

int mhclite_ds_gap(mhclite_ctx* ctx, int64_t T, const float* H_res, float* l1_err, float* colsum_dev, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, H_res); MHCL_OPT_PTR(ctx, l1_err); MHCL_OPT_PTR(ctx, colsum_dev);
    MHCL_DEVICE(ctx);
    launch_ds_gap(ctx, T, H_res, l1_err, colsum_dev, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "ds_gap");
    return MHCLITE_OK;
}

int mhclite_ds_gap_stats(mhclite_ctx* ctx, int64_t T, const float* H_res, float* stats, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    MHCL_PTR(ctx, stats);
    MHCL_DEVICE(ctx);
    if (T == 0) return check_cuda(ctx, cudaMemsetAsync(stats, 0, 4 * sizeof(float), (cudaStream_t)stream), "memset stats");
    MHCL_PTR(ctx, H_res);
    launch_ds_gap_stats(ctx, T, H_res, stats, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "ds_gap_stats");
    return MHCLITE_OK;
}

int mhclite_log_inv_nu_histogram(mhclite_ctx* ctx, int64_t T, const float* X, int bins, float lo, float hi,
                                 unsigned long long* hist, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (bins < 1 || bins > 4096 || !(hi > lo)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "bins must be in [1,4096] and hi > lo");
    if (!hist || ((uintptr_t)hist & 7)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "hist null or not 8-byte aligned");
    MHCL_DEVICE(ctx);
    if (T == 0)
        return check_cuda(ctx, cudaMemsetAsync(hist, 0, (size_t)(bins + 1) * 8, (cudaStream_t)stream), "memset hist");
    MHCL_PTR(ctx, X);
    launch_log_inv_nu_hist(ctx, T, X, bins, lo, hi, hist, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "log_inv_nu_hist");
    return MHCLITE_OK;
}

int mhclite_depth_product(mhclite_ctx* ctx, int64_t T, const float* H_res, float* P, int first, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, H_res); MHCL_PTR(ctx, P);
    if (H_res == P) return fail(ctx, MHCLITE_ERR_BAD_ARG, "H_res and P must not alias");
    MHCL_DEVICE(ctx);
    launch_depth_product(ctx, T, H_res, P, first, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "depth_product");
    return MHCLITE_OK;
}

int mhclite_relative_range(mhclite_ctx* ctx, int64_t T, const float* X, float* nu, void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    MHCL_PTR(ctx, X); MHCL_PTR(ctx, nu);
    MHCL_DEVICE(ctx);
    launch_relative_range(ctx, T, X, nu, (cudaStream_t)stream);
    MHCL_LAUNCH_CHECK(ctx, "relative_range");
    return MHCLITE_OK;
}

// ---- whole step from host buffers ----------------------------------------------------------------
namespace {
struct StepStaging {
    mhclite_bf16 *x, *y, *g, *du, *u, *x_next, *dy, *dx;
    float *H_res, *H_pre, *H_post, *a, *p, *rstd, *dH_res, *dH_post;
    size_t bytes;
};
StepStaging plan_step(int n, int C, int64_t T, void* base) {
    StepStaging s;
    char* p = (char*)base;
    size_t off = 0;
    const size_t big = (size_t)T * n * C * sizeof(mhclite_bf16), small = (size_t)T * C * sizeof(mhclite_bf16);
    const int nf = ipow_fact(n), N = n_cols(n, 0);        // sized for all n! permutations: a subset needs less
    auto take = [&](size_t b) { void* q = p + off; off += align256(b); return q; };
    s.x = (mhclite_bf16*)take(big); s.y = (mhclite_bf16*)take(small); s.g = (mhclite_bf16*)take(big);
    s.du = (mhclite_bf16*)take(small); s.u = (mhclite_bf16*)take(small); s.x_next = (mhclite_bf16*)take(big);
    s.dy = (mhclite_bf16*)take(small); s.dx = (mhclite_bf16*)take(big);
    s.H_res = (float*)take((size_t)T * n * n * 4); s.H_pre = (float*)take((size_t)T * n * 4);
    s.H_post = (float*)take((size_t)T * n * 4); s.a = (float*)take((size_t)T * nf * 4);
    s.p = (float*)take((size_t)T * N * 4); s.rstd = (float*)take((size_t)T * 4);
    s.dH_res = (float*)take((size_t)T * n * n * 4); s.dH_post = (float*)take((size_t)T * n * 4);
    s.bytes = off;
    return s;
}
}  // namespace

size_t mhclite_step_host_bytes(int n, int C, int64_t T) {
    if (n < 2 || n > kMaxN || C <= 0 || T < 0) return 0;
    return plan_step(n, C, T, nullptr).bytes;
}

int mhclite_step_host(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x_host, const mhclite_bf16* y_host,
                      const mhclite_bf16* g_host, const mhclite_bf16* du_host, const float* W, const float* b,
                      const float* alpha, const float* gain, float eps, mhclite_bf16* u_host,
                      mhclite_bf16* x_next_host, mhclite_bf16* dy_host, mhclite_bf16* dx_host, float* dW, float* db,
                      float* dalpha, float* dgain, int accumulate_params, void* staging, size_t staging_bytes,
                      void* stream) {
    MHCL_REQUIRE_CTX(ctx); MHCL_REQUIRE_T(ctx, T);
    if (T == 0) return MHCLITE_OK;
    if (!x_host || !y_host || !g_host || !du_host || !u_host || !x_next_host || !dy_host || !dx_host)
        return fail(ctx, MHCLITE_ERR_BAD_ARG, "null host pointer");
    if (!staging || ((uintptr_t)staging & 255)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "staging null or not 256-byte aligned");
    const StepStaging s = plan_step(ctx->n, ctx->C, T, staging);
    if (staging_bytes < s.bytes)
        return fail(ctx, MHCLITE_ERR_WORKSPACE, "staging of %zu bytes needed, %zu given", s.bytes, staging_bytes);
    MHCL_DEVICE(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    int rc;
    // copy streams and events of the context, made on the first call
    if (!ctx->copy_in) {
        if ((rc = check_cuda(ctx, cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking), "copy-in stream"))) return rc;
        if ((rc = check_cuda(ctx, cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking), "copy-out stream"))) return rc;
        cudaEvent_t* evs[2] = {&ctx->ev_fork, &ctx->ev_join};
        for (cudaEvent_t* e : evs)
            if ((rc = check_cuda(ctx, cudaEventCreateWithFlags(e, cudaEventDisableTiming), "cudaEventCreate"))) return rc;
        for (int k = 0; k < MHCLITE_STEP_CHUNKS; ++k) {
            if ((rc = check_cuda(ctx, cudaEventCreateWithFlags(&ctx->ev_in[k], cudaEventDisableTiming), "cudaEventCreate"))) return rc;
            if ((rc = check_cuda(ctx, cudaEventCreateWithFlags(&ctx->ev_cmp[k], cudaEventDisableTiming), "cudaEventCreate"))) return rc;
        }
    }
    // Tokens are independent: the step runs in up to MHCLITE_STEP_CHUNKS chunks of tokens, so that the
    // host->device copies of chunk c + 1 (copy-in stream), the kernels of chunk c (the caller's stream) and
    // the device->host copies of chunk c - 1 (copy-out stream) overlap; PCIe carries both directions at once.
    // The parameter gradients of the chunks add up (accumulate from the second chunk on).
    int64_t chunk = round_up64((T + MHCLITE_STEP_CHUNKS - 1) / MHCLITE_STEP_CHUNKS, 128);
    if (chunk < 256) chunk = 256;
    const int nchunks = (int)((T + chunk - 1) / chunk);
    const int n = ctx->n, C = ctx->C, nf = ctx->nfact, N = ctx_cols(ctx, 0);
#define MHCL_CUDA(call, what) if ((rc = check_cuda(ctx, call, what))) return rc
    MHCL_CUDA(cudaEventRecord(ctx->ev_fork, st), "event record");
    MHCL_CUDA(cudaStreamWaitEvent(ctx->copy_in, ctx->ev_fork, 0), "stream wait");
    MHCL_CUDA(cudaStreamWaitEvent(ctx->copy_out, ctx->ev_fork, 0), "stream wait");
    for (int c = 0; c < nchunks; ++c) {
        const int64_t t0 = (int64_t)c * chunk, Tc = (t0 + chunk <= T) ? chunk : T - t0;
        const size_t big = (size_t)Tc * n * C * sizeof(mhclite_bf16), small = (size_t)Tc * C * sizeof(mhclite_bf16);
        const int64_t ob = t0 * n * C, os = t0 * C;            // element offsets of [T][n][C] and [T][C] tensors
        MHCL_CUDA(cudaMemcpyAsync(s.x + ob, x_host + ob, big, cudaMemcpyHostToDevice, ctx->copy_in), "copy x");
        MHCL_CUDA(cudaMemcpyAsync(s.y + os, y_host + os, small, cudaMemcpyHostToDevice, ctx->copy_in), "copy y");
        MHCL_CUDA(cudaMemcpyAsync(s.g + ob, g_host + ob, big, cudaMemcpyHostToDevice, ctx->copy_in), "copy g");
        MHCL_CUDA(cudaMemcpyAsync(s.du + os, du_host + os, small, cudaMemcpyHostToDevice, ctx->copy_in), "copy du");
        MHCL_CUDA(cudaEventRecord(ctx->ev_in[c], ctx->copy_in), "event record");
        MHCL_CUDA(cudaStreamWaitEvent(st, ctx->ev_in[c], 0), "stream wait");
        float *H_res = s.H_res + t0 * n * n, *H_pre = s.H_pre + t0 * n, *H_post = s.H_post + t0 * n, *av = s.a + t0 * nf,
              *pv = s.p + t0 * N, *rs = s.rstd + t0, *dH_res = s.dH_res + t0 * n * n, *dH_post = s.dH_post + t0 * n;
        if ((rc = mhclite_pre_fwd_fused(ctx, Tc, s.x + ob, W, b, alpha, gain, eps, H_res, H_pre, H_post, av, pv, rs, s.u + os,
                                        stream))) return rc;
        if ((rc = mhclite_postres_fwd(ctx, Tc, s.x + ob, s.y + os, H_res, H_post, s.x_next + ob, stream))) return rc;
        if ((rc = mhclite_postres_bwd(ctx, Tc, s.x + ob, s.y + os, H_res, H_post, s.g + ob, s.dy + os, dH_res, dH_post, nullptr,
                                      0, stream))) return rc;
        if ((rc = mhclite_tail_bwd_fused(ctx, Tc, s.x + ob, W, alpha, gain, eps, av, pv, rs, H_res, H_pre, H_post, s.g + ob,
                                         s.du + os, dH_res, dH_post, s.dx + ob, dW, db, dalpha, dgain,
                                         (c > 0 || accumulate_params) ? 1 : 0, stream))) return rc;
        MHCL_CUDA(cudaEventRecord(ctx->ev_cmp[c], st), "event record");
        MHCL_CUDA(cudaStreamWaitEvent(ctx->copy_out, ctx->ev_cmp[c], 0), "stream wait");
        MHCL_CUDA(cudaMemcpyAsync(u_host + os, s.u + os, small, cudaMemcpyDeviceToHost, ctx->copy_out), "copy u");
        MHCL_CUDA(cudaMemcpyAsync(x_next_host + ob, s.x_next + ob, big, cudaMemcpyDeviceToHost, ctx->copy_out), "copy x_next");
        MHCL_CUDA(cudaMemcpyAsync(dy_host + os, s.dy + os, small, cudaMemcpyDeviceToHost, ctx->copy_out), "copy dy");
        MHCL_CUDA(cudaMemcpyAsync(dx_host + ob, s.dx + ob, big, cudaMemcpyDeviceToHost, ctx->copy_out), "copy dx");
    }
    // join: everything, the last copies included, is ordered before later work on the caller's stream
    MHCL_CUDA(cudaEventRecord(ctx->ev_join, ctx->copy_out), "event record");
    MHCL_CUDA(cudaStreamWaitEvent(st, ctx->ev_join, 0), "stream wait");
#undef MHCL_CUDA
    return MHCLITE_OK;
}

int64_t mhclite_kernel_launches(const mhclite_ctx* ctx) { return ctx ? ctx->launches : 0; }

int mhclite_device_status(mhclite_ctx* ctx) {
    MHCL_REQUIRE_CTX(ctx);
    if (!ctx->status_word) return MHCLITE_OK;
    MHCL_DEVICE(ctx);
    int v[5] = {0, 0, 0, 0, 0};
    int rc = check_cuda(ctx, cudaMemcpy(v, ctx->status_word, sizeof(v), cudaMemcpyDeviceToHost), "read status word");
    if (rc) return rc;
    if (v[0] != 0)
        return fail(ctx, v[0], "a kernel gave up on a bounded wait (kernel %d, wait %d, block %d, index %d)", v[1], v[2],
                    v[3], v[4]);
    return MHCLITE_OK;
}

int mhclite_set_kernel_timing(mhclite_ctx* ctx, int on) {
    MHCL_REQUIRE_CTX(ctx);
    MHCL_DEVICE(ctx);
    if (on) {
        for (int k = 0; k < MHCLITE_KERNEL_COUNT; ++k)
            for (int e = 0; e < 2; ++e)
                if (!ctx->ev[k][e]) {
                    int rc = check_cuda(ctx, cudaEventCreate(&ctx->ev[k][e]), "cudaEventCreate");
                    if (rc) return rc;
                }
    }
    ctx->timing = on != 0;
    return MHCLITE_OK;
}

int mhclite_kernel_time_ms(mhclite_ctx* ctx, int kernel, float* ms) {
    MHCL_REQUIRE_CTX(ctx);
    if (kernel < 0 || kernel >= MHCLITE_KERNEL_COUNT || !ms) return fail(ctx, MHCLITE_ERR_BAD_ARG, "bad kernel id");
    if (!ctx->ev[kernel][0]) return fail(ctx, MHCLITE_ERR_BAD_ARG, "kernel timing was never switched on");
    if (!ctx->ev_recorded[kernel])
        return fail(ctx, MHCLITE_ERR_BAD_ARG, "kernel %d has not been launched since timing was switched on", kernel);
    return check_cuda(ctx, cudaEventElapsedTime(ms, ctx->ev[kernel][0], ctx->ev[kernel][1]), "cudaEventElapsedTime");
}

}  // extern "C"
