// Allocation-free variant of mhclite_coeffs_bwd.
//
// Some callers cannot obtain device memory at the point where they need the mappings' gradient: code
// that runs inside a framework's memory-pool callback or under a caching allocator that must not be
// re-entered, a process whose memory budget is fixed up front, a plug-in that is handed only its inputs
// and outputs.  For them the scratch that mhclite_coeffs_bwd takes from the caller's workspace lives
// here in a fixed array in the library's device image instead.  Every GPU that loads the library
// carries the array (kStaticScratchBytes) until the process exits, which is why it is kept modest.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace mhcl {

constexpr size_t kStaticScratchBytes = 4u << 20;        // 4 MiB: e.g. n = 4, C = 1024 up to about 27 000 tokens

// The scratch itself.  In host code this name is only a handle for the runtime's symbol look-up,
// never a device address: kernels get the pointer obtained by cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_setup_mutex;
static void* g_scratch_addr[kMaxDevices];               // per device, filled on first use

// Device address of the array on the current device (looked up once per device).
static cudaError_t static_scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = p;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

}  // namespace mhcl

using namespace mhcl;

extern "C" {

size_t mhclite_static_scratch_bytes(void) { return kStaticScratchBytes; }

int mhclite_coeffs_bwd_static(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* W, const float* alpha,
                              const float* gain, float eps, const float* a_saved, const float* p_saved,
                              const float* rstd, const float* H_pre, const float* H_post, const float* dH_res,
                              const float* dH_pre, const float* dH_post, mhclite_bf16* dx, int accumulate_dx,
                              float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                              void* stream) {
    (void)eps;
    if (!ctx) return MHCLITE_ERR_BAD_ARG;
    ctx->err[0] = 0;
    if (T < 0) return fail(ctx, MHCLITE_ERR_BAD_ARG, "T < 0");
    if (T == 0) return MHCLITE_OK;
    const void* ptrs[] = {x, W, alpha, gain, a_saved, p_saved, rstd, H_pre, H_post, dH_res, dH_pre, dH_post,
                          dx, dW, db, dalpha, dgain};
    for (const void* p : ptrs)
        if (!p || ((uintptr_t)p & 15)) return fail(ctx, MHCLITE_ERR_BAD_ARG, "null or misaligned pointer");
    if (ctx->device >= kMaxDevices) return fail(ctx, MHCLITE_ERR_BAD_ARG, "device index %d not supported", ctx->device);
    // scratch of this call: e [T][Npad], kappa [T], G [nC][Npad] (fp32), each 256-byte aligned
    const int N = ctx_cols(ctx, 0), Npad = round_up(N, 8), nC = ctx->n * ctx->C;
    auto up256 = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t o_kappa = up256((size_t)T * Npad * 4), o_G = o_kappa + up256((size_t)T * 4);
    const size_t need = o_G + up256((size_t)nC * Npad * 4);
    if (need > kStaticScratchBytes)
        return fail(ctx, MHCLITE_ERR_WORKSPACE,
                    "mhclite_coeffs_bwd_static: n=%d C=%d T=%lld needs %zu bytes of scratch, the built-in array holds "
                    "%zu; use mhclite_coeffs_bwd with a workspace", ctx->n, ctx->C, (long long)T, need,
                    kStaticScratchBytes);

    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e == cudaSuccess && prev != ctx->device) e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaSetDevice");
    void* base = nullptr;
    int rc = check_cuda(ctx, static_scratch_address(ctx->device, &base), "cudaGetSymbolAddress(static scratch)");
    if (rc == MHCLITE_OK) {
        float* e = (float*)base;
        float* kappa = (float*)((char*)base + o_kappa);
        float* G = (float*)((char*)base + o_G);
        cudaStream_t s = (cudaStream_t)stream;
        if (!accumulate_params) {
            rc = check_cuda(ctx, cudaMemsetAsync(db, 0, (size_t)N * sizeof(float), s), "memset db");
            if (rc == MHCLITE_OK) rc = check_cuda(ctx, cudaMemsetAsync(dalpha, 0, 3 * sizeof(float), s), "memset dalpha");
        }
        if (rc == MHCLITE_OK) {
            // every region of the array that the kernels read is written first within this call: e and
            // kappa by the activation backward, G by a memset inside launch_proj_bwd_dw
            launch_lite_act_bwd(ctx, T, Npad, a_saved, p_saved, rstd, alpha, H_pre, H_post, dH_res, dH_pre, dH_post,
                                e, nullptr, nullptr, 0, kappa, db, dalpha, s);
            launch_proj_bwd_dx(ctx, T, N, Npad, x, W, gain, e, kappa, dx, accumulate_dx, s);
            launch_proj_bwd_dw(ctx, T, N, Npad, x, W, gain, e, G, dW, dgain, accumulate_params, s);
            rc = check_cuda(ctx, cudaGetLastError(), "coeffs_bwd_static launch");
        }
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return rc;
}

}  // extern "C"
