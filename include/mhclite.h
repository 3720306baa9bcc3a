/*
 * mhclite.h -- C ABI of the mHC-lite residual-mixing library for NVIDIA B200 (sm_100a).
 *
 * The library computes, for every token independently, the dynamic residual
 * mixing step of a Hyper-Connections layer with n residual streams of C channels:
 *
 *     x_{l+1} = H_res x_l + H_post^T f(H_pre x_l)                        (paper Eq. (1))
 *
 * with the mHC-lite mappings (paper Eq. (4), (5)):
 *
 *     x' = RMSNorm(flatten(x_l))                        flatten is stream-major, m = j*C + c
 *     z  = alpha (.) (x' W) + b                         columns [res (n!) | pre (n) | post (n)]
 *     H_pre = sigmoid(z_pre), H_post = 2 sigmoid(z_post), a = softmax(z_res)
 *     H_res = sum_k a_k P_k                             P_k[i][sigma_k(i)] = 1, sigma in lexicographic order
 *
 * and, as a comparison path, the mHC mapping of paper Eq. (2),
 * H_res = SK(exp(mat(z_res))) with `iters` Sinkhorn-Knopp iterations (one
 * iteration = normalise all columns, then all rows).  The sublayer f is the
 * caller's: the forward is split in "before f" (coeffs, premix) and "after f"
 * (postres); the backward in "before f's backward" (postres_bwd) and "after"
 * (premix_bwd, coeffs_bwd, or the fused tail).
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers on the context's device unless the name ends
 *     in _host.  The caller owns every buffer, including the workspace; the
 *     library allocates no device memory.  All pointers must be 16-byte aligned.
 *   - bf16 tensors are raw 16-bit patterns (mhclite_bf16); fp32 tensors are float.
 *   - Layouts are dense row-major: x [T][n][C], y/u/du/dy [T][C], H_res [T][n][n]
 *     (row i = output stream), H_pre/H_post [T][n], W [n*C][N], N = n!+2n
 *     (n*n+2n for the SK path).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and never synchronise the device.  Calls that use the
 *     workspace (coeffs_fwd, coeffs_bwd, the fused calls, the SK calls) must not
 *     overlap on the GPU with another call on the same context.
 *   - Return value: MHCLITE_OK (0) or a negative mhclite_status.  Nothing is
 *     launched when arguments are rejected.  T == 0 is a valid no-op.
 *   - Arithmetic: bf16 in, fp32 accumulate, bf16 (activations) or fp32
 *     (coefficients, parameter gradients) out.
 */
#ifndef MHCLITE_H_
#define MHCLITE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MHCLITE_API __attribute__((visibility("default")))
#else
#define MHCLITE_API
#endif

typedef uint16_t mhclite_bf16;
typedef struct mhclite_ctx mhclite_ctx;

typedef enum mhclite_status {
    MHCLITE_OK = 0,
    MHCLITE_ERR_BAD_ARG = -1,      /* n not in [2,5], C % 8 != 0, T < 0, null / misaligned pointer, ... */
    MHCLITE_ERR_CUDA = -2,         /* a CUDA runtime call or launch failed; see mhclite_last_error */
    MHCLITE_ERR_WORKSPACE = -3,    /* workspace missing or smaller than mhclite_workspace_bytes */
    MHCLITE_ERR_TIMEOUT = -4       /* a bounded device-side wait gave up (status word, never a trap) */
} mhclite_status;

/* ---- context -------------------------------------------------------------------------------- */

/* Creates a context for n streams (2..5) of C channels (multiple of 8) on CUDA device `device`,
 * and uploads the permutation tables to that device's constant memory.  *out is written on success. */
MHCLITE_API int mhclite_create(mhclite_ctx** out, int n, int C, int device);
MHCLITE_API int mhclite_destroy(mhclite_ctx* ctx);

/* Human-readable name of a status code (static string). */
MHCLITE_API const char* mhclite_status_string(int status);
/* Text of the last error recorded on this context (valid until the next call on it). */
MHCLITE_API const char* mhclite_last_error(const mhclite_ctx* ctx);

/* Permutation table of paper Theorem 3.1 / Section 3.2: sigma_host[k*n + i] = sigma_k(i), the n!
 * permutations of (0..n-1) in lexicographic order, k = 0 the identity.  Host buffer of n!*n bytes. */
MHCLITE_API int mhclite_perm_table(int n, uint8_t* sigma_host);
/* The same table read back from the device's constant memory (what the kernels index). */
MHCLITE_API int mhclite_perm_table_device(mhclite_ctx* ctx, uint8_t* sigma_host);

/* Scratch the workspace-using calls need for up to T tokens (kind: 0 = mHC-lite, 1 = SK path). */
MHCLITE_API size_t mhclite_workspace_bytes(int n, int C, int64_t T, int kind);
/* Attaches caller-owned device scratch (256-byte aligned).  It must stay valid until replaced. */
MHCLITE_API int mhclite_set_workspace(mhclite_ctx* ctx, void* workspace, size_t bytes);

/* ---- forward -------------------------------------------------------------------------------- */

/* Paper Eq. (4), (5): the mappings of every token.
 *   in : x [T,n,C] bf16, W [nC,N] f32, b [N] f32, alpha [3] f32 = (res, pre, post), gain [nC] f32
 *        (RMSNorm weight), eps (RMSNorm epsilon, host scalar)
 *   out: H_res [T,n,n], H_pre [T,n], H_post [T,n] f32;
 *        saved for the backward: a_saved [T,n!] (softmax weights), p_saved [T,N] (x' W before alpha
 *        and bias), rstd [T] (1/sqrt(mean(x^2)+eps)).  */
MHCLITE_API int mhclite_coeffs_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                       const float* W, const float* b, const float* alpha, const float* gain, float eps,
                       float* H_res, float* H_pre, float* H_post,
                       float* a_saved, float* p_saved, float* rstd, void* stream);

/* Paper Eq. (1), inner term: u[t,c] = sum_j H_pre[t,j] x[t,j,c].  u [T,C] bf16. */
MHCLITE_API int mhclite_premix_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* H_pre,
                       mhclite_bf16* u, void* stream);

/* Paper Eq. (1): x_next[t,i,c] = sum_j H_res[t,i,j] x[t,j,c] + H_post[t,i] y[t,c].  x_next [T,n,C] bf16. */
MHCLITE_API int mhclite_postres_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const mhclite_bf16* y,
                        const float* H_res, const float* H_post, mhclite_bf16* x_next, void* stream);

/* coeffs_fwd followed by premix_fwd with x read once (same results as the two calls). */
MHCLITE_API int mhclite_pre_fwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                          const float* W, const float* b, const float* alpha, const float* gain, float eps,
                          float* H_res, float* H_pre, float* H_post,
                          float* a_saved, float* p_saved, float* rstd, mhclite_bf16* u, void* stream);

/* ---- backward (exact gradient of Eq. (1), (4), (5)) ------------------------------------------ */

/* Gradient of postres_fwd given g = dL/dx_next [T,n,C] bf16:
 *   dy[t,c]      = sum_i H_post[t,i] g[t,i,c]                        [T,C] bf16
 *   dH_post[t,i] = <g[t,i,:], y[t,:]>, dH_res[t,i,j] = <g[t,i,:], x[t,j,:]>     f32
 *   dx[t,j,c]   (+)= sum_i H_res[t,i,j] g[t,i,c]    (skipped when dx is NULL; added to dx when
 *                                                    accumulate_dx != 0, else stored)           */
MHCLITE_API int mhclite_postres_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const mhclite_bf16* y,
                        const float* H_res, const float* H_post, const mhclite_bf16* g,
                        mhclite_bf16* dy, float* dH_res, float* dH_post,
                        mhclite_bf16* dx, int accumulate_dx, void* stream);

/* Gradient of premix_fwd given du = dL/du [T,C] bf16:
 *   dH_pre[t,j] = <du[t,:], x[t,j,:]>;  dx[t,j,c] (+)= H_pre[t,j] du[t,c]  (dx may be NULL). */
MHCLITE_API int mhclite_premix_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x, const float* H_pre,
                       const mhclite_bf16* du, float* dH_pre,
                       mhclite_bf16* dx, int accumulate_dx, void* stream);

/* Gradient of coeffs_fwd: from (dH_res, dH_pre, dH_post) back through the permutation sum, softmax,
 * sigmoids, the affine maps and RMSNorm.
 *   dx [T,n,C] bf16 (+)= dL/dx through the mappings;  dW [nC,N], db [N], dalpha [3], dgain [nC] f32,
 *   summed over the T tokens (added to the buffers when accumulate_params != 0, else stored). */
MHCLITE_API int mhclite_coeffs_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                       const float* W, const float* alpha, const float* gain, float eps,
                       const float* a_saved, const float* p_saved, const float* rstd,
                       const float* H_pre, const float* H_post,
                       const float* dH_res, const float* dH_pre, const float* dH_post,
                       mhclite_bf16* dx, int accumulate_dx,
                       float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                       void* stream);

/* Allocation-free variant of mhclite_coeffs_bwd (the paper has no counterpart: this is a property of
 * the library, not of the method).  It is for callers that cannot hand the library a workspace because
 * they cannot allocate device memory where the call is made: code running inside an allocator or
 * memory-pool callback, a process with a memory budget fixed at start-up, a plug-in that only ever
 * sees its inputs and outputs.  Same arguments, same results as mhclite_coeffs_bwd, but the scratch is
 * a fixed array of mhclite_static_scratch_bytes() bytes inside the library's device image (every GPU
 * that loads the library holds it until the process exits) and no workspace needs to be attached.
 *   - The call needs about 4 * (T * Np + T + n * C * Np) bytes of it, Np = n!+2n rounded up to 8;
 *     problem sizes that need more than the array holds are rejected with MHCLITE_ERR_WORKSPACE
 *     and nothing is launched.
 *   - The call allocates and frees nothing.  The first call on each device looks up the array's
 *     device address (a synchronous, one-time set-up): make that first call before any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents; each call
 *     rewrites or clears every part it reads, so back-to-back calls on one stream are fine, but two
 *     calls that overlap on the GPU (different streams, different contexts) race on it. */
MHCLITE_API size_t mhclite_static_scratch_bytes(void);
MHCLITE_API int mhclite_coeffs_bwd_static(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                       const float* W, const float* alpha, const float* gain, float eps,
                       const float* a_saved, const float* p_saved, const float* rstd,
                       const float* H_pre, const float* H_post,
                       const float* dH_res, const float* dH_pre, const float* dH_post,
                       mhclite_bf16* dx, int accumulate_dx,
                       float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                       void* stream);

/* premix_bwd + coeffs_bwd + the H_res^T g term of postres_bwd, writing the complete dx once:
 *   dx[t,j,c] = sum_i H_res[t,i,j] g[t,i,c] + H_pre[t,j] du[t,c] + (gradient through the mappings).
 * dH_res and dH_post come from a preceding mhclite_postres_bwd call made with dx = NULL. */
MHCLITE_API int mhclite_tail_bwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                           const float* W, const float* alpha, const float* gain, float eps,
                           const float* a_saved, const float* p_saved, const float* rstd,
                           const float* H_res, const float* H_pre, const float* H_post,
                           const mhclite_bf16* g, const mhclite_bf16* du,
                           const float* dH_res, const float* dH_post,
                           mhclite_bf16* dx,
                           float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                           void* stream);

/* ---- mHC comparison path (paper Eq. (2)): H_res = SK_iters(exp(mat(z_res))) ------------------ */

/* W_sk [nC, n*n+2n], b_sk [n*n+2n], columns [res (row-major n x n) | pre | post].  iters in [1,64]
 * (the paper's mHC uses 20).  The largest residual logit is subtracted before exp. */
MHCLITE_API int mhc_sk20_coeffs_fwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                        const float* W_sk, const float* b_sk, const float* alpha, const float* gain,
                        float eps, int iters,
                        float* H_res, float* H_pre, float* H_post, float* p_saved, float* rstd,
                        void* stream);
/* Gradient of mhc_sk20_coeffs_fwd; the SK iterates are recomputed from p_saved, not stored. */
MHCLITE_API int mhc_sk20_coeffs_bwd(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                        const float* W_sk, const float* b_sk, const float* alpha, const float* gain,
                        float eps, int iters,
                        const float* p_saved, const float* rstd, const float* H_pre, const float* H_post,
                        const float* dH_res, const float* dH_pre, const float* dH_post,
                        mhclite_bf16* dx, int accumulate_dx,
                        float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                        void* stream);

/* The SK path's counterpart of mhclite_tail_bwd_fused: dH_pre, the SK activation backward and the
 * projection backward, with dx = H_res^T g + H_pre du + (gradient through the mappings) written once.
 * dH_res and dH_post come from mhclite_postres_bwd called with dx = NULL (the streaming calls
 * premix_* / postres_* take coefficients, so they serve both paths). */
MHCLITE_API int mhc_sk20_tail_bwd_fused(mhclite_ctx* ctx, int64_t T, const mhclite_bf16* x,
                        const float* W_sk, const float* b_sk, const float* alpha, const float* gain,
                        float eps, int iters,
                        const float* p_saved, const float* rstd,
                        const float* H_res, const float* H_pre, const float* H_post,
                        const mhclite_bf16* g, const mhclite_bf16* du,
                        const float* dH_res, const float* dH_post,
                        mhclite_bf16* dx,
                        float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                        void* stream);

/* ---- doubly-stochastic diagnostics (paper Section 3.1 footnote) -------------------------------- */

/* Per token: l1_err[t] = ||H 1 - 1||_1 + ||H^T 1 - 1||_1 and colsum_dev[t] = max_j |sum_i H[i][j] - 1|
 * of H = H_res[t] (either output may be NULL). */
MHCLITE_API int mhclite_ds_gap(mhclite_ctx* ctx, int64_t T, const float* H_res, float* l1_err, float* colsum_dev,
                   void* stream);

/* Product of the residual mappings over depth (paper Section 3.1: prod_l H_res_l must stay doubly stochastic
 * for the signal to keep its norm across layers).  Per token: P[t] <- H_res[t] P[t], later layers multiplying
 * on the left as x_{l+1} = H_l x_l composes; with first != 0, P[t] <- H_res[t].  P is [T][n][n] fp32, updated
 * in place, and must not alias H_res.  Its gap is read with mhclite_ds_gap(P). */
MHCLITE_API int mhclite_depth_product(mhclite_ctx* ctx, int64_t T, const float* H_res, float* P, int first,
                                      void* stream);

/* Relative range of paper Eq. (3), per token: nu[t] = (smallest positive entry) / (largest entry) of the
 * n x n matrix X[t] (0 when no entry is positive); 1/nu bounds the Sinkhorn-Knopp iteration count. */
MHCLITE_API int mhclite_relative_range(mhclite_ctx* ctx, int64_t T, const float* X, float* nu, void* stream);

/* ---- whole step from host buffers -------------------------------------------------------------- */

/* Bytes of device staging mhclite_step_host needs for T tokens. */
MHCLITE_API size_t mhclite_step_host_bytes(int n, int C, int64_t T);

/* One forward + backward pass of the layer (paper Eq. (1), (4), (5) and their gradient) with the
 * activations in HOST memory and the sublayer's results supplied: copies x, y, g = dL/dx_next and
 * du = dL/du host->device into `staging`, runs pre_fwd_fused, postres_fwd, postres_bwd and
 * tail_bwd_fused, and copies u, x_next, dy, dx device->host.  Parameters and their gradients stay on
 * the device.  The tokens are processed in up to eight chunks so that the copies in, the kernels and the
 * copies out of successive chunks overlap (two copy streams owned by the context, made on the first call
 * and tied to `stream` by events: the call stays ordered on `stream`); the parameter gradients of the chunks
 * add up.  Host buffers should be page-locked for the copies to be asynchronous; results are valid once
 * `stream` has been synchronised.  `staging` is caller-owned device scratch (256-byte aligned) of
 * at least mhclite_step_host_bytes; the context's workspace must be attached as well. */
MHCLITE_API int mhclite_step_host(mhclite_ctx* ctx, int64_t T,
                      const mhclite_bf16* x_host, const mhclite_bf16* y_host,
                      const mhclite_bf16* g_host, const mhclite_bf16* du_host,
                      const float* W, const float* b, const float* alpha, const float* gain, float eps,
                      mhclite_bf16* u_host, mhclite_bf16* x_next_host,
                      mhclite_bf16* dy_host, mhclite_bf16* dx_host,
                      float* dW, float* db, float* dalpha, float* dgain, int accumulate_params,
                      void* staging, size_t staging_bytes, void* stream);

/* Per-kernel device time, for roofline accounting.  With timing on, the library records a pair of CUDA
 * events on the call's stream around each launch of the kernels below (a few microseconds of overhead
 * per launch: switch it off for throughput runs).  mhclite_kernel_time_ms returns the duration of the
 * most recent launch of that kernel; the caller must have synchronised the stream since.  A kernel that
 * the problem size routes around (the fallbacks replace some of them) has no time: MHCLITE_ERR_BAD_ARG. */
typedef enum mhclite_kernel {
    MHCLITE_KERNEL_PROJ_FWD = 0,     /* tensor-core projection + sum of squares        reads x            */
    MHCLITE_KERNEL_ACT_PREMIX = 1,   /* mappings + pre-mix                              reads x, writes u  */
    MHCLITE_KERNEL_POSTRES_FWD = 2,  /* merge                                           reads x, y; writes x_next */
    MHCLITE_KERNEL_POSTRES_BWD = 3,  /* merge backward                                  reads g, x, y; writes dy  */
    MHCLITE_KERNEL_TAIL_PRE = 4,     /* dH_pre + activation backward                    reads x, du        */
    MHCLITE_KERNEL_TAIL_MMA = 5,     /* projection backward + dx + dW                   reads x, g, du; writes dx */
    MHCLITE_KERNEL_COUNT = 6
} mhclite_kernel;
MHCLITE_API int mhclite_set_kernel_timing(mhclite_ctx* ctx, int on);
MHCLITE_API int mhclite_kernel_time_ms(mhclite_ctx* ctx, int kernel, float* ms);

/* Synchronous check of the device status word: kernels that wait on hardware barriers do so with a bound
 * and, instead of hanging, record MHCLITE_ERR_TIMEOUT there and return.  Copies one int device->host
 * (synchronises the device); returns MHCLITE_OK or the recorded status. */
MHCLITE_API int mhclite_device_status(mhclite_ctx* ctx);

/* Number of kernels this context has launched since it was created (for accounting; host counter). */
MHCLITE_API int64_t mhclite_kernel_launches(const mhclite_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MHCLITE_H_ */
