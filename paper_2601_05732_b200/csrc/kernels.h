// Launchers of the library's kernels (host side). Each enqueues on the given stream and returns.
#pragma once
#include "common.cuh"

namespace mhcl {

// stream_kernels.cu
void launch_premix_fwd(const mhclite_ctx* c, int64_t T, const void* x, const float* H_pre, void* u, cudaStream_t s);
void launch_postres_fwd(const mhclite_ctx* c, int64_t T, const void* x, const void* y, const float* H_res,
                        const float* H_post, void* x_next, cudaStream_t s);
void launch_postres_bwd(const mhclite_ctx* c, int64_t T, const void* x, const void* y, const float* H_res,
                        const float* H_post, const void* g, void* dy, float* dH_res, float* dH_post, void* dx,
                        int acc, cudaStream_t s);
void launch_premix_bwd(const mhclite_ctx* c, int64_t T, const void* x, const float* H_pre, const void* du,
                       float* dH_pre, void* dx, int acc, cudaStream_t s);
void launch_tail_mix(const mhclite_ctx* c, int64_t T, const void* x, const void* g, const void* du, const float* H_res,
                     const float* H_pre, float* dH_pre, void* dx, cudaStream_t s);
void launch_ds_gap(const mhclite_ctx* c, int64_t T, const float* H_res, float* l1, float* cdev, cudaStream_t s);
void launch_ds_gap_stats(const mhclite_ctx* c, int64_t T, const float* H_res, float* stats, cudaStream_t s);
void launch_log_inv_nu_hist(const mhclite_ctx* c, int64_t T, const float* X, int bins, float lo, float hi,
                            unsigned long long* hist, cudaStream_t s);
void launch_depth_product(const mhclite_ctx* c, int64_t T, const float* H_res, float* P, int first, cudaStream_t s);
void launch_relative_range(const mhclite_ctx* c, int64_t T, const float* X, float* nu, cudaStream_t s);

// proj_kernels.cu : RMSNorm statistics + the skinny projection and its gradient
// proj_mma.cu: W' = diag(gain) W packed as bf16 hi/lo MMA fragments; qpart[s][t][c] = partial x W' of K slice s,
// ssq[s][t] = partial sum of squares (the activation kernels add the slices and apply rstd)
void launch_pack_w(const mhclite_ctx* c, const ProjPlan& p, int N, const float* W, const float* gain, void* Wp,
                   cudaStream_t s);
void launch_proj_fwd_mma(const mhclite_ctx* c, int64_t T, const ProjPlan& p, const void* x, const void* Wp,
                         float* qpart, float* ssq, cudaStream_t s);
// dx[t,m] (+)= sum_c e[t,c] gain[m] W[m,c] - x[t,m] kappa[t]   (e = rstd*alpha*dz)
void launch_proj_bwd_dx(const mhclite_ctx* c, int64_t T, int N, int Npad, const void* x, const float* W,
                        const float* gain, const float* e, const float* kappa, void* dx, int acc, cudaStream_t s);
// G[m,c] = sum_t x[t,m] e[t,c];  dW (+)= gain (.) G ;  dgain[m] (+)= sum_c W[m,c] G[m,c]
void launch_proj_bwd_dw(const mhclite_ctx* c, int64_t T, int N, int Npad, const void* x, const float* W,
                        const float* gain, const float* e, float* G, float* dW, float* dgain, int acc,
                        cudaStream_t s);

// proj_tc.cu : the same projection on tcgen05 / TMA / tensor memory (up to 256 columns); tail_tc.cu : the
// backward of wide projections (n = 5) on tcgen05
bool tensor_maps_available();
bool launch_tail_g_tc(const mhclite_ctx* c, int64_t T, const TailPlan& p, const void* x, const void* ehi,
                      const void* elo, float* Gpart, int* status, cudaStream_t s);
size_t tail_wb_bytes(int n, int C, int Kp);
bool launch_tail_dx_tc(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                       const void* du, const void* ehi, const float* kappa, const float* H_res, const float* H_pre,
                       const float* W, const float* gain, void* Wb, void* dx, int acc_dx, int* status, cudaStream_t s);
// tail_ftc.cu : narrow projections, dx and the G partials [f_splits][nC][Kp] in one tcgen05 kernel
void plan_tail_ftc(int n, int C, int64_t T, int sm_count, TailPlan* p);
bool launch_tail_ftc_prep(const mhclite_ctx* c, int N, const TailPlan& p, const float* W, const float* gain, void* Wf,
                          float* zero_db, float* zero_dalpha, cudaStream_t s);
bool launch_tail_ftc(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                     const void* du, const void* ehi, const void* elo, const float* kappa, const float* H_res,
                     const float* H_pre, const float* W, const float* gain, void* Wf, bool wf_packed, void* dx,
                     int acc_dx, float* Gpart, int* status, cudaStream_t s);
// db[N], dalpha[3] (+)= the nparts per-block partials alone (for a backward that does not end in launch_tail_finish)
void launch_dpart_sum(const mhclite_ctx* c, int N, const float* dpart, int nparts, float* db, float* dalpha, int acc_params,
                      cudaStream_t s);
// dpart (null: none): nparts per-block partials of db / dalpha, added up into db[N], dalpha[3] by the same launch
void launch_tail_finish(const mhclite_ctx* c, int N, int Kp, int splits, const float* W, const float* gain,
                        const float* Gpart, float* dW, float* dgain, int acc_params, cudaStream_t s,
                        const float* dpart = nullptr, int nparts = 0, float* db = nullptr, float* dalpha = nullptr);
bool proj_tc_supported(int n, int C, int N);
int proj_tc_nq(int N);
void launch_pack_wt(const mhclite_ctx* c, const ProjPlan& p, int N, const float* W, const float* gain, void* Wt,
                    cudaStream_t s);
bool launch_proj_fwd_tc(const mhclite_ctx* c, int64_t T, int N, const ProjPlan& p, const void* x, const void* Wt,
                        float* qpart, float* ssq, int* status, cudaStream_t s);

// postres_proj.cu : the merge of one layer fused with the RMSNorm statistics and projection of the next
bool postres_proj_supported(int n, int C, int N);
bool launch_postres_proj(const mhclite_ctx* c, int64_t T, int N, const ProjPlan& pp, const void* x, const void* y,
                         const float* H_res, const float* H_post, void* x_next, const void* Wt, float* qpart, float* ssq,
                         int* status, cudaStream_t s);

// act_kernels.cu : per-token activations, H_res assembly and their gradients
void launch_lite_act_fwd(const mhclite_ctx* c, int64_t T, const ProjPlan& pp, const float* qpart, const float* ssq,
                         float eps, const float* b, const float* alpha, float* H_res, float* H_pre, float* H_post,
                         float* a_saved, float* p_saved, float* rstd, cudaStream_t s);
void launch_lite_act_bwd(const mhclite_ctx* c, int64_t T, int Npad, const float* a, const float* p, const float* rstd,
                         const float* alpha, const float* H_pre, const float* H_post, const float* dH_res,
                         const float* dH_pre, const float* dH_post, float* e, void* ehi, void* elo, int Kp,
                         float* kappa, float* db, float* dalpha, cudaStream_t s);
// mappings + pre-mix in one kernel; dH_pre + activation backward in one kernel (the fused call sequences)
void launch_lite_act_premix(const mhclite_ctx* c, int64_t T, const ProjPlan& pp, const float* qpart, const float* ssq,
                            float eps, const float* b, const float* alpha, float* H_res, float* H_pre, float* H_post,
                            float* a_saved, float* p_saved, float* rstd, const void* x, void* u, cudaStream_t s,
                            float* u_rstd = nullptr, float eps_u = 0.f);
// u_rstd[t] = (mean_c u[t,c]^2 + eps)^-1/2 of a stored u [T][C] (bf16), one warp per token
void launch_row_rstd(const mhclite_ctx* c, int64_t T, const void* u, float eps, float* u_rstd, cudaStream_t s);
int launch_lite_tailpre(const mhclite_ctx* c, int64_t T, const void* x, const void* du, const float* a, const float* p,
                        const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                        const float* dH_res, const float* dH_post, float* dH_pre_ws, float* e, int Npad, void* ehi,
                        void* elo, int Kp, float* kappa, float* db, float* dalpha, cudaStream_t s);
// the SK path's counterparts of the two fused kernels above
void launch_sk_act_premix(const mhclite_ctx* c, int64_t T, int iters, const ProjPlan& pp, const float* qpart,
                          const float* ssq, float eps, const float* b, const float* alpha, float* H_res, float* H_pre,
                          float* H_post, float* p_saved, float* rstd, const void* x, void* u, cudaStream_t s);
int launch_sk_tailpre(const mhclite_ctx* c, int64_t T, int iters, const void* x, const void* du, const float* p,
                      const float* b, const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                      const float* dH_res, const float* dH_post, float* e, int Npad, void* ehi, void* elo, int Kp,
                      float* kappa, float* db, float* dalpha, cudaStream_t s);
void launch_sk_act_fwd(const mhclite_ctx* c, int64_t T, int iters, const ProjPlan& pp, const float* qpart,
                       const float* ssq, float eps, const float* b, const float* alpha, float* H_res, float* H_pre,
                       float* H_post, float* p_saved, float* rstd, cudaStream_t s);
void launch_sk_act_bwd(const mhclite_ctx* c, int64_t T, int Npad, int iters, const float* p, const float* b,
                       const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                       const float* dH_res, const float* dH_pre, const float* dH_post, float* e, void* ehi, void* elo,
                       int Kp, float* kappa, float* db, float* dalpha, cudaStream_t s);

// tail_mma.cu : tensor-core projection / RMSNorm backward, optionally fused with the rest of dx (g != NULL)
void launch_tail_mma(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                     const void* du, const void* ehi, const void* elo, const float* kappa, const float* H_res,
                     const float* H_pre, const float* W, const float* gain, void* dx, int acc_dx, float* Gpart,
                     float* dW, float* dgain, int acc_params, cudaStream_t s);

}  // namespace mhcl
