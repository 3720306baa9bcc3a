// Streaming kernels of paper Eq. (1) and its gradient: stream pre-mix, post/residual merge and their
// backward passes.  All are HBM-bound scans: 16-byte vector loads/stores of bf16, fp32 accumulation,
// the tiny per-token coefficients read through the read-only path.
#include "common.cuh"
#include "kernels.h"

namespace mhcl {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------------
// u[t,c] = sum_j H_pre[t,j] x[t,j,c]                                              (Eq. (1), H_pre x_l)
// ------------------------------------------------------------------------------------------------
template <int N_>
__global__ void __launch_bounds__(kThreads) premix_fwd_k(int64_t T, int C8, const uint4* __restrict__ x,
                                                         const float* __restrict__ H_pre, uint4* __restrict__ u) {
    const int64_t total = T * C8;
    for (int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * kThreads) {
        const int64_t t = idx / C8;
        const int cv = (int)(idx - t * C8);
        float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        uint4 v[N_];
#pragma unroll
        for (int j = 0; j < N_; ++j) v[j] = ld_stream(x + (t * N_ + j) * C8 + cv);
#pragma unroll
        for (int j = 0; j < N_; ++j) {
            const float h = __ldg(H_pre + t * N_ + j);
            float f[8];
            unpack8(v[j], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(h, f[e], acc[e]);
        }
        st_stream(u + idx, pack8(acc));
    }
}

// ------------------------------------------------------------------------------------------------
// x_next[t,i,c] = sum_j H_res[t,i,j] x[t,j,c] + H_post[t,i] y[t,c]                          (Eq. (1))
// ------------------------------------------------------------------------------------------------
template <int N_>
__global__ void __launch_bounds__(kThreads, (N_ <= 4 ? 3 : 2)) postres_fwd_k(int64_t T, int C8, const uint4* __restrict__ x,
                                                          const uint4* __restrict__ y, const float* __restrict__ H_res,
                                                          const float* __restrict__ H_post, uint4* __restrict__ x_next) {
    const int64_t total = T * C8;
    for (int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * kThreads) {
        const int64_t t = idx / C8;
        const int cv = (int)(idx - t * C8);
        uint4 v[N_];
#pragma unroll
        for (int j = 0; j < N_; ++j) v[j] = ld_stream(x + (t * N_ + j) * C8 + cv);
        const uint4 yv = ld_stream(y + idx);
        float xf[N_][8], yf[8];
#pragma unroll
        for (int j = 0; j < N_; ++j) unpack8(v[j], xf[j]);
        unpack8(yv, yf);
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            const float hp = __ldg(H_post + t * N_ + i);
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = hp * yf[e];
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                const float h = __ldg(H_res + (t * N_ + i) * N_ + j);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = fmaf(h, xf[j][e], acc[e]);
            }
            st_stream(x_next + (t * N_ + i) * C8 + cv, pack8(acc));
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Gradient of the merge, one warp per token:
//   dy = sum_i H_post[i] g_i ; dH_post[i] = <g_i,y> ; dH_res[i][j] = <g_i,x_j> ; dx_j (+)= sum_i H_res[i][j] g_i
// ------------------------------------------------------------------------------------------------
template <int N_, bool WRITE_DX, bool ACC_DX>
__global__ void __launch_bounds__(kThreads) postres_bwd_k(int64_t T, int C8, const uint4* __restrict__ x,
                                                          const uint4* __restrict__ y, const float* __restrict__ H_res,
                                                          const float* __restrict__ H_post, const uint4* __restrict__ g,
                                                          uint4* __restrict__ dy, float* __restrict__ dH_res,
                                                          float* __restrict__ dH_post, uint4* dx) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
    for (int64_t t = warp0; t < T; t += nwarps) {
        float hpost[N_], hres[N_][N_];
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            hpost[i] = __ldg(H_post + t * N_ + i);
#pragma unroll
            for (int j = 0; j < N_; ++j) hres[i][j] = __ldg(H_res + (t * N_ + i) * N_ + j);
        }
        float r_res[N_][N_], r_post[N_];
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            r_post[i] = 0.f;
#pragma unroll
            for (int j = 0; j < N_; ++j) r_res[i][j] = 0.f;
        }
        for (int cv = lane; cv < C8; cv += 32) {
            uint4 gv[N_], xv[N_];
#pragma unroll
            for (int i = 0; i < N_; ++i) gv[i] = ld_stream(g + (t * N_ + i) * C8 + cv);
#pragma unroll
            for (int j = 0; j < N_; ++j) xv[j] = ld_stream(x + (t * N_ + j) * C8 + cv);
            const uint4 yv = ld_stream(y + t * C8 + cv);
            float gf[N_][8], yf[8], dyf[8];
            unpack8(yv, yf);
#pragma unroll
            for (int e = 0; e < 8; ++e) dyf[e] = 0.f;
#pragma unroll
            for (int i = 0; i < N_; ++i) {
                unpack8(gv[i], gf[i]);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    dyf[e] = fmaf(hpost[i], gf[i][e], dyf[e]);
                    r_post[i] = fmaf(gf[i][e], yf[e], r_post[i]);
                }
            }
            st_stream(dy + t * C8 + cv, pack8(dyf));
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                float xf[8];
                unpack8(xv[j], xf);
                float dxf[8];
                if (WRITE_DX) {
                    if (ACC_DX) {
                        const uint4 old = dx[(t * N_ + j) * C8 + cv];
                        unpack8(old, dxf);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) dxf[e] = 0.f;
                    }
                }
#pragma unroll
                for (int i = 0; i < N_; ++i) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        r_res[i][j] = fmaf(gf[i][e], xf[e], r_res[i][j]);
                        if (WRITE_DX) dxf[e] = fmaf(hres[i][j], gf[i][e], dxf[e]);
                    }
                }
                if (WRITE_DX) st_stream(dx + (t * N_ + j) * C8 + cv, pack8(dxf));
            }
        }
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            r_post[i] = warp_sum(r_post[i]);
#pragma unroll
            for (int j = 0; j < N_; ++j) r_res[i][j] = warp_sum(r_res[i][j]);
        }
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < N_; ++i) {
                dH_post[t * N_ + i] = r_post[i];
#pragma unroll
                for (int j = 0; j < N_; ++j) dH_res[(t * N_ + i) * N_ + j] = r_res[i][j];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Gradient of the pre-mix, one warp per token:  dH_pre[j] = <du,x_j> ; dx_j (+)= H_pre[j] du
// ------------------------------------------------------------------------------------------------
template <int N_, bool WRITE_DX, bool ACC_DX>
__global__ void __launch_bounds__(kThreads) premix_bwd_k(int64_t T, int C8, const uint4* __restrict__ x,
                                                         const float* __restrict__ H_pre, const uint4* __restrict__ du,
                                                         float* __restrict__ dH_pre, uint4* dx) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
    for (int64_t t = warp0; t < T; t += nwarps) {
        float h[N_], r[N_];
#pragma unroll
        for (int j = 0; j < N_; ++j) { h[j] = __ldg(H_pre + t * N_ + j); r[j] = 0.f; }
        for (int cv = lane; cv < C8; cv += 32) {
            uint4 xv[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) xv[j] = ld_stream(x + (t * N_ + j) * C8 + cv);
            float df[8];
            unpack8(ld_stream(du + t * C8 + cv), df);
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                float xf[8];
                unpack8(xv[j], xf);
#pragma unroll
                for (int e = 0; e < 8; ++e) r[j] = fmaf(df[e], xf[e], r[j]);
                if (WRITE_DX) {
                    float o[8];
                    if (ACC_DX) {
                        unpack8(dx[(t * N_ + j) * C8 + cv], o);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] = 0.f;
                    }
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] = fmaf(h[j], df[e], o[e]);
                    st_stream(dx + (t * N_ + j) * C8 + cv, pack8(o));
                }
            }
        }
#pragma unroll
        for (int j = 0; j < N_; ++j) r[j] = warp_sum(r[j]);
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < N_; ++j) dH_pre[t * N_ + j] = r[j];
        }
    }
}

// ------------------------------------------------------------------------------------------------
// First pass of the fused backward tail, one warp per token:
//   dH_pre[j] = <du,x_j> ;  dx_j = sum_i H_res[i][j] g_i + H_pre[j] du      (gradient of Eq. (1) w.r.t. x_l
//   with the mappings held fixed; the gradient through the mappings is added by the projection backward)
// ------------------------------------------------------------------------------------------------
template <int N_>
__global__ void __launch_bounds__(kThreads) tail_mix_k(int64_t T, int C8, const uint4* __restrict__ x,
                                                       const uint4* __restrict__ g, const uint4* __restrict__ du,
                                                       const float* __restrict__ H_res, const float* __restrict__ H_pre,
                                                       float* __restrict__ dH_pre, uint4* __restrict__ dx) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
    for (int64_t t = warp0; t < T; t += nwarps) {
        float hpre[N_], hres[N_][N_], r[N_];
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            hpre[i] = __ldg(H_pre + t * N_ + i);
            r[i] = 0.f;
#pragma unroll
            for (int j = 0; j < N_; ++j) hres[i][j] = __ldg(H_res + (t * N_ + i) * N_ + j);
        }
        for (int cv = lane; cv < C8; cv += 32) {
            uint4 gv[N_], xv[N_];
#pragma unroll
            for (int i = 0; i < N_; ++i) gv[i] = ld_stream(g + (t * N_ + i) * C8 + cv);
#pragma unroll
            for (int j = 0; j < N_; ++j) xv[j] = ld_stream(x + (t * N_ + j) * C8 + cv);
            float df[8], gf[N_][8];
            unpack8(ld_stream(du + t * C8 + cv), df);
#pragma unroll
            for (int i = 0; i < N_; ++i) unpack8(gv[i], gf[i]);
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                float xf[8], o[8];
                unpack8(xv[j], xf);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    r[j] = fmaf(df[e], xf[e], r[j]);
                    o[e] = hpre[j] * df[e];
                }
#pragma unroll
                for (int i = 0; i < N_; ++i)
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] = fmaf(hres[i][j], gf[i][e], o[e]);
                st_stream(dx + (t * N_ + j) * C8 + cv, pack8(o));
            }
        }
#pragma unroll
        for (int j = 0; j < N_; ++j) r[j] = warp_sum(r[j]);
        if (lane == 0 && dH_pre) {
#pragma unroll
            for (int j = 0; j < N_; ++j) dH_pre[t * N_ + j] = r[j];
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Doubly-stochastic gap of H_res (Section 3.1, footnote), one thread per token.
// ------------------------------------------------------------------------------------------------
__global__ void ds_gap_k(int64_t T, int n, const float* __restrict__ H, float* l1, float* cdev) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float* h = H + t * n * n;
    float err = 0.f, cmax = 0.f;
    for (int i = 0; i < n; ++i) {
        float rs = 0.f, cs = 0.f;
        for (int j = 0; j < n; ++j) { rs += h[i * n + j]; cs += h[j * n + i]; }
        err += fabsf(rs - 1.f) + fabsf(cs - 1.f);
        cmax = fmaxf(cmax, fabsf(cs - 1.f));
    }
    if (l1) l1[t] = err;
    if (cdev) cdev[t] = cmax;
}

// Product of the residual mappings over depth, one thread per token: P <- H P (later layers multiply on the
// left, as x_{l+1} = H_l x_l composes); first layer: P <- H.
__global__ void depth_product_k(int64_t T, int n, const float* __restrict__ H, float* P, int first) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float* h = H + t * n * n;
    float* p = P + t * n * n;
    float out[kMaxN * kMaxN];
    for (int i = 0; i < n; ++i)
        for (int k = 0; k < n; ++k) {
            float acc = 0.f;
            if (first) acc = h[i * n + k];
            else for (int j = 0; j < n; ++j) acc = fmaf(h[i * n + j], p[j * n + k], acc);
            out[i * n + k] = acc;
        }
    for (int e = 0; e < n * n; ++e) p[e] = out[e];
}

// Eq. (3): nu = smallest positive entry / largest entry of each n x n matrix (0 when no entry is positive).
__global__ void relative_range_k(int64_t T, int n, const float* __restrict__ X, float* __restrict__ nu) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float* x = X + t * n * n;
    float lo = 3.4e38f, hi = -3.4e38f;
    for (int e = 0; e < n * n; ++e) {
        const float v = x[e];
        hi = fmaxf(hi, v);
        if (v > 0.f) lo = fminf(lo, v);
    }
    nu[t] = (hi > 0.f) ? lo / hi : 0.f;
}

// Population statistics of the doubly-stochastic gap over all tokens in one pass (the procedure behind the paper's
// Fig. 3): stats = { max l1-error, sum of l1-errors, max column-sum deviation, sum of column-sum deviations }.
// Non-negative floats order like their bit patterns, so the maxima are integer atomics.
__global__ void __launch_bounds__(256) ds_gap_stats_k(int64_t T, int n, const float* __restrict__ H, float* stats) {
    float l1m = 0.f, l1s = 0.f, cdm = 0.f, cds = 0.f;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
        const float* h = H + t * n * n;
        float err = 0.f, cmax = 0.f;
        for (int i = 0; i < n; ++i) {
            float rs = 0.f, cs = 0.f;
            for (int j = 0; j < n; ++j) { rs += h[i * n + j]; cs += h[j * n + i]; }
            err += fabsf(rs - 1.f) + fabsf(cs - 1.f);
            cmax = fmaxf(cmax, fabsf(cs - 1.f));
        }
        l1m = fmaxf(l1m, err); l1s += err; cdm = fmaxf(cdm, cmax); cds += cmax;
    }
    l1m = warp_max(l1m); cdm = warp_max(cdm); l1s = warp_sum(l1s); cds = warp_sum(cds);
    __shared__ float red[4][8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { red[0][w] = l1m; red[1][w] = l1s; red[2][w] = cdm; red[3][w] = cds; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 1; k < 8; ++k) { red[0][0] = fmaxf(red[0][0], red[0][k]); red[1][0] += red[1][k];
                                       red[2][0] = fmaxf(red[2][0], red[2][k]); red[3][0] += red[3][k]; }
        atomicMax(reinterpret_cast<int*>(stats), __float_as_int(red[0][0]));
        atomicAdd(stats + 1, red[1][0]);
        atomicMax(reinterpret_cast<int*>(stats + 2), __float_as_int(red[2][0]));
        atomicAdd(stats + 3, red[3][0]);
    }
}

// Histogram over the tokens of log10(1 / nu), nu the relative range of Eq. (3) (the procedure behind the paper's
// Fig. 4): `bins` equal bins on [lo, hi), values outside clamped to the end bins; hist[bins] counts matrices without a
// positive entry (nu = 0).
__global__ void __launch_bounds__(256) log_inv_nu_hist_k(int64_t T, int n, const float* __restrict__ X, int bins, float lo,
                                                         float hi, unsigned long long* hist) {
    extern __shared__ unsigned int sh[];
    for (int b = threadIdx.x; b <= bins; b += blockDim.x) sh[b] = 0;
    __syncthreads();
    const float scale = (float)bins / (hi - lo);
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
        const float* x = X + t * n * n;
        float mn = 3.4e38f, mx = -3.4e38f;
        for (int e = 0; e < n * n; ++e) {
            const float v = x[e];
            mx = fmaxf(mx, v);
            if (v > 0.f) mn = fminf(mn, v);
        }
        int b = bins;
        if (mx > 0.f) {
            const float l = log10f(mx / mn);
            b = (int)floorf((l - lo) * scale);
            b = b < 0 ? 0 : (b >= bins ? bins - 1 : b);
        }
        atomicAdd(&sh[b], 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b <= bins; b += blockDim.x)
        if (sh[b]) atomicAdd(hist + b, (unsigned long long)sh[b]);
}

// ---- launchers -----------------------------------------------------------------------------------
static int grid_for(int64_t items, int sm_count, int per_sm) {
    int64_t blocks = (items + kThreads - 1) / kThreads;
    int64_t cap = (int64_t)sm_count * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

void launch_premix_fwd(const mhclite_ctx* c, int64_t T, const void* x, const float* H_pre, void* u, cudaStream_t s) {
    c->launches += 1;
    const int C8 = c->C / 8;
    const int grid = grid_for(T * C8, c->sm_count, 8);
    MHCL_DISPATCH_N(c->n, premix_fwd_k<N_><<<grid, kThreads, 0, s>>>(T, C8, (const uint4*)x, H_pre, (uint4*)u));
}

void launch_postres_fwd(const mhclite_ctx* c, int64_t T, const void* x, const void* y, const float* H_res,
                        const float* H_post, void* x_next, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_POSTRES_FWD, s);
    const int C8 = c->C / 8;
    const int grid = grid_for(T * C8, c->sm_count, 8);
    MHCL_DISPATCH_N(c->n, postres_fwd_k<N_><<<grid, kThreads, 0, s>>>(T, C8, (const uint4*)x, (const uint4*)y, H_res,
                                                                       H_post, (uint4*)x_next));
}

void launch_postres_bwd(const mhclite_ctx* c, int64_t T, const void* x, const void* y, const float* H_res,
                        const float* H_post, const void* g, void* dy, float* dH_res, float* dH_post, void* dx,
                        int acc, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_POSTRES_BWD, s);
    const int C8 = c->C / 8;
    const int grid = grid_for(T * 32, c->sm_count, 8);
#define MHCL_PB(W, A) postres_bwd_k<N_, W, A><<<grid, kThreads, 0, s>>>(T, C8, (const uint4*)x, (const uint4*)y, \
        H_res, H_post, (const uint4*)g, (uint4*)dy, dH_res, dH_post, (uint4*)dx)
    MHCL_DISPATCH_N(c->n, if (!dx) MHCL_PB(false, false); else if (acc) MHCL_PB(true, true); else MHCL_PB(true, false));
#undef MHCL_PB
}

void launch_premix_bwd(const mhclite_ctx* c, int64_t T, const void* x, const float* H_pre, const void* du,
                       float* dH_pre, void* dx, int acc, cudaStream_t s) {
    c->launches += 1;
    const int C8 = c->C / 8;
    const int grid = grid_for(T * 32, c->sm_count, 8);
#define MHCL_MB(W, A) premix_bwd_k<N_, W, A><<<grid, kThreads, 0, s>>>(T, C8, (const uint4*)x, H_pre, (const uint4*)du, \
        dH_pre, (uint4*)dx)
    MHCL_DISPATCH_N(c->n, if (!dx) MHCL_MB(false, false); else if (acc) MHCL_MB(true, true); else MHCL_MB(true, false));
#undef MHCL_MB
}

void launch_tail_mix(const mhclite_ctx* c, int64_t T, const void* x, const void* g, const void* du, const float* H_res,
                     const float* H_pre, float* dH_pre, void* dx, cudaStream_t s) {
    c->launches += 1;
    const int C8 = c->C / 8;
    const int grid = grid_for(T * 32, c->sm_count, 8);
    MHCL_DISPATCH_N(c->n, tail_mix_k<N_><<<grid, kThreads, 0, s>>>(T, C8, (const uint4*)x, (const uint4*)g, (const uint4*)du,
                                                                    H_res, H_pre, dH_pre, (uint4*)dx));
}

void launch_ds_gap(const mhclite_ctx* c, int64_t T, const float* H_res, float* l1, float* cdev, cudaStream_t s) {
    c->launches += 1;
    const int grid = (int)((T + 127) / 128);
    ds_gap_k<<<grid, 128, 0, s>>>(T, c->n, H_res, l1, cdev);
}

void launch_ds_gap_stats(const mhclite_ctx* c, int64_t T, const float* H_res, float* stats, cudaStream_t s) {
    c->launches += 1;
    cudaMemsetAsync(stats, 0, 4 * sizeof(float), s);
    int64_t blocks = (T + 255) / 256;
    if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
    ds_gap_stats_k<<<(unsigned)blocks, 256, 0, s>>>(T, c->n, H_res, stats);
}

void launch_log_inv_nu_hist(const mhclite_ctx* c, int64_t T, const float* X, int bins, float lo, float hi,
                            unsigned long long* hist, cudaStream_t s) {
    c->launches += 1;
    cudaMemsetAsync(hist, 0, (size_t)(bins + 1) * sizeof(unsigned long long), s);
    int64_t blocks = (T + 255) / 256;
    if (blocks > c->sm_count * 8) blocks = c->sm_count * 8;
    log_inv_nu_hist_k<<<(unsigned)blocks, 256, (size_t)(bins + 1) * sizeof(unsigned int), s>>>(T, c->n, X, bins, lo, hi, hist);
}

void launch_depth_product(const mhclite_ctx* c, int64_t T, const float* H_res, float* P, int first, cudaStream_t s) {
    c->launches += 1;
    depth_product_k<<<(unsigned)((T + 127) / 128), 128, 0, s>>>(T, c->n, H_res, P, first);
}

void launch_relative_range(const mhclite_ctx* c, int64_t T, const float* X, float* nu, cudaStream_t s) {
    c->launches += 1;
    relative_range_k<<<(unsigned)((T + 127) / 128), 128, 0, s>>>(T, c->n, X, nu);
}

}  // namespace mhcl
