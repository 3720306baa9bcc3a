// Per-token activations of the dynamic mappings and their gradients.
//
// mHC-lite (paper Eq. (4), (5)): z = alpha (.) p + b ; H_pre = sigmoid ; H_post = 2 sigmoid ;
// a = softmax(z_res) ; H_res = sum_k a_k P_k.  One warp per token: lanes hold the logits, the softmax
// reductions are warp shuffles, and H_res[i][j] is the sum of the (n-1)! weights whose permutation
// sends i to j (constant-memory index lists).
//
// mHC (paper Eq. (2)): H_res = SK(exp(mat(z_res))), `iters` x (normalise columns, then rows); one
// thread per token with the n x n matrix in registers.  The backward stores only the 2*iters*n
// normalisers and walks the iterates back (X = Y * s), instead of keeping every iterate.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"

namespace mhcl {

// Where the activation backward leaves e = rstd * alpha (.) dz for the projection backward: as fp32 rows
// (CUDA-core kernels) and / or as a bf16 pair hi + lo (tensor-core kernel).  Null pointers are skipped.
struct EOut {
    float* e; int Npad;
    __nv_bfloat16 *ehi, *elo; int Kp;
};
__device__ __forceinline__ void store_e(const EOut& o, int64_t t, int c, float v) {
    if (o.e) o.e[t * o.Npad + c] = v;
    if (o.ehi) {
        __nv_bfloat16 h, l;
        split_bf16(v, h, l);
        o.ehi[t * o.Kp + c] = h;
        o.elo[t * o.Kp + c] = l;
    }
}
__device__ __forceinline__ void pad_e(const EOut& o, int64_t t, int N, int first, int step) {
    if (o.e) for (int c = N + first; c < o.Npad; c += step) o.e[t * o.Npad + c] = 0.f;
    if (o.ehi) for (int c = N + first; c < o.Kp; c += step) {
        o.ehi[t * o.Kp + c] = __float2bfloat16_rn(0.f);
        o.elo[t * o.Kp + c] = __float2bfloat16_rn(0.f);
    }
}

constexpr int kActThreads = 256;
constexpr int kActWarps = kActThreads / 32;
constexpr int kMaxCols = kMaxFact + 2 * kMaxN;   // 130

__device__ __forceinline__ float sigmoidf_(float z) { return 1.f / (1.f + expf(-z)); }

// ------------------------------------------------------------------------------------------------
// Adds the K-slice partials of the projection, applies rstd and stores p_saved / rstd for one token.
// Returns p for the columns this lane owns: col = lane + 32 s.
__device__ __forceinline__ void finish_projection(int64_t t, int64_t T, int N, int Npad, int ksplit, float inv_nC,
                                                  float eps, const float* __restrict__ qpart,
                                                  const float* __restrict__ ssq, float* __restrict__ p_saved,
                                                  float* __restrict__ rstd, int lane, float (&pv)[5]) {
    float ss = 0.f;
    for (int s = 0; s < ksplit; ++s) ss += __ldg(ssq + (int64_t)s * T + t);
    const float r = 1.f / sqrtf(ss * inv_nC + eps);
    if (lane == 0) rstd[t] = r;
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const int c = lane + 32 * k;
        pv[k] = 0.f;
        if (c < N) {
            float q = 0.f;
            for (int s = 0; s < ksplit; ++s) q += __ldg(qpart + ((int64_t)s * T + t) * Npad + c);
            pv[k] = r * q;
            p_saved[t * N + c] = pv[k];
        }
    }
}

__global__ void __launch_bounds__(kActThreads) lite_act_fwd_k(int64_t T, int n, int nf, int Npad, int ksplit,
                                                             float inv_nC, float eps, const float* __restrict__ qpart,
                                                             const float* __restrict__ ssq,
                                                             const float* __restrict__ b, const float* __restrict__ alpha,
                                                             float* __restrict__ H_res, float* __restrict__ H_pre,
                                                             float* __restrict__ H_post, float* __restrict__ a_saved,
                                                             float* __restrict__ p_saved, float* __restrict__ rstd) {
    __shared__ float a_s[kActWarps][kMaxFact + 8];
    __shared__ float p_s[kActWarps][kMaxCols + 6];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int N = nf + 2 * n, per = nf / n, nn = n * n;
    const PermTables& tab = c_perm[n];
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    const int64_t nwarps = (int64_t)gridDim.x * kActWarps;
    for (int64_t t = (int64_t)blockIdx.x * kActWarps + w; t < T; t += nwarps) {
        float pv[5];
        finish_projection(t, T, N, Npad, ksplit, inv_nC, eps, qpart, ssq, p_saved, rstd, lane, pv);
#pragma unroll
        for (int k = 0; k < 5; ++k) if (lane + 32 * k < N) p_s[w][lane + 32 * k] = pv[k];
        __syncwarp();
        const float* pt = p_s[w];
        float z[4], m = -INFINITY;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int k = lane + 32 * s;
            z[s] = -INFINITY;
            if (k < nf) { z[s] = fmaf(a_res, pt[k], __ldg(b + k)); m = fmaxf(m, z[s]); }
        }
        m = warp_max(m);
        float sum = 0.f;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            z[s] = (lane + 32 * s < nf) ? expf(z[s] - m) : 0.f;
            sum += z[s];
        }
        sum = warp_sum(sum);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int k = lane + 32 * s;
            if (k < nf) {
                const float a = z[s] / sum;
                a_s[w][k] = a;
                a_saved[t * nf + k] = a;
            }
        }
        if (lane < 2 * n) {
            const int c = nf + lane;
            const float zz = fmaf(lane < n ? a_pre : a_post, pt[c], __ldg(b + c));
            const float sg = sigmoidf_(zz);
            if (lane < n) H_pre[t * n + lane] = sg; else H_post[t * n + lane - n] = 2.f * sg;
        }
        __syncwarp();
        if (lane < nn) {
            float h = 0.f;
            for (int r = 0; r < per; ++r) h += a_s[w][tab.klist[lane * per + r]];
            H_res[t * nn + lane] = h;
        }
        __syncwarp();
    }
}

// Shared tail of both backward kernels: from dz of one column to e, kappa, db, dalpha partials.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kActThreads) lite_act_bwd_k(
    int64_t T, int n, int nf, float inv_nC, const float* __restrict__ a_saved, const float* __restrict__ p,
    const float* __restrict__ rstd, const float* __restrict__ alpha, const float* __restrict__ H_pre,
    const float* __restrict__ H_post, const float* __restrict__ dH_res, const float* __restrict__ dH_pre,
    const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa, float* db, float* dalpha) {
    __shared__ float dh_s[kActWarps][32];
    __shared__ float red[kActWarps][kMaxCols + 3];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int N = nf + 2 * n, nn = n * n;
    const PermTables& tab = c_perm[n];
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    float db_res[4] = {0, 0, 0, 0}, db_gate = 0.f, dal_res = 0.f, dal_gate = 0.f;
    const int64_t nwarps = (int64_t)gridDim.x * kActWarps;
    for (int64_t t = (int64_t)blockIdx.x * kActWarps + w; t < T; t += nwarps) {
        const float* pt = p + t * N;
        const float rs = __ldg(rstd + t);
        if (lane < nn) dh_s[w][lane] = dH_res[t * nn + lane];
        __syncwarp();
        float a[4], da[4], dot = 0.f;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int k = lane + 32 * s;
            a[s] = 0.f; da[s] = 0.f;
            if (k < nf) {
                a[s] = a_saved[t * nf + k];
                float d = 0.f;
                for (int i = 0; i < n; ++i) d += dh_s[w][i * n + tab.sigma[k * n + i]];   // Eq. (5): dL/da_k
                da[s] = d;
                dot = fmaf(a[s], d, dot);
            }
        }
        dot = warp_sum(dot);
        float kap = 0.f;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            const int k = lane + 32 * s;
            if (k < nf) {
                const float dz = a[s] * (da[s] - dot);
                const float ed = a_res * dz, pv = pt[k];
                store_e(eo, t, k, rs * ed);
                kap = fmaf(ed, pv, kap);
                db_res[s] += dz;
                dal_res = fmaf(dz, pv, dal_res);
            }
        }
        if (lane < 2 * n) {
            const int c = nf + lane;
            float dz;
            if (lane < n) { const float h = H_pre[t * n + lane]; dz = dH_pre[t * n + lane] * h * (1.f - h); }
            else { const float h = H_post[t * n + lane - n]; dz = dH_post[t * n + lane - n] * h * (1.f - 0.5f * h); }
            const float ed = (lane < n ? a_pre : a_post) * dz, pv = pt[c];
            store_e(eo, t, c, rs * ed);
            kap = fmaf(ed, pv, kap);
            db_gate += dz;
            dal_gate = fmaf(dz, pv, dal_gate);
        }
        pad_e(eo, t, N, lane, 32);
        kap = warp_sum(kap);
        if (lane == 0) kappa[t] = rs * rs * kap * inv_nC;
        __syncwarp();
    }
    // block reduction of the parameter-gradient partials, then one atomic per column per block
#pragma unroll
    for (int s = 0; s < 4; ++s) if (lane + 32 * s < nf) red[w][lane + 32 * s] = db_res[s];
    if (lane < 2 * n) red[w][nf + lane] = db_gate;
    const float d0 = warp_sum(dal_res);
    const float d1 = warp_sum(lane < n ? dal_gate : 0.f);
    const float d2 = warp_sum((lane >= n && lane < 2 * n) ? dal_gate : 0.f);
    if (lane == 0) { red[w][N] = d0; red[w][N + 1] = d1; red[w][N + 2] = d2; }
    __syncthreads();
    for (int c = threadIdx.x; c < N + 3; c += kActThreads) {
        float v = 0.f;
#pragma unroll
        for (int ww = 0; ww < kActWarps; ++ww) v += red[ww][c];
        if (c < N) atomicAdd(db + c, v); else atomicAdd(dalpha + (c - N), v);
    }
}

// ------------------------------------------------------------------------------------------------
template <int N_>
__device__ __forceinline__ void sk_forward(float (&M)[N_][N_], int iters, float* cs_store, float* rs_store) {
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < N_; ++j) {
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < N_; ++i) s += M[i][j];
            if (cs_store) cs_store[it * N_ + j] = s;
#pragma unroll
            for (int i = 0; i < N_; ++i) M[i][j] = M[i][j] / s;
        }
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < N_; ++j) s += M[i][j];
            if (rs_store) rs_store[it * N_ + i] = s;
#pragma unroll
            for (int j = 0; j < N_; ++j) M[i][j] = M[i][j] / s;
        }
    }
}

template <int N_>
__device__ __forceinline__ void sk_load_m0(const float* pt, const float* b, float a_res, float (&M)[N_][N_]) {
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < N_; ++i)
#pragma unroll
        for (int j = 0; j < N_; ++j) {
            M[i][j] = fmaf(a_res, pt[i * N_ + j], __ldg(b + i * N_ + j));
            m = fmaxf(m, M[i][j]);
        }
#pragma unroll
    for (int i = 0; i < N_; ++i)
#pragma unroll
        for (int j = 0; j < N_; ++j) M[i][j] = expf(M[i][j] - m);
}

template <int N_>
__global__ void __launch_bounds__(128) sk_act_fwd_k(int64_t T, int iters, int Npad, int ksplit, float inv_nC, float eps,
                                                    const float* __restrict__ qpart, const float* __restrict__ ssq,
                                                    const float* __restrict__ b, const float* __restrict__ alpha,
                                                    float* __restrict__ H_res, float* __restrict__ H_pre,
                                                    float* __restrict__ H_post, float* __restrict__ p_saved,
                                                    float* __restrict__ rstd) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    constexpr int N = N_ * N_ + 2 * N_;
    float ss = 0.f;
    for (int s = 0; s < ksplit; ++s) ss += __ldg(ssq + (int64_t)s * T + t);
    const float r = 1.f / sqrtf(ss * inv_nC + eps);
    rstd[t] = r;
    float pt[N];
#pragma unroll
    for (int c = 0; c < N; ++c) {
        float q = 0.f;
        for (int s = 0; s < ksplit; ++s) q += __ldg(qpart + ((int64_t)s * T + t) * Npad + c);
        pt[c] = r * q;
        p_saved[t * N + c] = pt[c];
    }
    float M[N_][N_];
    sk_load_m0<N_>(pt, b, __ldg(alpha), M);
    sk_forward<N_>(M, iters, nullptr, nullptr);
#pragma unroll
    for (int i = 0; i < N_; ++i)
#pragma unroll
        for (int j = 0; j < N_; ++j) H_res[t * N_ * N_ + i * N_ + j] = M[i][j];
    const float a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
#pragma unroll
    for (int j = 0; j < N_; ++j) {
        H_pre[t * N_ + j] = sigmoidf_(fmaf(a_pre, pt[N_ * N_ + j], __ldg(b + N_ * N_ + j)));
        H_post[t * N_ + j] = 2.f * sigmoidf_(fmaf(a_post, pt[N_ * N_ + N_ + j], __ldg(b + N_ * N_ + N_ + j)));
    }
}

constexpr int kSkMaxIters = 64;

template <int N_>
__global__ void __launch_bounds__(128) sk_act_bwd_k(
    int64_t T, int iters, float inv_nC, const float* __restrict__ p, const float* __restrict__ b,
    const float* __restrict__ rstd, const float* __restrict__ alpha, const float* __restrict__ H_pre,
    const float* __restrict__ H_post, const float* __restrict__ dH_res, const float* __restrict__ dH_pre,
    const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa, float* db, float* dalpha) {
    constexpr int N = N_ * N_ + 2 * N_;
    __shared__ float red[N + 3];
    for (int c = threadIdx.x; c < N + 3; c += blockDim.x) red[c] = 0.f;
    __syncthreads();
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < T) {
        const float* pt = p + t * N;
        const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
        float cs[kSkMaxIters * N_], rs[kSkMaxIters * N_];
        float Y[N_][N_];
        sk_load_m0<N_>(pt, b, a_res, Y);
        sk_forward<N_>(Y, iters, cs, rs);
        float d[N_][N_];
#pragma unroll
        for (int i = 0; i < N_; ++i)
#pragma unroll
            for (int j = 0; j < N_; ++j) d[i][j] = dH_res[t * N_ * N_ + i * N_ + j];
        for (int it = iters - 1; it >= 0; --it) {
            // rows: Y = X / s  ->  dX = (dY - <dY,Y>_row) / s ; X = Y s
#pragma unroll
            for (int i = 0; i < N_; ++i) {
                const float s = rs[it * N_ + i];
                float dot = 0.f;
#pragma unroll
                for (int j = 0; j < N_; ++j) dot = fmaf(d[i][j], Y[i][j], dot);
#pragma unroll
                for (int j = 0; j < N_; ++j) { d[i][j] = (d[i][j] - dot) / s; Y[i][j] *= s; }
            }
            // columns
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                const float s = cs[it * N_ + j];
                float dot = 0.f;
#pragma unroll
                for (int i = 0; i < N_; ++i) dot = fmaf(d[i][j], Y[i][j], dot);
#pragma unroll
                for (int i = 0; i < N_; ++i) { d[i][j] = (d[i][j] - dot) / s; Y[i][j] *= s; }
            }
        }
        // through exp: dz = dM0 * M0, with M0 taken from the logits again (not from the walk-back)
        sk_load_m0<N_>(pt, b, a_res, Y);
        const float r = __ldg(rstd + t);
        float kap = 0.f, dal0 = 0.f, dal1 = 0.f, dal2 = 0.f;
#pragma unroll
        for (int i = 0; i < N_; ++i)
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                const int c = i * N_ + j;
                const float dz = d[i][j] * Y[i][j], pv = pt[c], ed = a_res * dz;
                store_e(eo, t, c, r * ed);
                kap = fmaf(ed, pv, kap);
                dal0 = fmaf(dz, pv, dal0);
                atomicAdd(&red[c], dz);
            }
#pragma unroll
        for (int j = 0; j < N_; ++j) {
            {
                const int c = N_ * N_ + j;
                const float h = H_pre[t * N_ + j];
                const float dz = dH_pre[t * N_ + j] * h * (1.f - h), pv = pt[c], ed = a_pre * dz;
                store_e(eo, t, c, r * ed); kap = fmaf(ed, pv, kap); dal1 = fmaf(dz, pv, dal1);
                atomicAdd(&red[c], dz);
            }
            {
                const int c = N_ * N_ + N_ + j;
                const float h = H_post[t * N_ + j];
                const float dz = dH_post[t * N_ + j] * h * (1.f - 0.5f * h), pv = pt[c], ed = a_post * dz;
                store_e(eo, t, c, r * ed); kap = fmaf(ed, pv, kap); dal2 = fmaf(dz, pv, dal2);
                atomicAdd(&red[c], dz);
            }
        }
        pad_e(eo, t, N, 0, 1);
        kappa[t] = r * r * kap * inv_nC;
        atomicAdd(&red[N], dal0); atomicAdd(&red[N + 1], dal1); atomicAdd(&red[N + 2], dal2);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < N + 3; c += blockDim.x) {
        if (c < N) atomicAdd(db + c, red[c]); else atomicAdd(dalpha + (c - N), red[c]);
    }
}

// ---- launchers -----------------------------------------------------------------------------------
static int warp_grid(int64_t T, int sm_count) {
    int64_t blocks = (T + kActWarps - 1) / kActWarps;
    const int64_t cap = (int64_t)sm_count * 8;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

void launch_lite_act_fwd(const mhclite_ctx* c, int64_t T, const ProjPlan& pp, const float* qpart, const float* ssq,
                         float eps, const float* b, const float* alpha, float* H_res, float* H_pre, float* H_post,
                         float* a_saved, float* p_saved, float* rstd, cudaStream_t s) {
    c->launches += 1;
    lite_act_fwd_k<<<warp_grid(T, c->sm_count), kActThreads, 0, s>>>(
        T, c->n, c->nfact, pp.Npad, pp.ksplit, 1.f / (float)(c->n * c->C), eps, qpart, ssq, b, alpha, H_res, H_pre,
        H_post, a_saved, p_saved, rstd);
}

void launch_lite_act_bwd(const mhclite_ctx* c, int64_t T, int Npad, const float* a, const float* p, const float* rstd,
                         const float* alpha, const float* H_pre, const float* H_post, const float* dH_res,
                         const float* dH_pre, const float* dH_post, float* e, void* ehi, void* elo, int Kp,
                         float* kappa, float* db, float* dalpha, cudaStream_t s) {
    const EOut eo{e, Npad, (__nv_bfloat16*)ehi, (__nv_bfloat16*)elo, Kp};
    c->launches += 1;
    // fewer, longer-lived blocks: the parameter-gradient partials are reduced once per block
    int64_t blocks = (T + kActWarps * 8 - 1) / (kActWarps * 8);
    if (blocks > c->sm_count * 4) blocks = c->sm_count * 4;
    if (blocks < 1) blocks = 1;
    lite_act_bwd_k<<<(int)blocks, kActThreads, 0, s>>>(T, c->n, c->nfact, 1.f / (float)(c->n * c->C), a, p, rstd,
                                                        alpha, H_pre, H_post, dH_res, dH_pre, dH_post, eo, kappa, db,
                                                        dalpha);
}

void launch_sk_act_fwd(const mhclite_ctx* c, int64_t T, int iters, const ProjPlan& pp, const float* qpart,
                       const float* ssq, float eps, const float* b, const float* alpha, float* H_res, float* H_pre,
                       float* H_post, float* p_saved, float* rstd, cudaStream_t s) {
    c->launches += 1;
    const int grid = (int)((T + 127) / 128);
    const float inv = 1.f / (float)(c->n * c->C);
    MHCL_DISPATCH_N(c->n, sk_act_fwd_k<N_><<<grid, 128, 0, s>>>(T, iters, pp.Npad, pp.ksplit, inv, eps, qpart, ssq, b,
                                                                 alpha, H_res, H_pre, H_post, p_saved, rstd));
}

void launch_sk_act_bwd(const mhclite_ctx* c, int64_t T, int Npad, int iters, const float* p, const float* b,
                       const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                       const float* dH_res, const float* dH_pre, const float* dH_post, float* e, void* ehi, void* elo,
                       int Kp, float* kappa, float* db, float* dalpha, cudaStream_t s) {
    const EOut eo{e, Npad, (__nv_bfloat16*)ehi, (__nv_bfloat16*)elo, Kp};
    c->launches += 1;
    const int grid = (int)((T + 127) / 128);
    const float inv = 1.f / (float)(c->n * c->C);
    MHCL_DISPATCH_N(c->n, sk_act_bwd_k<N_><<<grid, 128, 0, s>>>(T, iters, inv, p, b, rstd, alpha, H_pre, H_post,
                                                                  dH_res, dH_pre, dH_post, eo, kappa, db, dalpha));
}

}  // namespace mhcl
