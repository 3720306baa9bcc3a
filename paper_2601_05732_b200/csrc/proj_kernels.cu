// Gradient of the skinny projection of paper Eq. (4) and of RMSNorm -- CUDA-core (fp32 FMA) version.
// With W' = diag(gain) W:
//   dx[t,m] (+)= sum_c e[t,c] W'[m,c] - x[t,m] kappa_t       (e, kappa from the activation backward)
//   G[m,c]  = sum_t x[t,m] e[t,c] ; dW = gain (.) G ; dgain[m] = sum_c W[m,c] G[m,c]
#include "common.cuh"
#include "kernels.h"

namespace mhcl {

// ------------------------------------------------------------------------------------------------
// backward w.r.t. x: tile of 64 tokens x 64 flattened channels, columns in chunks of 32
// ------------------------------------------------------------------------------------------------
constexpr int kPbThreads = 256;

template <bool ACC>
__global__ void __launch_bounds__(kPbThreads) proj_bwd_dx_k(int64_t T, int nC, int N, int Npad,
                                                            const __nv_bfloat16* __restrict__ x,
                                                            const float* __restrict__ W, const float* __restrict__ gain,
                                                            const float* __restrict__ e, const float* __restrict__ kappa,
                                                            __nv_bfloat16* dx) {
    __shared__ __align__(16) float wt[32][64];     // W'[m0+m][c0+c] stored as [c][m]
    __shared__ float es[64][33];
    const int tid = threadIdx.x;
    const int mg = tid & 7, tg = tid >> 3;         // 8 channels per thread, 2 tokens per thread
    const int m0 = blockIdx.x * 64;
    const int64_t t0 = (int64_t)blockIdx.y * 64;
    float acc[2][8];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[a][i] = 0.f;
    for (int c0 = 0; c0 < N; c0 += 32) {
        for (int i = tid; i < 32 * 64; i += kPbThreads) {
            const int m = i >> 5, c = i & 31;      // consecutive threads read consecutive columns of a row of W
            const int mm = m0 + m, cc = c0 + c;
            wt[c][m] = (mm < nC && cc < N) ? __ldg(W + (int64_t)mm * N + cc) * __ldg(gain + mm) : 0.f;
        }
        for (int i = tid; i < 64 * 32; i += kPbThreads) {
            const int t = i >> 5, c = i & 31;
            es[t][c] = (t0 + t < T && c0 + c < N) ? e[(t0 + t) * Npad + c0 + c] : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
            const float4 w0 = *reinterpret_cast<const float4*>(&wt[c][mg * 8]);
            const float4 w1 = *reinterpret_cast<const float4*>(&wt[c][mg * 8 + 4]);
            const float wv[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
            for (int a = 0; a < 2; ++a) {
                const float ev = es[tg * 2 + a][c];
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[a][i] = fmaf(ev, wv[i], acc[a][i]);
            }
        }
        __syncthreads();
    }
    const int m = m0 + mg * 8;
    if (m >= nC) return;
#pragma unroll
    for (int a = 0; a < 2; ++a) {
        const int64_t t = t0 + tg * 2 + a;
        if (t >= T) continue;
        float xf[8], o[8];
        unpack8(*reinterpret_cast<const uint4*>(x + t * nC + m), xf);
        const float kp = __ldg(kappa + t);
        if (ACC) unpack8(*reinterpret_cast<const uint4*>(dx + t * nC + m), o);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float v = fmaf(-xf[i], kp, acc[a][i]);
            o[i] = ACC ? o[i] + v : v;
        }
        *reinterpret_cast<uint4*>(dx + t * nC + m) = pack8(o);
    }
}

// ------------------------------------------------------------------------------------------------
// backward w.r.t. W: G[m,c] += sum over this block's tokens of x[t,m] e[t,c]
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) proj_bwd_dw_k(int64_t T, int nC, int N, int Npad, int64_t tok_per_split,
                                                     const __nv_bfloat16* __restrict__ x, const float* __restrict__ e,
                                                     float* G) {
    __shared__ float xs[32][64];
    __shared__ __align__(16) float es[32][32];
    const int tid = threadIdx.x;
    const int m = tid & 63, cq = tid >> 6;          // 64 channels x 4 groups of 8 columns
    const int m0 = blockIdx.x * 64, c0 = blockIdx.y * 32;
    const int64_t ta = (int64_t)blockIdx.z * tok_per_split;
    const int64_t tb = (ta + tok_per_split < T) ? ta + tok_per_split : T;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int64_t t0 = ta; t0 < tb; t0 += 32) {
        {   // x chunk: 32 tokens x 64 channels = 256 vectors of 8
            const int t = tid >> 3, pc = tid & 7;
            float f[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (t0 + t < tb && m0 + pc * 8 < nC) unpack8(*reinterpret_cast<const uint4*>(x + (t0 + t) * nC + m0 + pc * 8), f);
#pragma unroll
            for (int i = 0; i < 8; ++i) xs[t][pc * 8 + i] = f[i];
        }
        for (int i = tid; i < 32 * 32; i += 256) {
            const int t = i >> 5, c = i & 31;
            es[t][c] = (t0 + t < tb && c0 + c < N) ? e[(t0 + t) * Npad + c0 + c] : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int t = 0; t < 32; ++t) {
            const float xv = xs[t][m];
            const float4 e0 = *reinterpret_cast<const float4*>(&es[t][cq * 8]);
            const float4 e1 = *reinterpret_cast<const float4*>(&es[t][cq * 8 + 4]);
            acc[0] = fmaf(xv, e0.x, acc[0]); acc[1] = fmaf(xv, e0.y, acc[1]);
            acc[2] = fmaf(xv, e0.z, acc[2]); acc[3] = fmaf(xv, e0.w, acc[3]);
            acc[4] = fmaf(xv, e1.x, acc[4]); acc[5] = fmaf(xv, e1.y, acc[5]);
            acc[6] = fmaf(xv, e1.z, acc[6]); acc[7] = fmaf(xv, e1.w, acc[7]);
        }
        __syncthreads();
    }
    if (m0 + m < nC) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = c0 + cq * 8 + i;
            if (c < N) atomicAdd(G + (int64_t)(m0 + m) * Npad + c, acc[i]);
        }
    }
}

// dW (+)= gain (.) G ; dgain[m] (+)= sum_c W[m,c] G[m,c].  One warp per row m.
template <bool ACC>
__global__ void __launch_bounds__(256) proj_bwd_finish_k(int nC, int N, int Npad, const float* __restrict__ W,
                                                         const float* __restrict__ gain, const float* __restrict__ G,
                                                         float* dW, float* dgain) {
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (m >= nC) return;
    const float gm = __ldg(gain + m);
    float dg = 0.f;
    for (int c = lane; c < N; c += 32) {
        const float gv = G[(int64_t)m * Npad + c];
        const int64_t i = (int64_t)m * N + c;
        dW[i] = ACC ? dW[i] + gm * gv : gm * gv;
        dg = fmaf(__ldg(W + i), gv, dg);
    }
    dg = warp_sum(dg);
    if (lane == 0) dgain[m] = ACC ? dgain[m] + dg : dg;
}

// ---- launchers -----------------------------------------------------------------------------------
void launch_proj_bwd_dx(const mhclite_ctx* c, int64_t T, int N, int Npad, const void* x, const float* W,
                        const float* gain, const float* e, const float* kappa, void* dx, int acc, cudaStream_t s) {
    c->launches += 1;
    const int nC = c->n * c->C;
    dim3 grid((nC + 63) / 64, (unsigned)((T + 63) / 64));
    if (acc)
        proj_bwd_dx_k<true><<<grid, kPbThreads, 0, s>>>(T, nC, N, Npad, (const __nv_bfloat16*)x, W, gain, e, kappa,
                                                         (__nv_bfloat16*)dx);
    else
        proj_bwd_dx_k<false><<<grid, kPbThreads, 0, s>>>(T, nC, N, Npad, (const __nv_bfloat16*)x, W, gain, e, kappa,
                                                          (__nv_bfloat16*)dx);
}

void launch_proj_bwd_dw(const mhclite_ctx* c, int64_t T, int N, int Npad, const void* x, const float* W,
                        const float* gain, const float* e, float* G, float* dW, float* dgain, int acc,
                        cudaStream_t s) {
    c->launches += 1;
    const int nC = c->n * c->C;
    cudaMemsetAsync(G, 0, (size_t)nC * Npad * sizeof(float), s);
    const int mt = (nC + 63) / 64, ct = (N + 31) / 32;
    int64_t splits = ((int64_t)c->sm_count * 4 + mt * ct - 1) / (mt * ct);
    const int64_t max_splits = (T + 255) / 256;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    const int64_t per = round_up64((T + splits - 1) / splits, 32);
    splits = (T + per - 1) / per;
    dim3 grid(mt, ct, (unsigned)splits);
    proj_bwd_dw_k<<<grid, 256, 0, s>>>(T, nC, N, Npad, per, (const __nv_bfloat16*)x, e, G);
    const int fg = (nC + 7) / 8;
    if (acc) proj_bwd_finish_k<true><<<fg, 256, 0, s>>>(nC, N, Npad, W, gain, G, dW, dgain);
    else proj_bwd_finish_k<false><<<fg, 256, 0, s>>>(nC, N, Npad, W, gain, G, dW, dgain);
}

}  // namespace mhcl
