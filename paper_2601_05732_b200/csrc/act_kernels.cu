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
        const int64_t i = e_tiled_index(o.Kp, t, c);
        o.ehi[i] = h;
        o.elo[i] = l;
    }
}
__device__ __forceinline__ void pad_e(const EOut& o, int64_t t, int N, int first, int step) {
    if (o.e) for (int c = N + first; c < o.Npad; c += step) o.e[t * o.Npad + c] = 0.f;
    if (o.ehi) for (int c = N + first; c < o.Kp; c += step) {
        const int64_t i = e_tiled_index(o.Kp, t, c);
        o.ehi[i] = __float2bfloat16_rn(0.f);
        o.elo[i] = __float2bfloat16_rn(0.f);
    }
}

// Tokens past T in the last 128-token granule of the tiled e buffers are read by the tensor-core kernels:
// the granule is cleared before the activation backward fills its valid part.
static void clear_e_tail(int64_t T, void* ehi, void* elo, int Kp, cudaStream_t s) {
    if (!ehi || (T % kEGranule) == 0) return;
    const size_t gbytes = (size_t)Kp * kEGranule * 2, off = (size_t)(T / kEGranule) * gbytes;
    cudaMemsetAsync((char*)ehi + off, 0, gbytes, s);
    cudaMemsetAsync((char*)elo + off, 0, gbytes, s);
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

// Per-block shared state of the mHC-lite activation kernels.  The permutation tables are copied from
// constant memory once per block: lanes index them with different addresses, which the constant cache
// would serialise.
struct LiteShared {
    uint8_t sigma[kMaxFact * kMaxN];
    uint8_t klist[kMaxN * kMaxN * 24];
    float a_s[kActWarps][kMaxFact + 8];
    float p_s[kActWarps][kMaxCols + 6];
    float dh_s[kActWarps][32];
    float red[kActWarps][kMaxCols + 3];
};
// `table` (global memory, [nf][n]) replaces the constant-memory table when the context holds a subset of the
// permutations (paper Section 5); there are then no per-entry index lists, and H_res is assembled from sigma.
__device__ __forceinline__ void load_tables(LiteShared& sh, int n, int nf, const uint8_t* __restrict__ table) {
    if (table) {
        for (int i = threadIdx.x; i < nf * n; i += blockDim.x) sh.sigma[i] = table[i];
    } else {
        const PermTables& tab = c_perm[n];
        for (int i = threadIdx.x; i < kMaxFact * kMaxN; i += blockDim.x) { sh.sigma[i] = tab.sigma[i]; sh.klist[i] = tab.klist[i]; }
    }
    __syncthreads();
}

// Forward of one token by one warp, given its normalised projection row pt[0..N) (shared memory):
// z = alpha p + b, sigmoid gates, softmax, H_res = sum_k a_k P_k.
// Returns the gate of this lane: H_pre[lane] for lane < n, H_post[lane - n] for n <= lane < 2n.
__device__ __forceinline__ float lite_token_fwd_core(LiteShared& sh, int w, int lane, int64_t t, int n, int nf,
                                                     const float* pt, const float* __restrict__ b, float a_res,
                                                     float a_pre, float a_post, float* __restrict__ H_res,
                                                     float* __restrict__ H_pre, float* __restrict__ H_post,
                                                     float* __restrict__ a_saved, bool subset = false) {
    const int per = nf / n, nn = n * n;
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
            sh.a_s[w][k] = a;
            a_saved[t * nf + k] = a;
        }
    }
    float gate = 0.f;
    if (lane < 2 * n) {
        const int c = nf + lane;
        const float zz = fmaf(lane < n ? a_pre : a_post, pt[c], __ldg(b + c));
        gate = sigmoidf_(zz);
        if (lane < n) H_pre[t * n + lane] = gate; else { gate *= 2.f; H_post[t * n + lane - n] = gate; }
    }
    __syncwarp();
    if (lane < nn) {
        float h = 0.f;
        if (subset) {                                   // Eq. (5) over the table's rows: P_k[i][sigma_k(i)] = 1
            const int i = lane / n, j = lane - i * n;
            for (int k = 0; k < nf; ++k) h += (sh.sigma[k * n + i] == j) ? sh.a_s[w][k] : 0.f;
        } else {
            for (int r = 0; r < per; ++r) h += sh.a_s[w][sh.klist[lane * per + r]];
        }
        H_res[t * nn + lane] = h;
    }
    __syncwarp();
    return gate;
}

// The same, starting from the K-slice partials of the projection in global memory.
__device__ __forceinline__ float lite_token_fwd(LiteShared& sh, int w, int lane, int64_t t, int64_t T, int n, int nf,
                                                int Npad, int ksplit, float inv_nC, float eps,
                                                const float* __restrict__ qpart, const float* __restrict__ ssq,
                                                const float* __restrict__ b, float a_res, float a_pre, float a_post,
                                                float* __restrict__ H_res, float* __restrict__ H_pre,
                                                float* __restrict__ H_post, float* __restrict__ a_saved,
                                                float* __restrict__ p_saved, float* __restrict__ rstd, bool subset) {
    const int N = nf + 2 * n;
    float pv[5];
    finish_projection(t, T, N, Npad, ksplit, inv_nC, eps, qpart, ssq, p_saved, rstd, lane, pv);
#pragma unroll
    for (int k = 0; k < 5; ++k) if (lane + 32 * k < N) sh.p_s[w][lane + 32 * k] = pv[k];
    __syncwarp();
    return lite_token_fwd_core(sh, w, lane, t, n, nf, sh.p_s[w], b, a_res, a_pre, a_post, H_res, H_pre, H_post, a_saved,
                               subset);
}

__global__ void __launch_bounds__(kActThreads) lite_act_fwd_k(int64_t T, int n, int nf, int Npad, int ksplit,
                                                             float inv_nC, float eps, const float* __restrict__ qpart,
                                                             const float* __restrict__ ssq,
                                                             const float* __restrict__ b, const float* __restrict__ alpha,
                                                             float* __restrict__ H_res, float* __restrict__ H_pre,
                                                             float* __restrict__ H_post, float* __restrict__ a_saved,
                                                             float* __restrict__ p_saved, float* __restrict__ rstd,
                                                             const uint8_t* __restrict__ table) {
    __shared__ LiteShared sh;
    load_tables(sh, n, nf, table);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    const int64_t nwarps = (int64_t)gridDim.x * kActWarps;
    for (int64_t t = (int64_t)blockIdx.x * kActWarps + w; t < T; t += nwarps)
        lite_token_fwd(sh, w, lane, t, T, n, nf, Npad, ksplit, inv_nC, eps, qpart, ssq, b, a_res, a_pre, a_post,
                       H_res, H_pre, H_post, a_saved, p_saved, rstd, table != nullptr);
}

// Mappings + stream pre-mix in one kernel, in groups of kGroupTok tokens per block:
//   L: the group's projection partials are added, normalised and staged in shared memory by all threads
//      (one round of coalesced loads, so the per-token math below waits on no global load);
//   A: one warp per token: gates, softmax, H_res;
//   P: all threads stream the group's tokens: u[t,:] = sum_j H_pre[t,j] x[t,j,:]   (Eq. (1), inner term).
// Eight tokens (one per warp) and a grid of resident blocks only: a block then walks many groups, so that the blocks of
// an SM drift apart and one block's mappings run under the others' streaming.  (With 32-token groups and one or two
// groups per block, all blocks of a wave went through their phases together and HBM idled during L and A.)
constexpr int kGroupTok = 8;

template <int N_>
__global__ void __launch_bounds__(kActThreads, 4) lite_act_premix_k(
    int64_t T, int C8, int nf, int Npad, int ksplit, float inv_nC, float eps, const float* __restrict__ qpart,
    const float* __restrict__ ssq, const float* __restrict__ b, const float* __restrict__ alpha,
    float* __restrict__ H_res, float* __restrict__ H_pre, float* __restrict__ H_post, float* __restrict__ a_saved,
    float* __restrict__ p_saved, float* __restrict__ rstd, const uint4* __restrict__ x, uint4* __restrict__ u,
    const uint8_t* __restrict__ table) {
    __shared__ LiteShared sh;
    __shared__ float pg[kGroupTok][kMaxCols + 3];
    __shared__ float rg[kGroupTok];
    __shared__ float hg[kGroupTok][kMaxN];
    load_tables(sh, N_, nf, table);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int N = nf + 2 * N_;
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    const int64_t ngroups = (T + kGroupTok - 1) / kGroupTok;
    for (int64_t grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
        // descending: the projection kernel before this one read x in ascending order and left its last lines in L2
        const int64_t t0 = (ngroups - 1 - grp) * kGroupTok;
        const int nt = (T - t0 < kGroupTok) ? (int)(T - t0) : kGroupTok;
        // L
        if (tid < nt) {
            float ss = 0.f;
            for (int s = 0; s < ksplit; ++s) ss += __ldg(ssq + (int64_t)s * T + t0 + tid);
            const float r = 1.f / sqrtf(ss * inv_nC + eps);
            rg[tid] = r;
            rstd[t0 + tid] = r;
        }
        for (int i = tid; i < nt * N; i += kActThreads) {
            const int tl = i / N, c = i - tl * N;
            float q = 0.f;
            for (int s = 0; s < ksplit; ++s) q += __ldg(qpart + ((int64_t)s * T + t0 + tl) * Npad + c);
            pg[tl][c] = q;
        }
        __syncthreads();
        for (int i = tid; i < nt * N; i += kActThreads) {
            const int tl = i / N, c = i - tl * N;
            const float pv = pg[tl][c] * rg[tl];
            pg[tl][c] = pv;
            p_saved[(t0 + tl) * N + c] = pv;
        }
        __syncthreads();
        // A
        for (int tl = w; tl < nt; tl += kActWarps) {
            const float gate = lite_token_fwd_core(sh, w, lane, t0 + tl, N_, nf, pg[tl], b, a_res, a_pre, a_post, H_res,
                                                   H_pre, H_post, a_saved, table != nullptr);
            if (lane < N_) hg[tl][lane] = gate;
        }
        __syncthreads();
        // P (two vectors per thread in flight: the loads of the second are issued before the first is used)
        for (int i0 = tid; i0 < nt * C8; i0 += 2 * kActThreads) {
            const int i1 = i0 + kActThreads;
            const bool has1 = i1 < nt * C8;
            const int tl0 = i0 / C8, cv0 = i0 - tl0 * C8;
            const int tl1 = has1 ? i1 / C8 : tl0, cv1 = has1 ? i1 - tl1 * C8 : cv0;
            uint4 v0[N_], v1[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) v0[j] = ld_stream(x + ((t0 + tl0) * N_ + j) * C8 + cv0);
#pragma unroll
            for (int j = 0; j < N_; ++j) v1[j] = ld_stream(x + ((t0 + tl1) * N_ + j) * C8 + cv1);
            {
                float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
                for (int j = 0; j < N_; ++j) {
                    const float h = hg[tl0][j];
                    float f[8];
                    unpack8(v0[j], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(h, f[e], acc[e]);
                }
                st_stream(u + (t0 + tl0) * C8 + cv0, pack8(acc));
            }
            if (has1) {
                float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
                for (int j = 0; j < N_; ++j) {
                    const float h = hg[tl1][j];
                    float f[8];
                    unpack8(v1[j], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(h, f[e], acc[e]);
                }
                st_stream(u + (t0 + tl1) * C8 + cv1, pack8(acc));
            }
        }
        __syncthreads();
    }
}

// Backward of one token by one warp (gradient of Eq. (4), (5)): from dH_res, dH_post (global) and this
// lane's dH_pre (lane j < n holds dH_pre[j]) to e = rstd alpha dz, kappa, and the db / dalpha partials.
struct LiteBwdAcc { float db_res[4], db_gate, dal_res, dal_gate; };

__device__ __forceinline__ void lite_token_bwd(LiteShared& sh, int w, int lane, int64_t t, int n, int nf, float inv_nC,
                                               const float* a_tok, const float* pt, float rs, float a_res, float a_pre,
                                               float a_post, const float* hpre_tok, const float* hpost_tok,
                                               const float* dhres_tok, float dhpre_lane, const float* dhpost_tok,
                                               const EOut& eo, float* __restrict__ kappa, LiteBwdAcc& acc) {
    // *_tok point at this token's rows (global or shared memory)
    const int N = nf + 2 * n, nn = n * n;
    if (lane < nn) sh.dh_s[w][lane] = dhres_tok[lane];
    __syncwarp();
    float a[4], da[4], dot = 0.f;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int k = lane + 32 * s;
        a[s] = 0.f; da[s] = 0.f;
        if (k < nf) {
            a[s] = a_tok[k];
            float d = 0.f;
            for (int i = 0; i < n; ++i) d += sh.dh_s[w][i * n + sh.sigma[k * n + i]];   // Eq. (5): dL/da_k
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
            acc.db_res[s] += dz;
            acc.dal_res = fmaf(dz, pv, acc.dal_res);
        }
    }
    if (lane < 2 * n) {
        const int c = nf + lane;
        float dz;
        if (lane < n) { const float h = hpre_tok[lane]; dz = dhpre_lane * h * (1.f - h); }
        else { const float h = hpost_tok[lane - n]; dz = dhpost_tok[lane - n] * h * (1.f - 0.5f * h); }
        const float ed = (lane < n ? a_pre : a_post) * dz, pv = pt[c];
        store_e(eo, t, c, rs * ed);
        kap = fmaf(ed, pv, kap);
        acc.db_gate += dz;
        acc.dal_gate = fmaf(dz, pv, acc.dal_gate);
    }
    pad_e(eo, t, N, lane, 32);
    kap = warp_sum(kap);
    if (lane == 0) kappa[t] = rs * rs * kap * inv_nC;
    __syncwarp();
}

// Block reduction of the parameter-gradient partials, then one atomic per column per block.
__device__ __forceinline__ void lite_bwd_reduce(LiteShared& sh, int w, int lane, int n, int nf, const LiteBwdAcc& acc,
                                                float* db, float* dalpha) {
    const int N = nf + 2 * n;
#pragma unroll
    for (int s = 0; s < 4; ++s) if (lane + 32 * s < nf) sh.red[w][lane + 32 * s] = acc.db_res[s];
    if (lane < 2 * n) sh.red[w][nf + lane] = acc.db_gate;
    const float d0 = warp_sum(acc.dal_res);
    const float d1 = warp_sum(lane < n ? acc.dal_gate : 0.f);
    const float d2 = warp_sum((lane >= n && lane < 2 * n) ? acc.dal_gate : 0.f);
    if (lane == 0) { sh.red[w][N] = d0; sh.red[w][N + 1] = d1; sh.red[w][N + 2] = d2; }
    __syncthreads();
    for (int c = threadIdx.x; c < N + 3; c += kActThreads) {
        float v = 0.f;
#pragma unroll
        for (int ww = 0; ww < kActWarps; ++ww) v += sh.red[ww][c];
        if (c < N) atomicAdd(db + c, v); else atomicAdd(dalpha + (c - N), v);
    }
}

__global__ void __launch_bounds__(kActThreads) lite_act_bwd_k(
    int64_t T, int n, int nf, float inv_nC, const float* __restrict__ a_saved, const float* __restrict__ p,
    const float* __restrict__ rstd, const float* __restrict__ alpha, const float* __restrict__ H_pre,
    const float* __restrict__ H_post, const float* __restrict__ dH_res, const float* __restrict__ dH_pre,
    const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa, float* db, float* dalpha,
    const uint8_t* __restrict__ table) {
    __shared__ LiteShared sh;
    load_tables(sh, n, nf, table);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    LiteBwdAcc acc = {{0, 0, 0, 0}, 0.f, 0.f, 0.f};
    const int64_t nwarps = (int64_t)gridDim.x * kActWarps;
    for (int64_t t = (int64_t)blockIdx.x * kActWarps + w; t < T; t += nwarps) {
        const float dhp = (lane < n) ? dH_pre[t * n + lane] : 0.f;
        lite_token_bwd(sh, w, lane, t, n, nf, inv_nC, a_saved + t * nf, p + t * (nf + 2 * n), __ldg(rstd + t), a_res,
                       a_pre, a_post, H_pre + t * n, H_post + t * n, dH_res + t * n * n, dhp, dH_post + t * n, eo,
                       kappa, acc);
    }
    lite_bwd_reduce(sh, w, lane, n, nf, acc, db, dalpha);
}

// First kernel of the fused backward tail, in groups of kGroupTok tokens per block:
//   L: the per-token inputs of the activation backward are copied to shared memory with cp.async
//      (they arrive while D streams);
//   D: one warp per token streams x and du: dH_pre[j] = <du, x_j>;
//   A: one warp per token: activation backward from shared memory (no global load on the way).
// (one token's staged inputs, as floats: a | p | dH_res | H_pre | H_post | dH_post | rstd)
template <int N_>
__global__ void __launch_bounds__(kActThreads, 4) lite_tailpre_k(
    int64_t T, int C8, int nf, float inv_nC, const uint4* __restrict__ x, const uint4* __restrict__ du,
    const float* __restrict__ a_saved, const float* __restrict__ p, const float* __restrict__ rstd,
    const float* __restrict__ alpha, const float* __restrict__ H_pre, const float* __restrict__ H_post,
    const float* __restrict__ dH_res, const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa,
    float* db, float* dalpha, const uint8_t* __restrict__ table) {
    __shared__ LiteShared sh;
    constexpr int NN = N_ * N_;
    constexpr int kFact = (N_ == 2) ? 2 : (N_ == 3) ? 6 : (N_ == 4) ? 24 : 120;
    constexpr int kStride = kFact + (kFact + 2 * N_) + NN + 3 * N_ + 1 + 1;
    constexpr int kGroupTok = 8;                               // one token per warp; see lite_act_premix_k
    __shared__ float in_s[kGroupTok][kStride];
    __shared__ float dhp_s[kGroupTok][kMaxN];
    load_tables(sh, N_, nf, table);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int N = nf + 2 * N_;
    const int o_p = nf, o_dhres = o_p + N, o_hpre = o_dhres + NN, o_hpost = o_hpre + N_, o_dhpost = o_hpost + N_,
              o_rstd = o_dhpost + N_, nin = o_rstd + 1;
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    LiteBwdAcc acc = {{0, 0, 0, 0}, 0.f, 0.f, 0.f};
    const int64_t ngroups = (T + kGroupTok - 1) / kGroupTok;
    for (int64_t grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
        const int64_t t0 = grp * kGroupTok;
        const int nt = (T - t0 < kGroupTok) ? (int)(T - t0) : kGroupTok;
        // L
        for (int i = tid; i < nt * nin; i += kActThreads) {
            const int tl = i / nin, c = i - tl * nin;
            const int64_t t = t0 + tl;
            const float* src;
            if (c < o_p) src = a_saved + t * nf + c;
            else if (c < o_dhres) src = p + t * N + (c - o_p);
            else if (c < o_hpre) src = dH_res + t * NN + (c - o_dhres);
            else if (c < o_hpost) src = H_pre + t * N_ + (c - o_hpre);
            else if (c < o_dhpost) src = H_post + t * N_ + (c - o_hpost);
            else if (c < o_rstd) src = dH_post + t * N_ + (c - o_dhpost);
            else src = rstd + t;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(&in_s[tl][c])), "l"(src) : "memory");
        }
        cp_async_commit();
        // D
        for (int tl = w; tl < nt; tl += kActWarps) {
            const int64_t t = t0 + tl;
            float r[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) r[j] = 0.f;
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
                }
            }
#pragma unroll
            for (int j = 0; j < N_; ++j) { r[j] = warp_sum(r[j]); if (lane == j) dhp_s[tl][j] = r[j]; }
        }
        cp_async_wait<0>();
        __syncthreads();
        // A
        for (int tl = w; tl < nt; tl += kActWarps) {
            const float* in = in_s[tl];
            const float dhp = (lane < N_) ? dhp_s[tl][lane] : 0.f;
            lite_token_bwd(sh, w, lane, t0 + tl, N_, nf, inv_nC, in, in + o_p, in[o_rstd], a_res, a_pre, a_post,
                           in + o_hpre, in + o_hpost, in + o_dhres, dhp, in + o_dhpost, eo, kappa, acc);
        }
        __syncthreads();
    }
    lite_bwd_reduce(sh, w, lane, N_, nf, acc, db, dalpha);
}

// ------------------------------------------------------------------------------------------------
// Thread-per-token versions for n <= 4 (n! <= 24 logits fit in registers).  A warp working on one token
// spends ~500 dependent instructions on shuffles and reductions; a thread working on one token spends a
// similar count for 32 tokens at once.  Inputs and outputs are staged in shared memory so that global
// traffic stays coalesced.
// ------------------------------------------------------------------------------------------------
template <int N_>
struct LiteDims {
    static constexpr int kFact = (N_ == 2) ? 2 : (N_ == 3) ? 6 : 24;
    static constexpr int kN = kFact + 2 * N_;
    static constexpr int kNN = N_ * N_;
    static constexpr int kPer = kFact / N_;
    static constexpr int kOut = kFact + kNN + 2 * N_;        // a | H_res | H_pre | H_post
    static constexpr int kIn = kFact + kN + kNN + 3 * N_ + 1; // a | p | dH_res | H_pre | H_post | dH_post | rstd
};

// The lexicographic permutation table as a compile-time constant: with the loops below fully unrolled
// every index into it is a constant, so the Birkhoff sum and its gradient become plain register adds.
template <int N_>
struct PermConst { unsigned char s[LiteDims<N_>::kFact][N_]; };

template <int N_>
__host__ __device__ constexpr PermConst<N_> make_perm_const() {
    PermConst<N_> t{};
    int cur[N_] = {};
    for (int i = 0; i < N_; ++i) cur[i] = i;
    for (int k = 0; k < LiteDims<N_>::kFact; ++k) {
        for (int i = 0; i < N_; ++i) t.s[k][i] = (unsigned char)cur[i];
        int a = N_ - 2;                              // successor in lexicographic order
        while (a >= 0 && cur[a] > cur[a + 1]) --a;
        if (a < 0) break;
        int b = N_ - 1;
        while (cur[b] < cur[a]) --b;
        int tmp = cur[a]; cur[a] = cur[b]; cur[b] = tmp;
        for (int lo = a + 1, hi = N_ - 1; lo < hi; ++lo, --hi) { tmp = cur[lo]; cur[lo] = cur[hi]; cur[hi] = tmp; }
    }
    return t;
}

template <int N_>
__device__ __forceinline__ void lite_thread_fwd(const float* prow, float* orow, const float* b_s, float a_res,
                                                float a_pre, float a_post, const uint8_t* klist_s) {
    using D = LiteDims<N_>;
    float z[D::kFact], m = -INFINITY;
#pragma unroll
    for (int k = 0; k < D::kFact; ++k) { z[k] = fmaf(a_res, prow[k], b_s[k]); m = fmaxf(m, z[k]); }
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < D::kFact; ++k) { z[k] = expf(z[k] - m); sum += z[k]; }
    constexpr PermConst<N_> tab = make_perm_const<N_>();
    (void)klist_s;
    float h[D::kNN];
#pragma unroll
    for (int e = 0; e < D::kNN; ++e) h[e] = 0.f;
#pragma unroll
    for (int k = 0; k < D::kFact; ++k) {
        const float a = z[k] / sum;
        orow[k] = a;
#pragma unroll
        for (int i = 0; i < N_; ++i) h[i * N_ + tab.s[k][i]] += a;          // Eq. (5): P_k[i][sigma_k(i)] = 1
    }
#pragma unroll
    for (int e = 0; e < D::kNN; ++e) orow[D::kFact + e] = h[e];
#pragma unroll
    for (int j = 0; j < N_; ++j) {
        orow[D::kFact + D::kNN + j] = sigmoidf_(fmaf(a_pre, prow[D::kFact + j], b_s[D::kFact + j]));
        orow[D::kFact + D::kNN + N_ + j] = 2.f * sigmoidf_(fmaf(a_post, prow[D::kFact + N_ + j], b_s[D::kFact + N_ + j]));
    }
}

constexpr int kTokGroup = 32;    // tokens per block iteration of the thread-per-token kernels

template <int N_, int GT, bool USTAT>
__global__ void __launch_bounds__(kActThreads, 3) lite_act_premix_t_k(
    int64_t T, int C8, int Npad, int ksplit, float inv_nC, float eps, const float* __restrict__ qpart,
    const float* __restrict__ ssq, const float* __restrict__ b, const float* __restrict__ alpha,
    float* __restrict__ H_res, float* __restrict__ H_pre, float* __restrict__ H_post, float* __restrict__ a_saved,
    float* __restrict__ p_saved, float* __restrict__ rstd, const uint4* __restrict__ x, uint4* __restrict__ u, float* __restrict__ u_rstd, float eps_u) {
    // USTAT: also u_rstd[t] = (mean_c u[t,c]^2 + eps_u)^-1/2 of the stored (rounded) u: the statistic of the RMSNorm that
    // usually opens the sublayer, so that the caller applies it as a row scale without another pass over u.
    // GT <= kTokGroup tokens per group: small when there are few tokens, so that every block walks several groups
    constexpr int gtok = GT;
    using D = LiteDims<N_>;
    __shared__ uint8_t klist_s[D::kNN * D::kPer];
    __shared__ float b_s[D::kN];
    __shared__ float pg[GT][D::kN + 1];
    __shared__ float og[GT][D::kOut + 1];
    __shared__ float rg[GT];
    const int tid = threadIdx.x;
    for (int i = tid; i < D::kNN * D::kPer; i += kActThreads) klist_s[i] = c_perm[N_].klist[i];
    for (int i = tid; i < D::kN; i += kActThreads) b_s[i] = __ldg(b + i);
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    __syncthreads();
    const int64_t ngroups = (T + gtok - 1) / gtok;
    for (int64_t grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
        // descending: the projection kernel before this one read x in ascending order and left its last lines in L2
        const int64_t t0 = (ngroups - 1 - grp) * gtok;
        const int nt = (T - t0 < gtok) ? (int)(T - t0) : gtok;
        // L: partials -> normalised projection rows in shared memory (and p_saved, rstd)
        if (tid < nt) {
            float ss = 0.f;
            for (int s = 0; s < ksplit; ++s) ss += __ldg(ssq + (int64_t)s * T + t0 + tid);
            const float r = 1.f / sqrtf(ss * inv_nC + eps);
            rg[tid] = r;
            rstd[t0 + tid] = r;
        }
        float qv[(GT * D::kN + kActThreads - 1) / kActThreads];
#pragma unroll
        for (int it = 0; it < (GT * D::kN + kActThreads - 1) / kActThreads; ++it) {
            const int i = tid + it * kActThreads;
            qv[it] = 0.f;
            if (i < nt * D::kN) {
                const int tl = i / D::kN, c = i - tl * D::kN;
                for (int s = 0; s < ksplit; ++s) qv[it] += __ldg(qpart + ((int64_t)s * T + t0 + tl) * Npad + c);
            }
        }
        __syncthreads();
#pragma unroll
        for (int it = 0; it < (GT * D::kN + kActThreads - 1) / kActThreads; ++it) {
            const int i = tid + it * kActThreads;
            if (i < nt * D::kN) {
                const int tl = i / D::kN, c = i - tl * D::kN;
                const float pv = qv[it] * rg[tl];
                pg[tl][c] = pv;
                p_saved[(t0 + tl) * D::kN + c] = pv;
            }
        }
        __syncthreads();
        // A: one thread per token
        if (tid < nt) lite_thread_fwd<N_>(pg[tid], og[tid], b_s, a_res, a_pre, a_post, klist_s);
        __syncthreads();
        // W: coalesced write-out of the mappings
        for (int i = tid; i < nt * D::kOut; i += kActThreads) {
            const int tl = i / D::kOut, c = i - tl * D::kOut;
            const int64_t t = t0 + tl;
            const float v = og[tl][c];
            if (c < D::kFact) a_saved[t * D::kFact + c] = v;
            else if (c < D::kFact + D::kNN) H_res[t * D::kNN + (c - D::kFact)] = v;
            else if (c < D::kFact + D::kNN + N_) H_pre[t * N_ + (c - D::kFact - D::kNN)] = v;
            else H_post[t * N_ + (c - D::kFact - D::kNN - N_)] = v;
        }
        // P: u[t,:] = sum_j H_pre[t,j] x[t,j,:]  (two vectors per thread in flight)
        if (USTAT) {
            // one warp per token here, so that a lane sums the squares of its own vectors in a register and the warp adds
            // them up once per token (warp-wide sums per vector, or shared-memory atomics, cost far more)
            const int lane = tid & 31;
            for (int tl = tid >> 5; tl < nt; tl += kActWarps) {
                const int64_t t = t0 + tl;
                float h[N_];
#pragma unroll
                for (int j = 0; j < N_; ++j) h[j] = og[tl][D::kFact + D::kNN + j];
                float sq = 0.f;
                for (int cv0 = lane; cv0 < C8; cv0 += 64) {
                    const bool has1 = cv0 + 32 < C8;
                    const int cv1 = has1 ? cv0 + 32 : cv0;
                    uint4 v0[N_], v1[N_];
#pragma unroll
                    for (int j = 0; j < N_; ++j) v0[j] = ld_stream(x + (t * N_ + j) * C8 + cv0);
#pragma unroll
                    for (int j = 0; j < N_; ++j) v1[j] = ld_stream(x + (t * N_ + j) * C8 + cv1);
                    float acc0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, acc1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
                    for (int j = 0; j < N_; ++j) {
                        float f0[8], f1[8];
                        unpack8(v0[j], f0);
                        unpack8(v1[j], f1);
#pragma unroll
                        for (int e = 0; e < 8; ++e) { acc0[e] = fmaf(h[j], f0[e], acc0[e]); acc1[e] = fmaf(h[j], f1[e], acc1[e]); }
                    }
                    const uint4 pk0 = pack8(acc0), pk1 = pack8(acc1);
                    st_stream(u + t * C8 + cv0, pk0);
                    if (has1) st_stream(u + t * C8 + cv1, pk1);
                    float r0[8], r1[8], s1 = 0.f;
                    unpack8(pk0, r0);                          // the statistic is over the values as stored
                    unpack8(pk1, r1);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { sq = fmaf(r0[e], r0[e], sq); s1 = fmaf(r1[e], r1[e], s1); }
                    if (has1) sq += s1;
                }
                sq = warp_sum(sq);                             // every lane of the warp is here: the token loop is warp-uniform
                if (lane == 0) u_rstd[t] = 1.f / sqrtf(sq / (float)(C8 * 8) + eps_u);
            }
        }
        const int total = USTAT ? 0 : nt * C8;
        for (int i0 = tid; i0 < total; i0 += 2 * kActThreads) {
            const int i1 = i0 + kActThreads;
            const bool has1 = i1 < total;
            const int tl0 = i0 / C8, cv0 = i0 - tl0 * C8;
            const int tl1 = has1 ? i1 / C8 : tl0, cv1 = has1 ? i1 - tl1 * C8 : cv0;
            uint4 v0[N_], v1[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) v0[j] = ld_stream(x + ((t0 + tl0) * N_ + j) * C8 + cv0);
#pragma unroll
            for (int j = 0; j < N_; ++j) v1[j] = ld_stream(x + ((t0 + tl1) * N_ + j) * C8 + cv1);
            float acc0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, acc1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                const float h0 = og[tl0][D::kFact + D::kNN + j], h1 = og[tl1][D::kFact + D::kNN + j];
                float f0[8], f1[8];
                unpack8(v0[j], f0);
                unpack8(v1[j], f1);
#pragma unroll
                for (int e = 0; e < 8; ++e) { acc0[e] = fmaf(h0, f0[e], acc0[e]); acc1[e] = fmaf(h1, f1[e], acc1[e]); }
            }
            st_stream(u + (t0 + tl0) * C8 + cv0, pack8(acc0));
            if (has1) st_stream(u + (t0 + tl1) * C8 + cv1, pack8(acc1));
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// First kernel of the fused backward tail for n <= 4 (n! + 2n <= 32 columns), one warp per token and one
// lane per projection column.  The warp streams x and du of its token for dH_pre[j] = <du, x_j> (gradient of
// Eq. (1) w.r.t. H_pre); the per-token inputs of the activation backward were requested before the stream
// and have arrived by its end.  Lane c then holds column c of the gradient of Eq. (4), (5):
//   res columns k: da_k = sum_i dH_res[i][sigma_k(i)], dz_k = a_k (da_k - <a, da>)   (the dot product is a warp sum)
//   pre / post columns: the sigmoid derivatives, dH_pre taken from the warp's own reduction
// e = rstd alpha (.) dz goes out as the tiled bf16 pair (and / or fp32 rows), kappa = rstd^2 sum_c alpha dz p / (nC)
// is a second warp sum, and the lane keeps its column of db and of sum_t dz p in registers until the end.
constexpr int kTpwVec = 2;      // 16-byte vectors per lane and tensor in flight

template <int N_>
__global__ void __launch_bounds__(256, 4) lite_tailpre_w_k(
    int64_t T, int C8, float inv_nC, const uint4* __restrict__ x, const uint4* __restrict__ du,
    const float* __restrict__ a_saved, const float* __restrict__ p, const float* __restrict__ rstd,
    const float* __restrict__ alpha, const float* __restrict__ H_pre, const float* __restrict__ H_post,
    const float* __restrict__ dH_res, const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa,
    float* db, float* dalpha) {
    using D = LiteDims<N_>;
    __shared__ float red[2][8][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int c = lane;
    const bool is_res = c < D::kFact, is_pre = !is_res && c < D::kFact + N_, is_post = !is_res && !is_pre && c < D::kN;
    const int jj = is_pre ? c - D::kFact : (is_post ? c - D::kFact - N_ : 0);
    int sg[N_];
#pragma unroll
    for (int i = 0; i < N_; ++i) sg[i] = is_res ? i * N_ + c_perm[N_].sigma[c * N_ + i] : 0;
    const float al = __ldg(alpha + (is_res ? 0 : (is_pre ? 1 : 2)));
    float db_c = 0.f, dal_c = 0.f;
    const int64_t warp0 = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * 256) >> 5;
    for (int64_t t = warp0; t < T; t += nwarps) {
        // per-token inputs of lane c, in flight during the stream
        const float av = is_res ? __ldg(a_saved + t * D::kFact + c) : 0.f;
        const float pv = c < D::kN ? __ldg(p + t * D::kN + c) : 0.f;
        const float rs = __ldg(rstd + t);
        float d = 0.f;
        if (is_res) {
#pragma unroll
            for (int i = 0; i < N_; ++i) d += __ldg(dH_res + t * D::kNN + sg[i]);          // Eq. (5): dL/da_k
        }
        const float h = is_pre ? __ldg(H_pre + t * N_ + jj) : (is_post ? __ldg(H_post + t * N_ + jj) : 0.f);
        const float dhp = is_post ? __ldg(dH_post + t * N_ + jj) : 0.f;
        float r[N_];
#pragma unroll
        for (int j = 0; j < N_; ++j) r[j] = 0.f;
        for (int cv0 = lane; cv0 < C8; cv0 += 32 * kTpwVec) {
            uint4 xv[kTpwVec][N_], dv[kTpwVec];
#pragma unroll
            for (int v = 0; v < kTpwVec; ++v) {
                const int cv = cv0 + 32 * v;
                if (cv < C8) {
#pragma unroll
                    for (int j = 0; j < N_; ++j) xv[v][j] = ld_stream(x + (t * N_ + j) * C8 + cv);
                    dv[v] = ld_stream(du + t * C8 + cv);
                } else {
#pragma unroll
                    for (int j = 0; j < N_; ++j) xv[v][j] = make_uint4(0, 0, 0, 0);
                    dv[v] = make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int v = 0; v < kTpwVec; ++v) {
                float df[8];
                unpack8(dv[v], df);
#pragma unroll
                for (int j = 0; j < N_; ++j) {
                    float xf[8];
                    unpack8(xv[v][j], xf);
#pragma unroll
                    for (int e = 0; e < 8; ++e) r[j] = fmaf(df[e], xf[e], r[j]);
                }
            }
        }
        float rj = 0.f;
#pragma unroll
        for (int j = 0; j < N_; ++j) { r[j] = warp_sum(r[j]); if (jj == j) rj = r[j]; }
        const float dot = warp_sum(av * d);
        float dz = 0.f;
        if (is_res) dz = av * (d - dot);
        else if (is_pre) dz = rj * h * (1.f - h);
        else if (is_post) dz = dhp * h * (1.f - 0.5f * h);
        const float ed = al * dz;
        const float kap = warp_sum(ed * pv);
        const float ev = rs * ed;
        db_c += dz;
        dal_c = fmaf(dz, pv, dal_c);
        if (eo.ehi && c < eo.Kp) {
            __nv_bfloat16 hi, lo;
            split_bf16(ev, hi, lo);
            const int64_t o = e_tiled_index(eo.Kp, t, c);
            eo.ehi[o] = hi;
            eo.elo[o] = lo;
        }
        if (eo.e && c < eo.Npad) eo.e[t * eo.Npad + c] = ev;
        if (lane == 0) kappa[t] = rs * rs * kap * inv_nC;
    }
    // parameter-gradient partials of this block: columns over the warps, then one atomic per column
    red[0][w][lane] = db_c;
    red[1][w][lane] = dal_c;
    __syncthreads();
    if (w == 0) {
        float sdb = 0.f, sdal = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) { sdb += red[0][k][lane]; sdal += red[1][k][lane]; }
        const float s_res = warp_sum(is_res ? sdal : 0.f), s_pre = warp_sum(is_pre ? sdal : 0.f),
                    s_post = warp_sum(is_post ? sdal : 0.f);
        if (dalpha) {
            if (c < D::kN) atomicAdd(db + c, sdb);
            if (lane == 0) { atomicAdd(dalpha, s_res); atomicAdd(dalpha + 1, s_pre); atomicAdd(dalpha + 2, s_post); }
        } else {                                           // per-block partials, summed by tail_finish_k
            float* part = db + (int64_t)blockIdx.x * kPartStride;
            if (c < D::kN) part[c] = sdb;
            if (lane == 0) { part[D::kN] = s_res; part[D::kN + 1] = s_pre; part[D::kN + 2] = s_post; }
        }
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
            const float r = 1.f / s;                     // one division per column / row, n multiplications
#pragma unroll
            for (int i = 0; i < N_; ++i) M[i][j] *= r;
        }
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < N_; ++j) s += M[i][j];
            if (rs_store) rs_store[it * N_ + i] = s;
            const float r = 1.f / s;
#pragma unroll
            for (int j = 0; j < N_; ++j) M[i][j] *= r;
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

// Backward of one token through the SK path (one thread): recomputes the forward keeping the 2 * iters * n
// normalisers, walks the iterates back (X = Y s), goes through exp, and emits e = rstd alpha dz, kappa and the
// token's contributions to db / dalpha (shared-memory accumulators red[N + 3]).
template <int N_>
__device__ __forceinline__ void sk_token_bwd(int64_t t, int iters, float inv_nC, const float* pt, const float* __restrict__ b,
                                             float r, float a_res, float a_pre, float a_post, const float* hpre,
                                             const float* hpost, const float* dhres, const float* dhpre,
                                             const float* dhpost, const EOut& eo, float* __restrict__ kappa, float* red) {
    constexpr int N = N_ * N_ + 2 * N_;
    float cs[kSkMaxIters * N_], rs[kSkMaxIters * N_];
    float Y[N_][N_];
    sk_load_m0<N_>(pt, b, a_res, Y);
    sk_forward<N_>(Y, iters, cs, rs);
    float d[N_][N_];
#pragma unroll
    for (int i = 0; i < N_; ++i)
#pragma unroll
        for (int j = 0; j < N_; ++j) d[i][j] = dhres[i * N_ + j];
    for (int it = iters - 1; it >= 0; --it) {
        // rows: Y = X / s  ->  dX = (dY - <dY,Y>_row) / s ; X = Y s
#pragma unroll
        for (int i = 0; i < N_; ++i) {
            const float s = rs[it * N_ + i], rinv = 1.f / s;
            float dot = 0.f;
#pragma unroll
            for (int j = 0; j < N_; ++j) dot = fmaf(d[i][j], Y[i][j], dot);
#pragma unroll
            for (int j = 0; j < N_; ++j) { d[i][j] = (d[i][j] - dot) * rinv; Y[i][j] *= s; }
        }
        // columns
#pragma unroll
        for (int j = 0; j < N_; ++j) {
            const float s = cs[it * N_ + j], rinv = 1.f / s;
            float dot = 0.f;
#pragma unroll
            for (int i = 0; i < N_; ++i) dot = fmaf(d[i][j], Y[i][j], dot);
#pragma unroll
            for (int i = 0; i < N_; ++i) { d[i][j] = (d[i][j] - dot) * rinv; Y[i][j] *= s; }
        }
    }
    // through exp: dz = dM0 * M0, with M0 taken from the logits again (not from the walk-back)
    sk_load_m0<N_>(pt, b, a_res, Y);
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
            const float h = hpre[j];
            const float dz = dhpre[j] * h * (1.f - h), pv = pt[c], ed = a_pre * dz;
            store_e(eo, t, c, r * ed); kap = fmaf(ed, pv, kap); dal1 = fmaf(dz, pv, dal1);
            atomicAdd(&red[c], dz);
        }
        {
            const int c = N_ * N_ + N_ + j;
            const float h = hpost[j];
            const float dz = dhpost[j] * h * (1.f - 0.5f * h), pv = pt[c], ed = a_post * dz;
            store_e(eo, t, c, r * ed); kap = fmaf(ed, pv, kap); dal2 = fmaf(dz, pv, dal2);
            atomicAdd(&red[c], dz);
        }
    }
    pad_e(eo, t, N, 0, 1);
    kappa[t] = r * r * kap * inv_nC;
    atomicAdd(&red[N], dal0); atomicAdd(&red[N + 1], dal1); atomicAdd(&red[N + 2], dal2);
}

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
    if (t < T)
        sk_token_bwd<N_>(t, iters, inv_nC, p + t * N, b, __ldg(rstd + t), __ldg(alpha), __ldg(alpha + 1), __ldg(alpha + 2),
                         H_pre + t * N_, H_post + t * N_, dH_res + t * N_ * N_, dH_pre + t * N_, dH_post + t * N_, eo,
                         kappa, red);
    __syncthreads();
    for (int c = threadIdx.x; c < N + 3; c += blockDim.x) {
        if (c < N) atomicAdd(db + c, red[c]); else atomicAdd(dalpha + (c - N), red[c]);
    }
}

// ------------------------------------------------------------------------------------------------
// The SK path's fused kernels, built like the mHC-lite ones so that the comparison is like for like:
// sk_act_premix_k = SK activation + stream pre-mix (one thread per token for the 20 iterations, then all threads
// stream the group's tokens); sk_tailpre_k = dH_pre stream (one warp per token) + SK backward (one thread per token).
// ------------------------------------------------------------------------------------------------
constexpr int kSkGroup = 64;     // tokens per block iteration (GS below: 64, or 32 / 16 when there are few tokens)

template <int N_, int GS>
__global__ void __launch_bounds__(kActThreads, 3) sk_act_premix_k(
    int64_t T, int C8, int iters, int Npad, int ksplit, float inv_nC, float eps, const float* __restrict__ qpart,
    const float* __restrict__ ssq, const float* __restrict__ b, const float* __restrict__ alpha,
    float* __restrict__ H_res, float* __restrict__ H_pre, float* __restrict__ H_post, float* __restrict__ p_saved,
    float* __restrict__ rstd, const uint4* __restrict__ x, uint4* __restrict__ u) {
    constexpr int NN = N_ * N_, N = NN + 2 * N_;
    __shared__ float pg[GS][N + 1];
    __shared__ float og[GS][N + 1];          // H_res | H_pre | H_post
    __shared__ float rg[GS];
    const int tid = threadIdx.x;
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    const int64_t ngroups = (T + GS - 1) / GS;
    for (int64_t grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
        // descending: the projection kernel before this one read x in ascending order and left its last lines in L2
        const int64_t t0 = (ngroups - 1 - grp) * GS;
        const int nt = (T - t0 < GS) ? (int)(T - t0) : GS;
        if (tid < nt) {
            float ss = 0.f;
            for (int s = 0; s < ksplit; ++s) ss += __ldg(ssq + (int64_t)s * T + t0 + tid);
            const float r = 1.f / sqrtf(ss * inv_nC + eps);
            rg[tid] = r;
            rstd[t0 + tid] = r;
        }
        __syncthreads();
        for (int i = tid; i < nt * N; i += kActThreads) {
            const int tl = i / N, c = i - tl * N;
            float q = 0.f;
            for (int s = 0; s < ksplit; ++s) q += __ldg(qpart + ((int64_t)s * T + t0 + tl) * Npad + c);
            const float pv = q * rg[tl];
            pg[tl][c] = pv;
            p_saved[(t0 + tl) * N + c] = pv;
        }
        __syncthreads();
        if (tid < nt) {                            // one thread per token: exp, the SK iterations, the gates
            float M[N_][N_];
            sk_load_m0<N_>(pg[tid], b, a_res, M);
            sk_forward<N_>(M, iters, nullptr, nullptr);
#pragma unroll
            for (int i = 0; i < N_; ++i)
#pragma unroll
                for (int j = 0; j < N_; ++j) og[tid][i * N_ + j] = M[i][j];
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                og[tid][NN + j] = sigmoidf_(fmaf(a_pre, pg[tid][NN + j], __ldg(b + NN + j)));
                og[tid][NN + N_ + j] = 2.f * sigmoidf_(fmaf(a_post, pg[tid][NN + N_ + j], __ldg(b + NN + N_ + j)));
            }
        }
        __syncthreads();
        for (int i = tid; i < nt * N; i += kActThreads) {
            const int tl = i / N, c = i - tl * N;
            const int64_t t = t0 + tl;
            const float v = og[tl][c];
            if (c < NN) H_res[t * NN + c] = v;
            else if (c < NN + N_) H_pre[t * N_ + (c - NN)] = v;
            else H_post[t * N_ + (c - NN - N_)] = v;
        }
        // u[t,:] = sum_j H_pre[t,j] x[t,j,:]  (two vectors per thread in flight)
        for (int i0 = tid; i0 < nt * C8; i0 += 2 * kActThreads) {
            const int i1 = i0 + kActThreads;
            const bool has1 = i1 < nt * C8;
            const int tl0 = i0 / C8, cv0 = i0 - tl0 * C8;
            const int tl1 = has1 ? i1 / C8 : tl0, cv1 = has1 ? i1 - tl1 * C8 : cv0;
            uint4 v0[N_], v1[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) v0[j] = ld_stream(x + ((t0 + tl0) * N_ + j) * C8 + cv0);
#pragma unroll
            for (int j = 0; j < N_; ++j) v1[j] = ld_stream(x + ((t0 + tl1) * N_ + j) * C8 + cv1);
            float acc0[8] = {0, 0, 0, 0, 0, 0, 0, 0}, acc1[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int j = 0; j < N_; ++j) {
                const float h0 = og[tl0][NN + j], h1 = og[tl1][NN + j];
                float f0[8], f1[8];
                unpack8(v0[j], f0);
                unpack8(v1[j], f1);
#pragma unroll
                for (int e = 0; e < 8; ++e) { acc0[e] = fmaf(h0, f0[e], acc0[e]); acc1[e] = fmaf(h1, f1[e], acc1[e]); }
            }
            st_stream(u + (t0 + tl0) * C8 + cv0, pack8(acc0));
            if (has1) st_stream(u + (t0 + tl1) * C8 + cv1, pack8(acc1));
        }
        __syncthreads();
    }
}

template <int N_, int GS>
__global__ void __launch_bounds__(kActThreads, 3) sk_tailpre_k(
    int64_t T, int C8, int iters, float inv_nC, const uint4* __restrict__ x, const uint4* __restrict__ du,
    const float* __restrict__ p, const float* __restrict__ b, const float* __restrict__ rstd,
    const float* __restrict__ alpha, const float* __restrict__ H_pre, const float* __restrict__ H_post,
    const float* __restrict__ dH_res, const float* __restrict__ dH_post, const EOut eo, float* __restrict__ kappa,
    float* db, float* dalpha) {
    constexpr int NN = N_ * N_, N = NN + 2 * N_;
    constexpr int o_dhres = N, o_hpre = o_dhres + NN, o_hpost = o_hpre + N_, o_dhpost = o_hpost + N_, o_rstd = o_dhpost + N_,
                  nin = o_rstd + 1;
    __shared__ float in_s[GS][nin];          // p | dH_res | H_pre | H_post | dH_post | rstd of the group's tokens
    __shared__ float dhp_s[GS][kMaxN];
    __shared__ float red[N + 3];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    for (int c = tid; c < N + 3; c += kActThreads) red[c] = 0.f;
    __syncthreads();
    const float a_res = __ldg(alpha), a_pre = __ldg(alpha + 1), a_post = __ldg(alpha + 2);
    const int64_t ngroups = (T + GS - 1) / GS;
    for (int64_t grp = blockIdx.x; grp < ngroups; grp += gridDim.x) {
        const int64_t t0 = grp * GS;
        const int nt = (T - t0 < GS) ? (int)(T - t0) : GS;
        // the per-token inputs of the SK backward travel to shared memory while the warps stream x and du
        for (int i = tid; i < nt * nin; i += kActThreads) {
            const int tl = i / nin, c = i - tl * nin;
            const int64_t t = t0 + tl;
            const float* src;
            if (c < o_dhres) src = p + t * N + c;
            else if (c < o_hpre) src = dH_res + t * NN + (c - o_dhres);
            else if (c < o_hpost) src = H_pre + t * N_ + (c - o_hpre);
            else if (c < o_dhpost) src = H_post + t * N_ + (c - o_hpost);
            else if (c < o_rstd) src = dH_post + t * N_ + (c - o_dhpost);
            else src = rstd + t;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(&in_s[tl][c])), "l"(src) : "memory");
        }
        cp_async_commit();
        // dH_pre[j] = <du, x_j>, one warp per token
        for (int tl = w; tl < nt; tl += kActWarps) {
            const int64_t t = t0 + tl;
            float r[N_];
#pragma unroll
            for (int j = 0; j < N_; ++j) r[j] = 0.f;
            for (int cv0 = lane; cv0 < C8; cv0 += 64) {
                uint4 xv[2][N_], dv[2];
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    const int cv = cv0 + 32 * v;
                    if (cv < C8) {
#pragma unroll
                        for (int j = 0; j < N_; ++j) xv[v][j] = ld_stream(x + (t * N_ + j) * C8 + cv);
                        dv[v] = ld_stream(du + t * C8 + cv);
                    } else {
#pragma unroll
                        for (int j = 0; j < N_; ++j) xv[v][j] = make_uint4(0, 0, 0, 0);
                        dv[v] = make_uint4(0, 0, 0, 0);
                    }
                }
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    float df[8];
                    unpack8(dv[v], df);
#pragma unroll
                    for (int j = 0; j < N_; ++j) {
                        float xf[8];
                        unpack8(xv[v][j], xf);
#pragma unroll
                        for (int e = 0; e < 8; ++e) r[j] = fmaf(df[e], xf[e], r[j]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < N_; ++j) { r[j] = warp_sum(r[j]); if (lane == j) dhp_s[tl][j] = r[j]; }
        }
        cp_async_wait<0>();
        __syncthreads();
        if (tid < nt) {
            const float* in = in_s[tid];
            sk_token_bwd<N_>(t0 + tid, iters, inv_nC, in, b, in[o_rstd], a_res, a_pre, a_post, in + o_hpre, in + o_hpost,
                             in + o_dhres, dhp_s[tid], in + o_dhpost, eo, kappa, red);
        }
        __syncthreads();
    }
    for (int c = tid; c < N + 3; c += kActThreads) {
        if (!dalpha) db[(int64_t)blockIdx.x * kPartStride + c] = red[c];      // per-block partials (tail_finish_k adds them)
        else if (c < N) atomicAdd(db + c, red[c]);
        else atomicAdd(dalpha + (c - N), red[c]);
    }
}

// u_rstd[t] = (mean_c u[t,c]^2 + eps)^-1/2, one warp per token: for the paths whose pre-mix kernel does not produce it.
__global__ void __launch_bounds__(kActThreads) row_rstd_k(int64_t T, int C8, const uint4* __restrict__ u, float eps,
                                                         float* __restrict__ u_rstd) {
    const int lane = threadIdx.x & 31;
    const int64_t nwarps = (int64_t)gridDim.x * kActWarps;
    for (int64_t t = (int64_t)blockIdx.x * kActWarps + (threadIdx.x >> 5); t < T; t += nwarps) {
        float s = 0.f;
        for (int cv = lane; cv < C8; cv += 32) {
            float f[8];
            unpack8(ld_stream(u + t * C8 + cv), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) s = fmaf(f[e], f[e], s);
        }
        s = warp_sum(s);
        if (lane == 0) u_rstd[t] = 1.f / sqrtf(s / (float)(C8 * 8) + eps);
    }
}

// ---- launchers -----------------------------------------------------------------------------------
static int warp_grid(int64_t T, int sm_count) {
    int64_t blocks = (T + kActWarps - 1) / kActWarps;
    const int64_t cap = (int64_t)sm_count * 8;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

// One block per group, at most `resident` of them (the blocks that fit the GPU at once).
static int resident_grid(int64_t T, int group, int resident) {
    const int64_t blocks = (T + group - 1) / group;
    return (int)(blocks < 1 ? 1 : (blocks > resident ? resident : blocks));
}

static int group_grid(int64_t T, int group, int sm_count) {
    int64_t blocks = (T + group - 1) / group;
    const int64_t cap = (int64_t)sm_count * 16;
    if (blocks > cap) blocks = cap;
    return (int)(blocks < 1 ? 1 : blocks);
}

void launch_lite_act_fwd(const mhclite_ctx* c, int64_t T, const ProjPlan& pp, const float* qpart, const float* ssq,
                         float eps, const float* b, const float* alpha, float* H_res, float* H_pre, float* H_post,
                         float* a_saved, float* p_saved, float* rstd, cudaStream_t s) {
    c->launches += 1;
    lite_act_fwd_k<<<warp_grid(T, c->sm_count), kActThreads, 0, s>>>(
        T, c->n, c->nfact, pp.Npad, pp.ksplit, 1.f / (float)(c->n * c->C), eps, qpart, ssq, b, alpha, H_res, H_pre,
        H_post, a_saved, p_saved, rstd, c->table_dev);
}

void launch_lite_act_bwd(const mhclite_ctx* c, int64_t T, int Npad, const float* a, const float* p, const float* rstd,
                         const float* alpha, const float* H_pre, const float* H_post, const float* dH_res,
                         const float* dH_pre, const float* dH_post, float* e, void* ehi, void* elo, int Kp,
                         float* kappa, float* db, float* dalpha, cudaStream_t s) {
    const EOut eo{e, Npad, (__nv_bfloat16*)ehi, (__nv_bfloat16*)elo, Kp};
    clear_e_tail(T, ehi, elo, Kp, s);
    c->launches += 1;
    // fewer, longer-lived blocks: the parameter-gradient partials are reduced once per block
    int64_t blocks = (T + kActWarps * 8 - 1) / (kActWarps * 8);
    if (blocks > c->sm_count * 4) blocks = c->sm_count * 4;
    if (blocks < 1) blocks = 1;
    lite_act_bwd_k<<<(int)blocks, kActThreads, 0, s>>>(T, c->n, c->nfact, 1.f / (float)(c->n * c->C), a, p, rstd,
                                                        alpha, H_pre, H_post, dH_res, dH_pre, dH_post, eo, kappa, db,
                                                        dalpha, c->table_dev);
}

void launch_lite_act_premix(const mhclite_ctx* c, int64_t T, const ProjPlan& pp, const float* qpart, const float* ssq,
                            float eps, const float* b, const float* alpha, float* H_res, float* H_pre, float* H_post,
                            float* a_saved, float* p_saved, float* rstd, const void* x, void* u, cudaStream_t s, float* u_rstd,
                            float eps_u) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_ACT_PREMIX, s);
    const int C8 = c->C / 8;
    const float inv = 1.f / (float)(c->n * c->C);
    // groups of 32 tokens unless that leaves resident block slots (three per SM) empty: then 16 or 8
    const int resident_t = c->sm_count * 3;
    // (but never groups of less than 256 KB of x: below that the phases' barriers cost more than the parallelism gains;
    //  measured at C = 1024 and 1536)
    int gmin = 8;
    while (gmin < kTokGroup && (int64_t)gmin * c->n * c->C * 2 < 256 * 1024) gmin <<= 1;
    int gtok = kTokGroup;
    while (gtok > gmin && (T + gtok - 1) / gtok < (int64_t)resident_t) gtok >>= 1;
    const int grid_t = group_grid(T, gtok, c->sm_count);
#define MHCL_AP_TGS(N_, G_, S_) lite_act_premix_t_k<N_, G_, S_><<<grid_t, kActThreads, 0, s>>>( \
        T, C8, pp.Npad, pp.ksplit, inv, eps, qpart, ssq, b, alpha, H_res, H_pre, H_post, a_saved, p_saved, rstd, \
        (const uint4*)x, (uint4*)u, u_rstd, eps_u)
#define MHCL_AP_TG(N_, G_) do { if (u_rstd) MHCL_AP_TGS(N_, G_, true); else MHCL_AP_TGS(N_, G_, false); } while (0)
#define MHCL_AP_T(N_) do { if (gtok == 8) MHCL_AP_TG(N_, 8); else if (gtok == 16) MHCL_AP_TG(N_, 16); else MHCL_AP_TG(N_, 32); } while (0)
    // one warp per token: n = 5 (120 logits do not fit a thread's registers) and every context that holds a
    // subset of the permutations (its table is data, not a compile-time constant)
#define MHCL_AP_W(N_) lite_act_premix_k<N_><<<resident_grid(T, kGroupTok, c->sm_count * 4), kActThreads, 0, s>>>( \
        T, C8, c->nfact, pp.Npad, pp.ksplit, inv, eps, qpart, ssq, b, alpha, H_res, H_pre, H_post, a_saved, \
        p_saved, rstd, (const uint4*)x, (uint4*)u, c->table_dev)
    const bool warp_kernel = c->table_dev || c->n > 4;
    if (c->table_dev) {
        MHCL_DISPATCH_N(c->n, MHCL_AP_W(N_));
    } else {
        switch (c->n) {
            case 2: MHCL_AP_T(2); break;
            case 3: MHCL_AP_T(3); break;
            case 4: MHCL_AP_T(4); break;
            default: MHCL_AP_W(5);
        }
    }
    if (u_rstd && warp_kernel) {                       // the warp-per-token kernel does not produce the statistic
        c->launches += 1;
        row_rstd_k<<<warp_grid(T, c->sm_count), kActThreads, 0, s>>>(T, C8, (const uint4*)u, eps_u, u_rstd);
    }
#undef MHCL_AP_W
#undef MHCL_AP_T
#undef MHCL_AP_TG
#undef MHCL_AP_TGS
}

void launch_row_rstd(const mhclite_ctx* c, int64_t T, const void* u, float eps, float* u_rstd, cudaStream_t s) {
    c->launches += 1;
    row_rstd_k<<<warp_grid(T, c->sm_count), kActThreads, 0, s>>>(T, c->C / 8, (const uint4*)u, eps, u_rstd);
}

// Returns the number of blocks launched (= partials written when dalpha is null; only the n <= 4 kernel of a context
// without a permutation subset writes partials).
int launch_lite_tailpre(const mhclite_ctx* c, int64_t T, const void* x, const void* du, const float* a, const float* p,
                        const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                        const float* dH_res, const float* dH_post, float* dH_pre_ws, float* e, int Npad, void* ehi,
                        void* elo, int Kp, float* kappa, float* db, float* dalpha, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_TAIL_PRE, s);
    const EOut eo{e, Npad, (__nv_bfloat16*)ehi, (__nv_bfloat16*)elo, Kp};
    clear_e_tail(T, ehi, elo, Kp, s);
    const int C8 = c->C / 8;
    const float inv = 1.f / (float)(c->n * c->C);
    // n <= 4: one warp per token streams for dH_pre and then does the activation backward with a lane per column
    const int blocks = balanced_warp_blocks(T, (int64_t)c->sm_count * 4);      // four blocks per SM fit
    (void)dH_pre_ws;
#define MHCL_TP_T(N_) lite_tailpre_w_k<N_><<<blocks, 256, 0, s>>>( \
        T, C8, inv, (const uint4*)x, (const uint4*)du, a, p, rstd, alpha, H_pre, H_post, dH_res, dH_post, eo, kappa, \
        db, dalpha)
#define MHCL_TP_W(N_) lite_tailpre_k<N_><<<resident_grid(T, 8, c->sm_count * 4), kActThreads, 0, s>>>( \
        T, C8, c->nfact, inv, (const uint4*)x, (const uint4*)du, a, p, rstd, alpha, H_pre, H_post, dH_res, \
        dH_post, eo, kappa, db, dalpha, c->table_dev)
    if (c->table_dev) {
        MHCL_DISPATCH_N(c->n, MHCL_TP_W(N_));
    } else {
        switch (c->n) {
            case 2: MHCL_TP_T(2); break;
            case 3: MHCL_TP_T(3); break;
            case 4: MHCL_TP_T(4); break;
            default: MHCL_TP_W(5);
        }
    }
#undef MHCL_TP_W
#undef MHCL_TP_T
    return blocks;
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
    clear_e_tail(T, ehi, elo, Kp, s);
    c->launches += 1;
    const int grid = (int)((T + 127) / 128);
    const float inv = 1.f / (float)(c->n * c->C);
    MHCL_DISPATCH_N(c->n, sk_act_bwd_k<N_><<<grid, 128, 0, s>>>(T, iters, inv, p, b, rstd, alpha, H_pre, H_post,
                                                                  dH_res, dH_pre, dH_post, eo, kappa, db, dalpha));
}

}  // namespace mhcl

namespace mhcl {

// Tokens per group of the SK path's fused kernels: as for the lite path's thread-per-token kernel, smaller groups when
// the full ones would leave resident block slots (three per SM) empty, but no group of less than 512 KB of x (the 20
// iterations per token make its per-group phase longer: at C = 1024 groups of 32 were slower than groups of 64).
static int sk_group_tokens(const mhclite_ctx* c, int64_t T) {
    int gmin = 16;
    while (gmin < kSkGroup && (int64_t)gmin * c->n * c->C * 2 < 512 * 1024) gmin <<= 1;
    int gs = kSkGroup;
    while (gs > gmin && 2 * ((T + gs - 1) / gs) <= (int64_t)c->sm_count * 3) gs >>= 1;   // halved groups still fit one wave
    return gs;
}

void launch_sk_act_premix(const mhclite_ctx* c, int64_t T, int iters, const ProjPlan& pp, const float* qpart,
                          const float* ssq, float eps, const float* b, const float* alpha, float* H_res, float* H_pre,
                          float* H_post, float* p_saved, float* rstd, const void* x, void* u, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_ACT_PREMIX, s);
    const int C8 = c->C / 8;
    const float inv = 1.f / (float)(c->n * c->C);
    const int gs = sk_group_tokens(c, T);
    const int grid = group_grid(T, gs, c->sm_count);
#define MHCL_SKAP(G_) MHCL_DISPATCH_N(c->n, (sk_act_premix_k<N_, G_><<<grid, kActThreads, 0, s>>>(                       \
        T, C8, iters, pp.Npad, pp.ksplit, inv, eps, qpart, ssq, b, alpha, H_res, H_pre, H_post, p_saved, rstd,           \
        (const uint4*)x, (uint4*)u)))
    if (gs == 16) { MHCL_SKAP(16); } else if (gs == 32) { MHCL_SKAP(32); } else { MHCL_SKAP(64); }
#undef MHCL_SKAP
}

int launch_sk_tailpre(const mhclite_ctx* c, int64_t T, int iters, const void* x, const void* du, const float* p,
                      const float* b, const float* rstd, const float* alpha, const float* H_pre, const float* H_post,
                      const float* dH_res, const float* dH_post, float* e, int Npad, void* ehi, void* elo, int Kp,
                      float* kappa, float* db, float* dalpha, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_TAIL_PRE, s);
    const EOut eo{e, Npad, (__nv_bfloat16*)ehi, (__nv_bfloat16*)elo, Kp};
    clear_e_tail(T, ehi, elo, Kp, s);
    const int C8 = c->C / 8;
    const float inv = 1.f / (float)(c->n * c->C);
    const int gs = sk_group_tokens(c, T);
    const int grid = group_grid(T, gs, c->sm_count);
#define MHCL_SKTP(G_) MHCL_DISPATCH_N(c->n, (sk_tailpre_k<N_, G_><<<grid, kActThreads, 0, s>>>(                         \
        T, C8, iters, inv, (const uint4*)x, (const uint4*)du, p, b, rstd, alpha, H_pre, H_post, dH_res, dH_post, eo,     \
        kappa, db, dalpha)))
    if (gs == 16) { MHCL_SKTP(16); } else if (gs == 32) { MHCL_SKTP(32); } else { MHCL_SKTP(64); }
#undef MHCL_SKTP
    return grid;
}

}  // namespace mhcl
