// Tensor-core backward of the projection of paper Eq. (4) (and of RMSNorm), fused with the rest of dx.
//
// Per token t, with e = rstd * alpha (.) dz (from the activation backward), W' = diag(gain) W and
// kappa_t = rstd^2 * sum_c (alpha dz)_c p_c / (nC):
//   (1) dxhat[t,m] = sum_c e[t,c] W'[m,c] - x[t,m] kappa_t          (projection + RMSNorm backward)
//   (2) G[m,c]    += x[t,m] e[t,c]                                    (dW = gain (.) G, dgain = sum_c W G)
//   FUSED:  dx[t,j,c] = sum_i H_res[t,i,j] g[t,i,c] + H_pre[t,j] du[t,c] + dxhat[t,j*C+c]   (written once)
//   else :  dx (+)= dxhat
//
// One CTA owns a slice of 64 channels (of every stream) and walks over a range of tokens in tiles of 32,
// so that the W' slice and the G accumulators stay on chip: x, g, du and e stream through shared memory
// (cp.async, double buffered, two CTAs per SM).  Both contractions run on mma.sync.m16n8k16 (bf16, fp32 accumulate):
//   (1) M = tokens, N = channels, K = projection columns; e and W' rounded to bf16 (this term is a small
//       part of a bf16 output); the columns of each n-tile are permuted so that a thread ends up with 8
//       consecutive channels of a token and stores 16 bytes.
//   (2) M = channels, N = projection columns, K = tokens; x is exact in bf16, e enters as a bf16 pair
//       hi + lo so that the fp32 parameter gradients keep ~1e-6 relative accuracy.
// The G partials of the token ranges are written to separate buffers and added by a finishing kernel
// (no atomics: bitwise reproducible).
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"

namespace mhcl {

constexpr int kTT = 32;            // tokens per tile
constexpr int kCS = 64;            // channels per slice (128 bytes of bf16 per row)
constexpr int kTailStages = 2;    // two CTAs per SM, each double-buffered

// Row swizzle of the 128-byte tiles: 8 consecutive rows get 8 different 16-byte slots (ldmatrix), and
// consecutive rows differ in bit 2 (a quarter warp reading 4 pieces of 2 consecutive rows is conflict free).
__device__ __forceinline__ int swz(int row) { return ((row & 1) << 2) | ((row >> 1) & 3); }

__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

struct TailArgs {
    int64_t T, tok_per_split;
    int C, N, Kp;                                  // channels per stream, projection columns, padded to 16
    const __nv_bfloat16 *x, *g, *du;               // g, du only when FUSED
    const __nv_bfloat16 *ehi, *elo;                // Kp columns per token, tiled (e_tiled_index)
    const float *kappa, *H_res, *H_pre;            // H_* only when FUSED
    const float *W, *gain;
    __nv_bfloat16* dx;
    float* Gpart;                                  // [splits][n*C][Kp]
};

template <int N_, int KS, bool FUSED>
struct TailCfg {
    static constexpr int kRows = N_ * kTT;                         // rows of the x / g tiles
    static constexpr int kX = kRows * 128;
    static constexpr int kDu = kTT * 128;
    static constexpr int kEStride = KS * 32 + 16;                  // bytes per row of an e tile (padded)
    static constexpr int kE = kTT * kEStride;
    static constexpr int kHresStride = N_ * N_ + 1;               // odd stride: rows of different tokens in different banks
    static constexpr int kCoefFloats = kTT * (1 + (FUSED ? kHresStride + N_ : 0));
    static constexpr int oG = kX, oDu = oG + (FUSED ? kX : 0), oEh = oDu + (FUSED ? kDu : 0), oEl = oEh + kE,
                         oCoef = oEl + kE;
    static constexpr int kStage = (oCoef + kCoefFloats * 4 + 127) / 128 * 128;
    static constexpr int kGroups = N_ * 2;                         // 32-channel groups of the slice
    static constexpr int kBfrag = kGroups * 4 * KS * 32 * 8;       // W' slice in B-fragment order (uint2 per lane)
    static constexpr int kSmem = kBfrag + kTailStages * kStage;
    static constexpr int kMT2 = (N_ * 4 + 7) / 8;                  // 16-channel m-tiles per warp in (2)
    static constexpr int kGP = (kGroups + 7) / 8;                  // 32-channel groups per warp in (1)
};

template <int N_, int KS, bool FUSED, bool ACC>
__global__ void __launch_bounds__(256, 2) tail_mma_k(const TailArgs a) {
    using Cfg = TailCfg<N_, KS, FUSED>;
    constexpr int NT8 = 2 * KS;                                    // 8-column tiles of the projection
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g8 = lane >> 2, q = lane & 3;
    const int c0 = blockIdx.x * kCS;
    const int64_t t_begin = (int64_t)blockIdx.y * a.tok_per_split;
    const int64_t t_end = (t_begin + a.tok_per_split < a.T) ? t_begin + a.tok_per_split : a.T;
    const int ntiles = (t_end > t_begin) ? (int)((t_end - t_begin + kTT - 1) / kTT) : 0;
    const int C = a.C, nC = N_ * a.C;
    unsigned char* stage0 = smem + Cfg::kBfrag;

    // ---- W' slice, bf16, in B-fragment order of (1), with the channel permutation ------------------
    // entry [((gid*4 + jn)*KS + kc)*32 + lane] = { W'[m][16kc+2q..+1], W'[m][16kc+8+2q..+1] },
    // m = stream j = gid/2, channel c0 + (gid%2)*32 + (g8>>1)*8 + jn*2 + (g8&1)
    {
        uint2* bf = reinterpret_cast<uint2*>(smem);
        for (int i = tid; i < Cfg::kGroups * 4 * KS * 32; i += 256) {
            const int l = i & 31, kc = (i >> 5) % KS, jn = ((i >> 5) / KS) & 3, gid = (i >> 5) / (KS * 4);
            const int gg = l >> 2, qq = l & 3;
            const int ch = c0 + (gid & 1) * 32 + (gg >> 1) * 8 + jn * 2 + (gg & 1);
            const int m = (gid >> 1) * C + ch;
            float w[4] = {0.f, 0.f, 0.f, 0.f};
            if (ch < C) {
                const float gm = __ldg(a.gain + m);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = kc * 16 + 2 * qq + (e & 1) + (e >> 1) * 8;
                    if (col < a.N) w[e] = __ldg(a.W + (int64_t)m * a.N + col) * gm;
                }
            }
            bf[i] = make_uint2(pack2(w[0], w[1]), pack2(w[2], w[3]));
        }
    }

    auto load = [&](int stage, int tile) {
        const uint32_t sb = smem_u32(stage0 + stage * Cfg::kStage);
        const int64_t tt0 = t_begin + (int64_t)tile * kTT;
        // x (and g) tiles: row = j*kTT + tl, 8 pieces of 16 bytes
        for (int i = tid; i < Cfg::kRows * 8; i += 256) {
            const int row = i >> 3, pc = i & 7;
            const int j = row / kTT, tl = row - j * kTT;
            const int64_t t = tt0 + tl;
            const int c = c0 + pc * 8;
            const bool ok = (t < t_end) && (c < C);
            const int64_t off = (t * N_ + j) * C + c;
            const uint32_t d = row * 128 + ((pc ^ swz(row)) << 4);
            cp_async16(sb + d, ok ? a.x + off : a.x, ok ? 16 : 0);
            if (FUSED) cp_async16(sb + Cfg::oG + d, ok ? a.g + off : a.x, ok ? 16 : 0);
        }
        if (FUSED) {
            for (int i = tid; i < kTT * 8; i += 256) {
                const int tl = i >> 3, pc = i & 7;
                const int64_t t = tt0 + tl;
                const int c = c0 + pc * 8;
                const bool ok = (t < t_end) && (c < C);
                cp_async16(sb + Cfg::oDu + tl * 128 + ((pc ^ swz(tl)) << 4), ok ? a.du + t * C + c : a.x, ok ? 16 : 0);
            }
        }
        for (int i = tid; i < kTT * KS * 2; i += 256) {            // e tiles: KS*2 pieces per row
            const int tl = i / (KS * 2), pc = i - tl * (KS * 2);
            const int64_t t = tt0 + tl;
            const bool ok = t < t_end;
            const int64_t off = ok ? e_tiled_index(a.Kp, t, pc * 8) : 0;
            cp_async16(sb + Cfg::oEh + tl * Cfg::kEStride + pc * 16, ok ? a.ehi + off : a.x, ok ? 16 : 0);
            cp_async16(sb + Cfg::oEl + tl * Cfg::kEStride + pc * 16, ok ? a.elo + off : a.x, ok ? 16 : 0);
        }
        for (int i = tid; i < Cfg::kCoefFloats; i += 256) {        // kappa | H_pre | H_res of the tile's tokens
            const float* src;
            int64_t idx;
            if (i < kTT) { src = a.kappa; idx = tt0 + i; if (idx >= t_end) idx = -1; }
            else if (i < kTT + kTT * N_) { src = a.H_pre; idx = tt0 * N_ + (i - kTT); if (idx >= t_end * N_) idx = -1; }
            else {
                const int r = i - kTT - kTT * N_, tl = r / Cfg::kHresStride, e = r - tl * Cfg::kHresStride;
                src = a.H_res; idx = (tt0 + tl) * N_ * N_ + e;
                if (e >= N_ * N_ || tt0 + tl >= t_end) idx = -1;
            }
            cp_async4(sb + Cfg::oCoef + i * 4, idx >= 0 ? (const void*)(src + idx) : (const void*)a.x, idx >= 0 ? 4 : 0);
        }
    };

    float G[Cfg::kMT2][NT8][4];
#pragma unroll
    for (int mi = 0; mi < Cfg::kMT2; ++mi)
#pragma unroll
        for (int j = 0; j < NT8; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) G[mi][j][e] = 0.f;

#pragma unroll
    for (int s = 0; s < kTailStages - 1; ++s) {
        if (s < ntiles) load(s, s);
        cp_async_commit();
    }
    const uint2* bfrag = reinterpret_cast<const uint2*>(smem);
    for (int it = 0; it < ntiles; ++it) {
        cp_async_wait<kTailStages - 2>();
        __syncthreads();
        {
            const int nxt = it + kTailStages - 1;
            if (nxt < ntiles) load(nxt % kTailStages, nxt);
            cp_async_commit();
        }
        const unsigned char* st = stage0 + (it % kTailStages) * Cfg::kStage;
        const uint32_t sb = smem_u32(st);
        const float* coef = reinterpret_cast<const float*>(st + Cfg::oCoef);
        const int64_t tt0 = t_begin + (int64_t)it * kTT;

        // ---- (1) dxhat and the fused dx ---------------------------------------------------------------
#pragma unroll
        for (int gi = 0; gi < Cfg::kGP; ++gi) {
            const int gid = warp + 8 * gi;
            if (gid >= Cfg::kGroups) break;
            const int j = gid >> 1, h = gid & 1;
            uint2 bw[4][KS];
#pragma unroll
            for (int jn = 0; jn < 4; ++jn)
#pragma unroll
                for (int kc = 0; kc < KS; ++kc) bw[jn][kc] = bfrag[((gid * 4 + jn) * KS + kc) * 32 + lane];
#pragma unroll
            for (int mt = 0; mt < kTT / 16; ++mt) {
                float acc[4][4];
#pragma unroll
                for (int jn = 0; jn < 4; ++jn)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[jn][e] = 0.f;
#pragma unroll
                for (int kc = 0; kc < KS; ++kc) {
                    uint32_t af[4];
                    const int row = mt * 16 + (lane & 15);
                    ldmatrix_x4(af, sb + Cfg::oEh + row * Cfg::kEStride + (2 * kc + (lane >> 4)) * 16);
#pragma unroll
                    for (int jn = 0; jn < 4; ++jn) mma_bf16(acc[jn], af, bw[jn][kc].x, bw[jn][kc].y);
                }
                const int pc = h * 4 + q;                          // this thread's 8 channels: c0 + 8 pc ..
                const int ch = c0 + pc * 8;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int tl = mt * 16 + g8 + half * 8;
                    const int64_t t = tt0 + tl;
                    if (t >= t_end || ch >= C) continue;
                    float o[8];
#pragma unroll
                    for (int jn = 0; jn < 4; ++jn) { o[2 * jn] = acc[jn][2 * half]; o[2 * jn + 1] = acc[jn][2 * half + 1]; }
                    float xf[8];
                    const int xrow = j * kTT + tl;
                    unpack8(*reinterpret_cast<const uint4*>(st + xrow * 128 + ((pc ^ swz(xrow)) << 4)), xf);
                    const float kp = coef[tl];
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[e] = fmaf(-xf[e], kp, o[e]);
                    if (FUSED) {
                        float df[8];
                        unpack8(*reinterpret_cast<const uint4*>(st + Cfg::oDu + tl * 128 + ((pc ^ swz(tl)) << 4)), df);
                        const float hp = coef[kTT + tl * N_ + j];
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] = fmaf(hp, df[e], o[e]);
#pragma unroll
                        for (int i = 0; i < N_; ++i) {
                            float gf[8];
                            const int grow = i * kTT + tl;
                            unpack8(*reinterpret_cast<const uint4*>(st + Cfg::oG + grow * 128 + ((pc ^ swz(grow)) << 4)), gf);
                            const float hr = coef[kTT + kTT * N_ + tl * Cfg::kHresStride + i * N_ + j];
#pragma unroll
                            for (int e = 0; e < 8; ++e) o[e] = fmaf(hr, gf[e], o[e]);
                        }
                    }
                    __nv_bfloat16* dst = a.dx + (t * N_ + j) * C + ch;
                    if (ACC) {
                        float old[8];
                        unpack8(*reinterpret_cast<const uint4*>(dst), old);
#pragma unroll
                        for (int e = 0; e < 8; ++e) o[e] += old[e];
                    }
                    st_stream(dst, pack8(o));
                }
            }
        }

        // ---- (2) G += x^T e -----------------------------------------------------------------------------
        // The e fragments are the same for every m-tile: they are fetched once per (k-step, column pair);
        // hi and lo products of one accumulator are kept apart in the issue order.
#pragma unroll
        for (int kt = 0; kt < kTT / 16; ++kt) {
            uint32_t af[Cfg::kMT2][4];
#pragma unroll
            for (int mi = 0; mi < Cfg::kMT2; ++mi) {
                const int mtile = warp + 8 * mi;                   // (stream j, 16-channel block cb)
                if (mtile < N_ * 4) {
                    // matrices: (t 0-7, piece 2cb), (t 0-7, piece 2cb+1), (t 8-15, piece 2cb), (t 8-15, piece 2cb+1)
                    const int j = mtile >> 2, cb = mtile & 3;
                    const int row = j * kTT + kt * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
                    const int pc = 2 * cb + ((lane >> 3) & 1);
                    ldmatrix_x4_trans(af[mi], sb + row * 128 + ((pc ^ swz(row)) << 4));
                }
            }
#pragma unroll
            for (int jp = 0; jp < KS; ++jp) {                      // pairs of 8-column tiles
                uint32_t bh[4], bl[4];
                // matrices: (t 0-7, cols 16jp..+7), (t 8-15, same), (t 0-7, cols 16jp+8..), (t 8-15, same)
                const int row = kt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const uint32_t off = row * Cfg::kEStride + (2 * jp + (lane >> 4)) * 16;
                ldmatrix_x4_trans(bh, sb + Cfg::oEh + off);
                ldmatrix_x4_trans(bl, sb + Cfg::oEl + off);
#pragma unroll
                for (int mi = 0; mi < Cfg::kMT2; ++mi) {
                    if (warp + 8 * mi < N_ * 4) {
                        mma_bf16(G[mi][2 * jp], af[mi], bh[0], bh[1]);
                        mma_bf16(G[mi][2 * jp + 1], af[mi], bh[2], bh[3]);
                    }
                }
#pragma unroll
                for (int mi = 0; mi < Cfg::kMT2; ++mi) {
                    if (warp + 8 * mi < N_ * 4) {
                        mma_bf16(G[mi][2 * jp], af[mi], bl[0], bl[1]);
                        mma_bf16(G[mi][2 * jp + 1], af[mi], bl[2], bl[3]);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();

    // ---- G partial of this token range ---------------------------------------------------------------
    float* Gp = a.Gpart + (int64_t)blockIdx.y * nC * a.Kp;
#pragma unroll
    for (int mi = 0; mi < Cfg::kMT2; ++mi) {
        const int mtile = warp + 8 * mi;
        if (mtile >= N_ * 4) break;
        const int j = mtile >> 2, cb = mtile & 3;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int ch = c0 + cb * 16 + g8 + half * 8;
            if (ch >= C) continue;
            float* row = Gp + (int64_t)(j * C + ch) * a.Kp;
#pragma unroll
            for (int jt = 0; jt < NT8; ++jt)
                *reinterpret_cast<float2*>(row + jt * 8 + 2 * q) = make_float2(G[mi][jt][2 * half], G[mi][jt][2 * half + 1]);
        }
    }
}

// dW (+)= gain (.) sum_s Gpart[s] ; dgain[m] (+)= sum_c W[m,c] sum_s Gpart[s][m,c].  One warp per row m.
template <bool ACC>
__global__ void __launch_bounds__(256) tail_finish_k(int nC, int N, int Kp, int splits, const float* __restrict__ W,
                                                     const float* __restrict__ gain, const float* __restrict__ Gpart,
                                                     float* dW, float* dgain, const float* __restrict__ dpart, int nparts,
                                                     float* db, float* dalpha) {
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
    // the first warps also add up the per-block partials of db and dalpha, one column each, in a fixed order
    if (dpart && m < N + 3) {
        float v = 0.f;
        for (int p0 = lane; p0 < nparts; p0 += 32) v += __ldg(dpart + (int64_t)p0 * kPartStride + m);
        v = warp_sum(v);
        if (lane == 0) {
            float* dst = m < N ? db + m : dalpha + (m - N);
            *dst = ACC ? *dst + v : v;
        }
    }
    if (m >= nC) return;
    const float gm = __ldg(gain + m);
    float dg = 0.f;
    for (int c = lane; c < N; c += 32) {
        float gv = 0.f;
        for (int s0 = 0; s0 < splits; s0 += 8) {                  // eight loads in flight, then a fixed-order sum
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                v[k] = (s0 + k < splits) ? __ldg(Gpart + ((int64_t)(s0 + k) * nC + m) * Kp + c) : 0.f;
#pragma unroll
            for (int k = 0; k < 8; k += 4) gv += (v[k] + v[k + 1]) + (v[k + 2] + v[k + 3]);
        }
        const int64_t i = (int64_t)m * N + c;
        dW[i] = ACC ? dW[i] + gm * gv : gm * gv;
        dg = fmaf(__ldg(W + i), gv, dg);
    }
    dg = warp_sum(dg);
    if (lane == 0) dgain[m] = ACC ? dgain[m] + dg : dg;
}

template <bool ACC>
__global__ void __launch_bounds__(256) dpart_sum_k(int N, const float* __restrict__ dpart, int nparts, float* db, float* dalpha) {
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (m >= N + 3) return;
    float v = 0.f;
    for (int p0 = lane; p0 < nparts; p0 += 32) v += __ldg(dpart + (int64_t)p0 * kPartStride + m);
    v = warp_sum(v);
    if (lane == 0) {
        float* dst = m < N ? db + m : dalpha + (m - N);
        *dst = ACC ? *dst + v : v;
    }
}

// ---- host side -------------------------------------------------------------------------------------
void launch_dpart_sum(const mhclite_ctx* c, int N, const float* dpart, int nparts, float* db, float* dalpha, int acc_params,
                      cudaStream_t s) {
    c->launches += 1;
    const int grid = (N + 3 + 7) / 8;
    if (acc_params) dpart_sum_k<true><<<grid, 256, 0, s>>>(N, dpart, nparts, db, dalpha);
    else dpart_sum_k<false><<<grid, 256, 0, s>>>(N, dpart, nparts, db, dalpha);
}

TailPlan plan_tail(int n, int C, int64_t T, int N, int sm_count) {
    TailPlan p;
    p.Kp = round_up(N, 16);
    p.KS = p.Kp / 16;
    // n = 5 always takes the tcgen05 pair of tail_tc.cu, also with a narrow projection (a subset of the permutations):
    // the fused tcgen05 kernel stops at n = 4, and the pair is about twice as fast as this file's mma.sync kernel
    p.supported = p.KS <= 3 && n <= 4;
    p.slices = (C + kCS - 1) / kCS;
    if (sm_count > 148) sm_count = 148;                       // the workspace is sized for at most 2 x 148 CTAs
    int64_t splits = (2 * sm_count) / p.slices;
    const int64_t max_splits = (T + kTT - 1) / kTT;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    p.tok_per_split = round_up64((T + splits - 1) / splits, kTT);
    if (p.tok_per_split < kTT) p.tok_per_split = kTT;
    p.splits = (int)((T + p.tok_per_split - 1) / p.tok_per_split);
    if (p.splits < 1) p.splits = 1;
    // tcgen05 kernels for the wide case
    p.tc = !p.supported && p.Kp <= 256 && ((n * C) % 8) == 0;
    p.g_mt = 512 / p.Kp; if (p.g_mt > 3) p.g_mt = 3;
    const int nC = n * C;
    if ((nC + 127) / 128 < p.g_mt) p.g_mt = (nC + 127) / 128;
    p.g_groups = (nC + 128 * p.g_mt - 1) / (128 * p.g_mt);
    int64_t gs = sm_count / p.g_groups;
    const int64_t max_gs = (T + kEGranule - 1) / kEGranule;
    if (gs > max_gs) gs = max_gs;
    if (gs < 1) gs = 1;
    p.g_tok_per_split = round_up64((T + gs - 1) / gs, kEGranule);
    if (p.g_tok_per_split < kEGranule) p.g_tok_per_split = kEGranule;
    p.g_splits = (int)((T + p.g_tok_per_split - 1) / p.g_tok_per_split);
    if (p.g_splits < 1) p.g_splits = 1;
    plan_tail_ftc(n, C, T, sm_count, &p);
    return p;
}

template <int N_, int KS>
static void launch_tail_t(const TailPlan& p, const TailArgs& a, bool fused, bool acc, cudaStream_t s) {
    dim3 grid(p.slices, p.splits);
#define MHCL_TAIL(F, A)                                                                                       \
    do {                                                                                                      \
        using Cfg = TailCfg<N_, KS, F>;                                                                       \
        cudaFuncSetAttribute(tail_mma_k<N_, KS, F, A>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem); \
        tail_mma_k<N_, KS, F, A><<<grid, 256, Cfg::kSmem, s>>>(a);                                            \
    } while (0)
    if (fused) MHCL_TAIL(true, false);
    else if (acc) MHCL_TAIL(false, true);
    else MHCL_TAIL(false, false);
#undef MHCL_TAIL
}

void launch_tail_mma(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                     const void* du, const void* ehi, const void* elo, const float* kappa, const float* H_res,
                     const float* H_pre, const float* W, const float* gain, void* dx, int acc_dx, float* Gpart,
                     float* dW, float* dgain, int acc_params, cudaStream_t s) {
    c->launches += 2;
    TailArgs a;
    a.T = T; a.tok_per_split = p.tok_per_split; a.C = c->C; a.N = N; a.Kp = p.Kp;
    a.x = (const __nv_bfloat16*)x; a.g = (const __nv_bfloat16*)g; a.du = (const __nv_bfloat16*)du;
    a.ehi = (const __nv_bfloat16*)ehi; a.elo = (const __nv_bfloat16*)elo;
    a.kappa = kappa; a.H_res = H_res; a.H_pre = H_pre; a.W = W; a.gain = gain;
    a.dx = (__nv_bfloat16*)dx; a.Gpart = Gpart;
    const bool fused = g != nullptr;
#define MHCL_TAIL_KS(N_)                                                          \
    switch (p.KS) {                                                               \
        case 1: launch_tail_t<N_, 1>(p, a, fused, acc_dx != 0, s); break;         \
        case 2: launch_tail_t<N_, 2>(p, a, fused, acc_dx != 0, s); break;         \
        default: launch_tail_t<N_, 3>(p, a, fused, acc_dx != 0, s); break;        \
    }
    {
        KernelTimer timer_(c, MHCLITE_KERNEL_TAIL_DX, s);
        MHCL_DISPATCH_N(c->n, MHCL_TAIL_KS(N_));
    }
#undef MHCL_TAIL_KS
    launch_tail_finish(c, N, p.Kp, p.splits, W, gain, Gpart, dW, dgain, acc_params, s);
}

// Counted by the caller.
void launch_tail_finish(const mhclite_ctx* c, int N, int Kp, int splits, const float* W, const float* gain,
                        const float* Gpart, float* dW, float* dgain, int acc_params, cudaStream_t s, const float* dpart,
                        int nparts, float* db, float* dalpha) {
    const int nC = c->n * c->C;
    int fg = (nC + 7) / 8;
    if (dpart && fg < (N + 3 + 7) / 8) fg = (N + 3 + 7) / 8;
    if (acc_params) tail_finish_k<true><<<fg, 256, 0, s>>>(nC, N, Kp, splits, W, gain, Gpart, dW, dgain, dpart, nparts, db, dalpha);
    else tail_finish_k<false><<<fg, 256, 0, s>>>(nC, N, Kp, splits, W, gain, Gpart, dW, dgain, dpart, nparts, db, dalpha);
}

}  // namespace mhcl
