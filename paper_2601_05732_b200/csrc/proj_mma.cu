// Tensor-core version of the skinny projection of paper Eq. (4): q[t,c] = sum_m x[t,m] W'[m,c] with
// W' = diag(gain) W, plus the sum of squares RMSNorm needs, in one pass over x.
//
// The activations are bf16 (exact MMA operands); W' is fp32 and is split into a bf16 pair hi + lo
// (two MMAs per tile, ~2^-17 relative operand error) so that the fp32 mappings keep ~1e-6 accuracy.
// The contraction runs on mma.sync.m16n8k16 (bf16 in, fp32 accumulate): the kernel is HBM-bound, the
// tensor work (2 * 2 nC N flop per token) only has to keep pace with the x stream.
//
// Tiling: one CTA = 128 tokens x one slice of the K = nC axis; x streams through shared memory in
// 64-wide K chunks (cp.async, 3-4 stages, XOR-swizzled rows so that ldmatrix is conflict free); W' is
// pre-packed once per call in MMA-fragment order so that each lane fetches its B fragments (hi and lo)
// with one 16-byte shared load.  Partial results of the K slices go to separate buffers that the
// activation kernel adds up: no atomics, bitwise reproducible.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"

namespace mhcl {

constexpr int kTileTok = 128;      // tokens per CTA
constexpr int kChunkK = 64;        // K elements per pipeline stage (4 MMA k-steps)
constexpr int kXStageBytes = kTileTok * kChunkK * 2;

// ------------------------------------------------------------------------------------------------
// Pack W' = diag(gain) W into B-fragment order, split in bf16 hi / lo.
//   Wp[((ks * NT + j) * 32 + lane)] = { b0_hi, b1_hi, b0_lo, b1_lo }   for k-step ks (16 rows of W'),
//   column tile j (8 columns), where b0 = W'[16 ks + 2q + {0,1}][8 j + g], b1 = same rows + 8.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_w_k(int nC, int N, int NT, int ksteps, const float* __restrict__ W,
                                                const float* __restrict__ gain, uint4* __restrict__ Wp) {
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx >= ksteps * NT * 32) return;
    const int lane = idx & 31, j = (idx >> 5) % NT, ks = (idx >> 5) / NT;
    const int g = lane >> 2, q = lane & 3;
    const int col = j * 8 + g;
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int k = ks * 16 + 2 * q + (e & 1) + (e >> 1) * 8;
        const float w = (k < nC && col < N) ? __ldg(W + (int64_t)k * N + col) * __ldg(gain + k) : 0.f;
        split_bf16(w, hi[e], lo[e]);
    }
    Wp[idx] = make_uint4(pack_bf16(hi[0], hi[1]), pack_bf16(hi[2], hi[3]), pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
}

// ------------------------------------------------------------------------------------------------
// Forward contraction.  8 warps = 2 (token halves of 64) x WN (column groups) x WK (k-steps of a chunk),
// WN * WK = 4.  Each warp owns 4 m-tiles x NTW n-tiles of fp32 accumulators.
// ------------------------------------------------------------------------------------------------
template <int NT, int WN>
struct FwdCfg {
    static constexpr int WK = 4 / WN;
    static constexpr int NTW = NT / WN;
    static constexpr int kWStage = 4 * NT * 512;                       // 4 k-steps x NT tiles x 32 lanes x 16 B
    static constexpr int kStage = kXStageBytes + kWStage;
    static constexpr int kStages = (NT <= 5) ? 4 : 3;
    static constexpr int kRow = NT * 8 + 4;                            // padded row of the epilogue staging (floats)
    static constexpr int kEpi = (WK * kTileTok * kRow + WK * kTileTok) * 4;
    static constexpr int kSmem = (kStages * kStage > kEpi) ? kStages * kStage : kEpi;
};

template <int NT, int WN>
__global__ void __launch_bounds__(256, (NT <= 5 ? 2 : 1))
proj_fwd_mma_k(int64_t T, int nC, int nchunks, int chunks_per_split, const __nv_bfloat16* __restrict__ x,
               const uint4* __restrict__ Wp, float* __restrict__ qpart, float* __restrict__ ssq) {
    using Cfg = FwdCfg<NT, WN>;
    constexpr int WK = Cfg::WK, NTW = Cfg::NTW, STAGES = Cfg::kStages;
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp & 1, wn = (warp >> 1) % WN, wk = (warp >> 1) / WN;
    const int64_t t0 = (int64_t)blockIdx.x * kTileTok;
    const int split = blockIdx.y;
    const int c_begin = split * chunks_per_split;
    const int c_end = (c_begin + chunks_per_split < nchunks) ? c_begin + chunks_per_split : nchunks;
    const int nloc = c_end - c_begin;

    float acc[4][NTW][4];
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int j = 0; j < NTW; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][j][e] = 0.f;
    float sq[4][2] = {{0, 0}, {0, 0}, {0, 0}, {0, 0}};

    auto load = [&](int stage, int chunk) {
        unsigned char* xs = smem + stage * Cfg::kStage;
        const uint32_t xs_u = smem_u32(xs);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int pidx = tid + 256 * i;
            const int row = pidx >> 3, pc = pidx & 7;
            const int k = chunk * kChunkK + pc * 8;
            const bool ok = (t0 + row < T) && (k < nC);
            const __nv_bfloat16* src = ok ? x + (t0 + row) * nC + k : x;
            cp_async16(xs_u + row * 128 + ((pc ^ (row & 7)) << 4), src, ok ? 16 : 0);
        }
        const uint4* wsrc = Wp + (int64_t)chunk * (Cfg::kWStage / 16);
        const uint32_t ws_u = xs_u + kXStageBytes;
        for (int i = tid; i < Cfg::kWStage / 16; i += 256) cp_async16(ws_u + i * 16, wsrc + i, 16);
    };

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < nloc) load(s, c_begin + s);
        cp_async_commit();
    }
    for (int i = 0; i < nloc; ++i) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {
            const int nxt = i + STAGES - 1;
            if (nxt < nloc) load(nxt % STAGES, c_begin + nxt);
            cp_async_commit();
        }
        const unsigned char* st = smem + (i % STAGES) * Cfg::kStage;
        const uint32_t xs_u = smem_u32(st);
        const uint4* ws = reinterpret_cast<const uint4*>(st + kXStageBytes);
#pragma unroll
        for (int ksi = 0; ksi < 4 / WK; ++ksi) {
            const int ks = wk + ksi * WK;
            uint32_t a[4][4];
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const int row = wm * 64 + mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int piece = 2 * ks + (lane >> 4);
                ldmatrix_x4(a[mt], xs_u + row * 128 + ((piece ^ (row & 7)) << 4));
            }
            if (wn == 0) {
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const float lo = bf16lo(a[mt][r]), hi = bf16hi(a[mt][r]);
                        sq[mt][r & 1] = fmaf(lo, lo, fmaf(hi, hi, sq[mt][r & 1]));
                    }
                }
            }
            // the hi and lo products of one accumulator are issued far apart: back-to-back MMAs on the same
            // accumulator would wait for each other
            uint4 bw[NTW];
#pragma unroll
            for (int j = 0; j < NTW; ++j) bw[j] = ws[(ks * NT + wn * NTW + j) * 32 + lane];
#pragma unroll
            for (int j = 0; j < NTW; ++j)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) mma_bf16(acc[mt][j], a[mt], bw[j].x, bw[j].y);
#pragma unroll
            for (int j = 0; j < NTW; ++j)
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) mma_bf16(acc[mt][j], a[mt], bw[j].z, bw[j].w);
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    // epilogue: add the WK partial tiles in shared memory, then coalesced stores of this K slice's result
    float* part = reinterpret_cast<float*>(smem);
    float* ssq_s = part + WK * kTileTok * Cfg::kRow;
    const int g = lane >> 2, q = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) {
        const int row = wm * 64 + mt * 16 + g;
#pragma unroll
        for (int j = 0; j < NTW; ++j) {
            const int col = (wn * NTW + j) * 8 + 2 * q;
            float* d0 = part + (wk * kTileTok + row) * Cfg::kRow + col;
            *reinterpret_cast<float2*>(d0) = make_float2(acc[mt][j][0], acc[mt][j][1]);
            *reinterpret_cast<float2*>(d0 + 8 * Cfg::kRow) = make_float2(acc[mt][j][2], acc[mt][j][3]);
        }
        if (wn == 0) {
            float s0 = sq[mt][0], s1 = sq[mt][1];
            s0 += __shfl_xor_sync(0xffffffffu, s0, 1); s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
            s1 += __shfl_xor_sync(0xffffffffu, s1, 1); s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
            if (q == 0) { ssq_s[wk * kTileTok + row] = s0; ssq_s[wk * kTileTok + row + 8] = s1; }
        }
    }
    __syncthreads();
    constexpr int NP = NT * 8, NP4 = NP / 4;
    for (int i = tid; i < kTileTok * NP4; i += 256) {
        const int row = i / NP4, c4 = i - row * NP4;
        if (t0 + row >= T) continue;
        float4 v = *reinterpret_cast<const float4*>(part + row * Cfg::kRow + c4 * 4);
#pragma unroll
        for (int w = 1; w < WK; ++w) {
            const float4 o = *reinterpret_cast<const float4*>(part + (w * kTileTok + row) * Cfg::kRow + c4 * 4);
            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
        }
        *reinterpret_cast<float4*>(qpart + ((int64_t)split * T + t0 + row) * NP + c4 * 4) = v;
    }
    if (tid < kTileTok && t0 + tid < T) {
        float s = ssq_s[tid];
#pragma unroll
        for (int w = 1; w < WK; ++w) s += ssq_s[w * kTileTok + tid];
        ssq[(int64_t)split * T + t0 + tid] = s;
    }
}

// ---- host side -------------------------------------------------------------------------------------
ProjPlan plan_proj(int n, int C, int64_t T, int N, int sm_count) {
    ProjPlan p;
    const int nt = (N + 7) / 8;
    p.NT = nt <= 5 ? nt : 20;                                // 6..20 column tiles run as 4 groups of 5
    p.Npad = p.NT * 8;
    p.nchunks = (n * C + kChunkK - 1) / kChunkK;
    p.ksteps = p.nchunks * 4;
    const int64_t tiles = (T + kTileTok - 1) / kTileTok;
    int ks = tiles > 0 ? (int)((2 * (int64_t)sm_count) / tiles) : 1;      // fill 2 CTAs per SM, one wave
    if (ks > kMaxKSplit) ks = kMaxKSplit;
    if (ks > p.nchunks) ks = p.nchunks;
    if (ks < 1) ks = 1;
    p.chunks_per_split = (p.nchunks + ks - 1) / ks;
    p.ksplit = (p.nchunks + p.chunks_per_split - 1) / p.chunks_per_split;
    return p;
}

void launch_pack_w(const mhclite_ctx* c, const ProjPlan& p, int N, const float* W, const float* gain, void* Wp,
                   cudaStream_t s) {
    c->launches += 1;
    const int total = p.ksteps * p.NT * 32;
    pack_w_k<<<(total + 255) / 256, 256, 0, s>>>(c->n * c->C, N, p.NT, p.ksteps, W, gain, (uint4*)Wp);
}

template <int NT, int WN>
static void launch_fwd_t(int64_t T, int nC, const ProjPlan& p, const void* x, const void* Wp, float* qpart, float* ssq,
                         cudaStream_t s) {
    using Cfg = FwdCfg<NT, WN>;
    cudaFuncSetAttribute(proj_fwd_mma_k<NT, WN>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem);
    dim3 grid((unsigned)((T + kTileTok - 1) / kTileTok), p.ksplit);
    proj_fwd_mma_k<NT, WN><<<grid, 256, Cfg::kSmem, s>>>(T, nC, p.nchunks, p.chunks_per_split, (const __nv_bfloat16*)x,
                                                         (const uint4*)Wp, qpart, ssq);
}

void launch_proj_fwd_mma(const mhclite_ctx* c, int64_t T, const ProjPlan& p, const void* x, const void* Wp,
                         float* qpart, float* ssq, cudaStream_t s) {
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_PROJ_FWD, s);
    const int nC = c->n * c->C;
    switch (p.NT) {
        case 1: launch_fwd_t<1, 1>(T, nC, p, x, Wp, qpart, ssq, s); break;
        case 2: launch_fwd_t<2, 1>(T, nC, p, x, Wp, qpart, ssq, s); break;
        case 3: launch_fwd_t<3, 1>(T, nC, p, x, Wp, qpart, ssq, s); break;
        case 4: launch_fwd_t<4, 1>(T, nC, p, x, Wp, qpart, ssq, s); break;
        case 5: launch_fwd_t<5, 1>(T, nC, p, x, Wp, qpart, ssq, s); break;
        default: launch_fwd_t<20, 4>(T, nC, p, x, Wp, qpart, ssq, s); break;
    }
}

}  // namespace mhcl
