// Layer-to-layer fusion for stacks of Hyper-Connections layers: the merge of layer l (paper Eq. (1))
//
//     x_{l+1}[t,i,:] = sum_j H_res[t,i,j] x_l[t,j,:] + H_post[t,i] y[t,:]
//
// writes x_{l+1} and, from the same tile while it is still in shared memory, produces what layer l+1 needs first
// (Eq. (4), first two lines): the RMSNorm sum of squares of x_{l+1} and the projection q = x_{l+1} W' with
// W' = diag(gain_{l+1}) W_{l+1}.  x_{l+1} is then not read again for the projection of the next layer.
//
// A CTA takes tiles of tm <= 128 tokens and walks the C / 64 channel blocks of a tile; per block ("stage"):
//   * TMA (128-byte swizzle) brings the n boxes of x_l [tm tokens x 64 channels], the box of y, and the n tiles of
//     W' (bf16 hi rows | lo rows, K-major) that belong to these channels of the n streams;
//   * sixteen merge warps (thread = token, four threads per token splitting the row's eight 16-byte pieces) compute
//     the n output boxes with packed fp32 FMAs and write them OVER the x boxes, in the same swizzled layout (a
//     thread has read every input of a piece before it writes there); they also add up the squares of the
//     rounded outputs;
//   * the output boxes are now both the data of a TMA store to x_{l+1} and the K-major A operand of
//     tcgen05.mma (M = 128, N = 2 Nq, K = 16) against the W' tiles; the accumulator [128 x 2 Nq] of a tile lives
//     in tensor memory (two of them, so the next tile's MMAs run under this tile's read-out).
// At the end of a tile the merge warps fetch the accumulator (hi + lo parts) and store the token's row of
// projection partials and its sum of squares, in the layout the activation kernels read.
// Every mbarrier wait is bounded; on a time-out the CTA raises its abort flag, records MHCLITE_ERR_TIMEOUT in the
// status word, lets copies in flight land, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"
#include "tc.cuh"

namespace mhcl {

constexpr int kPpRows = 128;                      // UMMA M: rows of the accumulator
constexpr int kPpBox = kPpRows * 128;             // bytes reserved per box: 128 rows x 64 channels of bf16
constexpr int kPpMergeWarps = 16;                 // four per lane quadrant: each takes two of a row's eight pieces
constexpr int kPpThreads = 128 + 32 * kPpMergeWarps;   // warp 0 loads, 1 issues MMAs, 2 stores, 3 idles; 4.. merge
constexpr int kPpMaxStages = 3;

struct PpCtl {
    uint64_t full[kPpMaxStages], merged[kPpMaxStages], empty[kPpMaxStages], acc_full[2], acc_empty[2], sq_ready[2];
    uint32_t tmem_base;
    int abort[3];
    float ssq_s[kPpMergeWarps / 4 - 1][kPpRows];   // the other warps' sums of squares of the tile that is being read out
};

struct PpArgs {
    int64_t T;
    int C, tm, ntiles, nq, n_out, stages, tmem_cols;
    const float *H_res, *H_post;
    float *qpart, *ssq;
    int* status;
};

__device__ __forceinline__ uint64_t pp_desc_k128(uint32_t addr) {     // K-major rows of 128 bytes, 128-byte swizzle
    return smem_desc(addr, 16, 1024, 2);
}
// Asks the L2 cache for a box ahead of the TMA load that will bring it to shared memory.
__device__ __forceinline__ void pp_prefetch(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void pp_tma_store(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}

template <int N_>
__global__ void __launch_bounds__(kPpThreads, 1)
postres_proj_k(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmy,
               const __grid_constant__ CUtensorMap tmo, const __grid_constant__ CUtensorMap tmw, const PpArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int w_tile = 2 * a.nq * 128;                         // hi rows then lo rows of one stream's 64 channels
    const int stage_bytes = (N_ + 1) * kPpBox + N_ * w_tile;
    const int umma_n = 2 * a.nq;
    PpCtl* ctl = reinterpret_cast<PpCtl*>(smem + a.stages * stage_bytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nchunk = a.C / 64;
    volatile int* abort = ctl->abort;

    if (tid == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);
            mbar_init(smem_u32(&ctl->merged[s]), kPpMergeWarps);
            mbar_init(smem_u32(&ctl->empty[s]), 2);            // the MMAs have read the boxes + the store has
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), 4);
            mbar_init(smem_u32(&ctl->sq_ready[b]), kPpMergeWarps - 4);
        }
        ctl->abort[0] = ctl->abort[1] = ctl->abort[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        // ---- loader: lane b < 2 n + 1 issues the copy of box b (x boxes, y box, W' tiles); lane 0 arms the barrier
        const int nb = 2 * N_ + 1;
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
            const int row0 = tile * a.tm;
            for (int cb = 0; cb < nchunk && ok; ++cb, ++it) {
                const int s = it % a.stages;
                if (lane == 0) ok = mbar_wait(smem_u32(&ctl->empty[s]), ((it / a.stages) & 1) ^ 1, abort, 1, it);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t full = smem_u32(&ctl->full[s]);
                if (lane == 0) mbar_expect_tx(full, (uint32_t)((N_ + 1) * a.tm * 128 + N_ * w_tile));
                __syncwarp();
                const uint32_t slot = smem_u32(smem + s * stage_bytes);
                // the boxes two stages ahead start their way from HBM to L2 now: with two or three slots, each busy
                // for a whole load + merge + store round, the loads alone keep too few bytes in flight
                int pcb = cb + a.stages, prow = row0;
                if (pcb >= nchunk) { pcb -= nchunk; prow = (tile + (int)gridDim.x) * a.tm; }
                const bool pf = pcb < nchunk && (int64_t)prow < a.T;
                if (lane < N_) {
                    tma_load_2d(slot + lane * kPpBox, &tmx, full, lane * a.C + cb * 64, row0);
                    if (pf) pp_prefetch(&tmx, lane * a.C + pcb * 64, prow);
                } else if (lane == N_) {
                    tma_load_2d(slot + N_ * kPpBox, &tmy, full, cb * 64, row0);
                    if (pf) pp_prefetch(&tmy, pcb * 64, prow);
                } else if (lane < nb) {
                    const int i = lane - N_ - 1;
                    tma_load_2d(slot + (N_ + 1) * kPpBox + i * w_tile, &tmw, full, i * a.C + cb * 64, 0);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_mn(kPpRows, umma_n, 0, 0);
            int it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x, ++tcount) {
                const int b = tcount & 1;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), ((tcount >> 1) & 1) ^ 1, abort, 2, tcount);
                for (int cb = 0; cb < nchunk && ok; ++cb, ++it) {
                    const int s = it % a.stages;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (it / a.stages) & 1, abort, 3, it) &&
                         mbar_wait(smem_u32(&ctl->merged[s]), (it / a.stages) & 1, abort, 4, it);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t slot = smem_u32(smem + s * stage_bytes);
#pragma unroll
                    for (int i = 0; i < N_; ++i) {
                        const uint64_t ad = pp_desc_k128(slot + i * kPpBox);
                        const uint64_t bd = pp_desc_k128(slot + (N_ + 1) * kPpBox + i * w_tile);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)             // 32 bytes further along the swizzled row per k-step
                            tc_mma(tmem + b * umma_n, ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 2), idesc,
                                   (cb > 0 || i > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) tc_commit(smem_u32(&ctl->acc_full[b]));
            }
        }
    } else if (warp == 2) {
        // ---- store: lane i sends box i of a merged stage to x_next, then the slot's share of `empty` ----
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
            const int row0 = tile * a.tm;
            for (int cb = 0; cb < nchunk && ok; ++cb, ++it) {
                const int s = it % a.stages;
                if (lane == 0) ok = mbar_wait(smem_u32(&ctl->merged[s]), (it / a.stages) & 1, abort, 5, it);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane < N_) {
                    pp_tma_store(&tmo, smem_u32(smem + s * stage_bytes) + lane * kPpBox, lane * a.C + cb * 64, row0);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->empty[s]));
            }
        }
        if (lane < N_) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    } else if (warp >= 4) {
        // ---- merge + read-out: thread = token row, the two warps of a lane quadrant share the row's pieces ----
        const int quad = warp & 3, half = (warp - 4) >> 2;
        const int row = quad * 32 + lane;
        int it = 0, tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < a.ntiles; tile += gridDim.x, ++tcount) {
            const int64_t t = (int64_t)tile * a.tm + row;
            const bool live = row < a.tm && t < a.T;
            uint64_t hr2[N_][N_], hp2[N_];
#pragma unroll
            for (int i = 0; i < N_; ++i) {
                const float hp = live ? __ldg(a.H_post + t * N_ + i) : 0.f;
                hp2[i] = pack2f(hp, hp);
#pragma unroll
                for (int j = 0; j < N_; ++j) {
                    const float h = live ? __ldg(a.H_res + (t * N_ + i) * N_ + j) : 0.f;
                    hr2[i][j] = pack2f(h, h);
                }
            }
            uint64_t sq2 = pack2f(0.f, 0.f);
            for (int cb = 0; cb < nchunk; ++cb, ++it) {
                const int s = it % a.stages;
                if (ok) ok = mbar_wait(smem_u32(&ctl->full[s]), (it / a.stages) & 1, abort, 6, it);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t slot = smem_u32(smem + s * stage_bytes);
                if (row < a.tm) {
#pragma unroll
                    for (int pp = 0; pp < 32 / kPpMergeWarps; ++pp) {
                        const int pc = half * (32 / kPpMergeWarps) + pp;       // 16-byte piece of the 128-byte row
                        const int po = row * 128 + ((pc ^ (row & 7)) << 4);
                        uint64_t xf[N_][4], yf[4];
#pragma unroll
                        for (int j = 0; j < N_; ++j) unpack8x2(lds128(slot + j * kPpBox + po), xf[j]);
                        unpack8x2(lds128(slot + N_ * kPpBox + po), yf);
#pragma unroll
                        for (int i = 0; i < N_; ++i) {
                            uint64_t o[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) o[k] = fma2(hp2[i], yf[k], pack2f(0.f, 0.f));
#pragma unroll
                            for (int j = 0; j < N_; ++j)
#pragma unroll
                                for (int k = 0; k < 4; ++k) o[k] = fma2(hr2[i][j], xf[j][k], o[k]);
                            const uint4 v = pack8x2(o);
                            sts128(slot + i * kPpBox + po, v);
                            uint64_t r[4];                                       // the next layer normalises what is stored
                            unpack8x2(v, r);
#pragma unroll
                            for (int k = 0; k < 4; ++k) sq2 = fma2(r[k], r[k], sq2);
                        }
                    }
                }
                // the boxes now hold x_next: visible to the TMA store and to the tensor cores, then signal
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->merged[s]));
            }
            if (!ok) break;
            const int b = tcount & 1;
            float sqa, sqb;
            unpack2f(sq2, sqa, sqb);
            const float sq = sqa + sqb;
            if (half != 0) {
                // the one buffer of partial sums is free once the tile before this one has been read out
                if (tcount > 0) ok = mbar_wait(smem_u32(&ctl->acc_empty[(tcount - 1) & 1]), ((tcount - 1) >> 1) & 1, abort, 9, tcount);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ctl->ssq_s[half - 1][row] = sq;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->sq_ready[b]));
            } else {
                ok = mbar_wait(smem_u32(&ctl->sq_ready[b]), (tcount >> 1) & 1, abort, 7, tcount) &&
                     mbar_wait(smem_u32(&ctl->acc_full[b]), (tcount >> 1) & 1, abort, 8, tcount);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16) + b * umma_n;
                float* qrow = a.qpart + t * a.n_out;
                for (int c0 = 0; c0 < a.nq; c0 += 16) {
                    float hi[16], lo[16];
                    tc_ld16(lane_base + c0, hi);
                    tc_ld16(lane_base + a.nq + c0, lo);
                    if (live) {
#pragma unroll
                        for (int e = 0; e < 16; e += 4)
                            if (c0 + e < a.nq)
                                *reinterpret_cast<float4*>(qrow + c0 + e) =
                                    make_float4(hi[e] + lo[e], hi[e + 1] + lo[e + 1], hi[e + 2] + lo[e + 2], hi[e + 3] + lo[e + 3]);
                    }
                }
                if (live) {
                    float tot = sq;
#pragma unroll
                    for (int h = 0; h < kPpMergeWarps / 4 - 1; ++h) tot += ctl->ssq_s[h][row];
                    a.ssq[t] = tot;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ctl->abort[0]) report_abort(abort, a.status, 5);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(a.tmem_cols) : "memory");
    }
}

// ---- host side -------------------------------------------------------------------------------------
// Tokens per tile: the multiple of 8 in [64, 128] for which ceil(tiles / SMs) rounds of that many rows are fewest
// (16384 tokens on 148 SMs: 147 tiles of 112 tokens in one round, where 128-token tiles leave 20 SMs idle).
static int pp_tile_rows(int64_t T, int sm_count) {
    int best = kPpRows;
    int64_t best_cost = INT64_MAX;
    for (int tm = kPpRows; tm >= 64; tm -= 8) {
        const int64_t tiles = (T + tm - 1) / tm;
        const int64_t cost = ((tiles + sm_count - 1) / sm_count) * (tm + 4);
        if (cost < best_cost) { best_cost = cost; best = tm; }
    }
    return best;
}

bool postres_proj_supported(int n, int C, int N) {
    const int nq = proj_tc_nq(N);
    return n >= 2 && n <= 4 && (C % 64) == 0 && 2 * nq <= 256 && tensor_maps_available() &&
           2 * ((n + 1) * kPpBox + n * 2 * nq * 128) + (int)sizeof(PpCtl) + 1024 <= 227 * 1024;
}

// x_next = merge(x, y), and the projection partials (one K slice: qpart[0][T][Npad], ssq[0][T]) of x_next against the
// packed W' of the next layer (Wt, see pack_wt_k).  False (nothing launched) when the shape is not supported.
bool launch_postres_proj(const mhclite_ctx* c, int64_t T, int N, const ProjPlan& pp, const void* x, const void* y,
                         const float* H_res, const float* H_post, void* x_next, const void* Wt, float* qpart, float* ssq,
                         int* status, cudaStream_t s) {
    const int n = c->n, C = c->C, nC = n * C;
    if (!postres_proj_supported(n, C, N)) return false;
    const int nq = proj_tc_nq(N), Kpad = pp.nchunks * 64;
    if (nq > pp.Npad) return false;
    PpArgs a;
    a.T = T; a.C = C; a.nq = nq; a.n_out = pp.Npad;
    a.tm = pp_tile_rows(T, c->sm_count);
    a.ntiles = (int)((T + a.tm - 1) / a.tm);
    const int stage_bytes = (n + 1) * kPpBox + n * 2 * nq * 128;
    a.stages = (227 * 1024 - (int)sizeof(PpCtl) - 1024) / stage_bytes;
    if (a.stages > kPpMaxStages) a.stages = kPpMaxStages;
    if (a.stages < 2) return false;
    a.tmem_cols = 32;
    while (a.tmem_cols < 2 * 2 * nq) a.tmem_cols *= 2;
    a.H_res = H_res; a.H_post = H_post; a.qpart = qpart; a.ssq = ssq; a.status = status;
    CUtensorMap tmx, tmy, tmo, tmw;
    if (!make_tensor_map_2d(&tmx, x, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, 64, (uint32_t)a.tm, 128)) return false;
    if (!make_tensor_map_2d(&tmy, y, (uint64_t)C, (uint64_t)T, (uint64_t)C, 64, (uint32_t)a.tm, 128)) return false;
    if (!make_tensor_map_2d(&tmo, x_next, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, 64, (uint32_t)a.tm, 128)) return false;
    if (!make_tensor_map_2d(&tmw, Wt, (uint64_t)Kpad, (uint64_t)(2 * nq), (uint64_t)Kpad, 64, (uint32_t)(2 * nq), 128)) return false;
    const int smem = a.stages * stage_bytes + (int)sizeof(PpCtl) + 1024;
    const int grid = a.ntiles < c->sm_count ? a.ntiles : c->sm_count;
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_POSTRES_FWD, s);
#define MHCL_PP(N_)                                                                                            \
    do {                                                                                                       \
        cudaFuncSetAttribute(postres_proj_k<N_>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);           \
        postres_proj_k<N_><<<grid, kPpThreads, smem, s>>>(tmx, tmy, tmo, tmw, a);                               \
    } while (0)
    switch (n) {
        case 2: MHCL_PP(2); break;
        case 3: MHCL_PP(3); break;
        default: MHCL_PP(4); break;
    }
#undef MHCL_PP
    return true;
}

}  // namespace mhcl
