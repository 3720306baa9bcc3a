// Blackwell tensor-core backward of the projection of paper Eq. (4) for wide projections (n = 5: 130
// columns), where the accumulators of the mma.sync kernel no longer fit the register file.
//
//   tail_g_tc_k :  G[m,c] = sum_t x[t,m] e[t,c]  (dW = gain (.) G, dgain = sum_c W G), a split-token GEMM
//                  with M = 128 rows of the flattened n*C axis per accumulator, N = Kp columns,
//                  K = tokens.  x tiles arrive by TMA (128-byte swizzle, [token][64 channels]) and are the
//                  MN-major A operand; the tiled e buffers (hi and lo, see e_tiled_index) are copied as they
//                  are (bulk copies) and form the MN-major B operand without swizzle.  hi and lo accumulate
//                  into the same fp32 accumulator in tensor memory; up to three accumulators per CTA share
//                  one pass over e.  Each token range writes its own partial (no atomics).
//
// Warp roles (192 threads): warp 0 = producer, warp 1 = MMA issuer and owner of the tensor memory,
// warps 2..5 = epilogue (tensor-memory lane quadrant = warp % 4).  All mbarrier waits are bounded; on a
// time-out the CTA raises its abort flag, records MHCLITE_ERR_TIMEOUT in the status word, lets copies in
// flight land, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"
#include "tc.cuh"

namespace mhcl {

constexpr int kGTok = 64;                       // tokens per stage of the G kernel (4 k-steps of 16)
constexpr int kGStages = 2;
constexpr int kGXBox = kGTok * 128;             // one TMA box: 64 tokens x 64 channels of bf16

struct GCtl {
    uint64_t full[kGStages], empty[kGStages], accum;
    uint32_t tmem_base;
    int abort;
};

template <int MT>
__global__ void __launch_bounds__(192, 1)
tail_g_tc_k(const __grid_constant__ CUtensorMap tmx, const __nv_bfloat16* __restrict__ ehi,
            const __nv_bfloat16* __restrict__ elo, int64_t T, int64_t tok_per_split, int nC, int Kp, int tmem_cols,
            float* __restrict__ Gpart, int* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int ncg = Kp >> 3;                                   // 8-column groups
    const int x_bytes = MT * 2 * kGXBox;
    const int e_bytes = ncg * (kGTok * 16);                    // one of hi / lo: [column group][64 tokens][16 B]
    const int stage_bytes = x_bytes + 2 * e_bytes;
    GCtl* ctl = reinterpret_cast<GCtl*>(smem + kGStages * stage_bytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = blockIdx.x * (MT * 128);
    const int64_t t_begin = (int64_t)blockIdx.y * tok_per_split;       // multiple of 128
    const int64_t t_end = (t_begin + tok_per_split < T) ? t_begin + tok_per_split : T;
    const int nblk = (t_end > t_begin) ? (int)((t_end - t_begin + kGTok - 1) / kGTok) : 0;
    volatile int* abort = &ctl->abort;

    if (tid == 0) {
        for (int s = 0; s < kGStages; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        mbar_init(smem_u32(&ctl->accum), 1);
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < nblk; ++i) {
                const int s = i % kGStages;
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ((i / kGStages) & 1) ^ 1, abort)) break;
                const uint32_t full = smem_u32(&ctl->full[s]);
                mbar_expect_tx(full, stage_bytes);
                const uint32_t dst = smem_u32(smem + s * stage_bytes);
                const int64_t t0 = t_begin + (int64_t)i * kGTok;
#pragma unroll
                for (int b = 0; b < MT * 2; ++b) tma_load_2d(dst + b * kGXBox, &tmx, full, m0 + b * 64, (int)t0);
                // the 64 tokens' pieces of every column group: 1 KB runs, 2 KB apart in the granule
                const int64_t gran = (t0 >> 7) * ncg * 1024 + (t0 & 64) * 8;       // element offset
                for (int cg = 0; cg < ncg; ++cg) {
                    bulk_load(dst + x_bytes + cg * 1024, ehi + gran + (int64_t)cg * 1024, 1024, full);
                    bulk_load(dst + x_bytes + e_bytes + cg * 1024, elo + gran + (int64_t)cg * 1024, 1024, full);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_mn(128, Kp, 1, 1);
            bool ok = true;
            for (int i = 0; i < nblk && ok; ++i) {
                const int s = i % kGStages;
                ok = mbar_wait(smem_u32(&ctl->full[s]), (i / kGStages) & 1, abort);
                if (!ok) break;
                tc_fence_after();
                const uint32_t xs = smem_u32(smem + s * stage_bytes), eh = xs + x_bytes, el = eh + e_bytes;
#pragma unroll
                for (int ks = 0; ks < kGTok / 16; ++ks) {
                    // B: columns = N (8-column groups 1 KB apart), tokens = K (8-token groups 128 B apart)
                    const uint64_t bh = smem_desc(eh + ks * 256, 128, 1024, 0);
                    const uint64_t bl = smem_desc(el + ks * 256, 128, 1024, 0);
#pragma unroll
                    for (int a = 0; a < MT; ++a) {
                        // A: 128 channels = two 64-channel swizzle groups one box apart, 8-token groups 1 KB apart
                        const uint64_t ad = smem_desc(xs + a * 2 * kGXBox + ks * 2048, kGXBox, 1024, 2);
                        tc_mma(tmem + a * Kp, ad, bh, idesc, (i > 0 || ks > 0) ? 1u : 0u);
                        tc_mma(tmem + a * Kp, ad, bl, idesc, 1u);
                    }
                }
                tc_commit(smem_u32(&ctl->empty[s]));
            }
            if (ok && nblk > 0) tc_commit(smem_u32(&ctl->accum));
        }
    } else {
        const int quad = warp & 3;
        bool ok = nblk == 0 || mbar_wait(smem_u32(&ctl->accum), 0, abort);
        ok = __all_sync(0xffffffffu, ok);
        if (ok && nblk > 0) {
            tc_fence_after();
            float* Gp = Gpart + (int64_t)blockIdx.y * nC * Kp;
#pragma unroll
            for (int a = 0; a < MT; ++a) {
                const int m = m0 + a * 128 + quad * 32 + lane;
                const uint32_t taddr = tmem + ((uint32_t)(quad * 32) << 16) + a * Kp;
                for (int c0 = 0; c0 < Kp; c0 += 16) {
                    float v[16];
                    tc_ld16(taddr + c0, v);
                    if (m < nC) {
                        float* row = Gp + (int64_t)m * Kp + c0;
#pragma unroll
                        for (int e = 0; e < 16; e += 4)
                            *reinterpret_cast<float4*>(row + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
                    }
                }
            }
        } else if (ok) {                                   // empty token range: the partial is zero
            float* Gp = Gpart + (int64_t)blockIdx.y * nC * Kp;
            for (int a = 0; a < MT; ++a) {
                const int m = m0 + a * 128 + quad * 32 + lane;
                if (m < nC) for (int c = 0; c < Kp; ++c) Gp[(int64_t)m * Kp + c] = 0.f;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ctl->abort) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        if (tid == 0) atomicExch(status, MHCLITE_ERR_TIMEOUT);
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    }
}

// ---- host side -------------------------------------------------------------------------------------
template <int MT>
static void launch_g_t(const TailPlan& p, const CUtensorMap& tmx, const void* ehi, const void* elo, int64_t T, int nC,
                       float* Gpart, int* status, cudaStream_t s) {
    const int stage_bytes = MT * 2 * kGXBox + 2 * (p.Kp >> 3) * (kGTok * 16);
    const int smem = kGStages * stage_bytes + (int)sizeof(GCtl) + 1024;
    int tmem_cols = 32;
    while (tmem_cols < MT * p.Kp) tmem_cols *= 2;
    cudaFuncSetAttribute(tail_g_tc_k<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    dim3 grid(p.g_groups, p.g_splits);
    tail_g_tc_k<MT><<<grid, 192, smem, s>>>(tmx, (const __nv_bfloat16*)ehi, (const __nv_bfloat16*)elo, T,
                                            p.g_tok_per_split, nC, p.Kp, tmem_cols, Gpart, status);
}

// G partials of every token range -> Gpart[g_splits][nC][Kp].  False when no tensor map could be made.
bool launch_tail_g_tc(const mhclite_ctx* c, int64_t T, const TailPlan& p, const void* x, const void* ehi,
                      const void* elo, float* Gpart, int* status, cudaStream_t s) {
    const int nC = c->n * c->C;
    CUtensorMap tmx;
    if (!make_tensor_map_2d(&tmx, x, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, 64, kGTok, 128)) return false;
    c->launches += 1;
    switch (p.g_mt) {
        case 1: launch_g_t<1>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
        case 2: launch_g_t<2>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
        default: launch_g_t<3>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
    }
    return true;
}

}  // namespace mhcl
