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

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z) : "memory");
}

constexpr int kGTok = 64;                       // tokens per stage of the G kernel (4 k-steps of 16)
constexpr int kGStages = 2;
constexpr int kGXBox = kGTok * 128;             // one TMA box: 64 tokens x 64 channels of bf16

struct GCtl {
    uint64_t full[kGStages], empty[kGStages], accum;
    uint32_t tmem_base;
    int abort[3];
};

template <int MT>
__global__ void __launch_bounds__(192, 1)
tail_g_tc_k(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmeh,
            const __grid_constant__ CUtensorMap tmel, int64_t T, int64_t tok_per_split, int nC, int Kp, int tmem_cols,
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
    volatile int* abort = ctl->abort;

    if (tid == 0) {
        for (int s = 0; s < kGStages; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        mbar_init(smem_u32(&ctl->accum), 1);
        ctl->abort[0] = ctl->abort[1] = ctl->abort[2] = 0;
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
        // Producer: lane b issues copy b of a stage (the x boxes, then the 64 tokens' pieces of every column group of e_hi
        // and of e_lo as one box each: 1 KB runs, 2 KB apart in the granule); lane 0 waits for the stage and arms it.
        // One thread issuing every copy in turn (forty-odd of them while e went by plain bulk copies) was what bound
        // this kernel.
        bool ok = true;
        for (int i = 0; i < nblk && ok; ++i) {
            const int s = i % kGStages;
            if (lane == 0) ok = mbar_wait(smem_u32(&ctl->empty[s]), ((i / kGStages) & 1) ^ 1, abort, 1, i);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t full = smem_u32(&ctl->full[s]);
            if (lane == 0) mbar_expect_tx(full, stage_bytes);
            __syncwarp();
            const uint32_t dst = smem_u32(smem + s * stage_bytes);
            const int64_t t0 = t_begin + (int64_t)i * kGTok;
            if (lane < MT * 2) {
                tma_load_2d(dst + lane * kGXBox, &tmx, full, m0 + lane * 64, (int)t0);
            } else if (lane < MT * 2 + 2) {
                const int lo = lane - MT * 2;
                tma_load_3d(dst + x_bytes + lo * e_bytes, lo ? &tmel : &tmeh, full, 0, (int)((t0 & 64) >> 3), (int)((t0 >> 7) * ncg));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_mn(128, Kp, 1, 1);
            bool ok = true;
            for (int i = 0; i < nblk && ok; ++i) {
                const int s = i % kGStages;
                ok = mbar_wait(smem_u32(&ctl->full[s]), (i / kGStages) & 1, abort, 2, i);
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
        bool ok = nblk == 0 || mbar_wait(smem_u32(&ctl->accum), 0, abort, 3, 0);
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
    if (ctl->abort[0]) report_abort(abort, status, 2);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
//   tail_dx_tc_k : dxhat[t,m] = sum_c e[t,c] W'[m,c] - x[t,m] kappa_t, fused with the rest of dx:
//                    MODE 1:  dx[t,j,c] = sum_i H_res[t,i,j] g[t,i,c] + H_pre[t,j] du[t,c] + dxhat[t,j*C+c]
//                    MODE 0:  dx = dxhat          MODE 2:  dx += dxhat
//   A CTA keeps the e tile of 128 tokens (hi part, one granule of the tiled buffer) in shared memory and
//   walks over blocks of 32 channels.  Per block the W' operand of all n streams ([n x 32 channels] x Kp,
//   packed by pack_wb_k, K-major without swizzle) streams through a ring one k-step at a time; one
//   tcgen05.mma per k-step (M = 128 tokens, N = n x 32 channels, K = 16) leaves dxhat of all n streams in
//   one of up to three tensor-memory buffers.  Eight epilogue warps (thread = token, two warps per lane
//   quadrant) combine it with x, g and du, which TMA delivers per 32-token quadrant (64-byte swizzle;
//   3-D maps [token][stream][channel], so that a block that sticks out of C is clipped) through a ring of up
//   to six slots (load number l goes to slot l mod 6: the next loads of two quadrants are under way
//   while all four still work), write dx over the g boxes of the slot and hand those to a TMA store.
//   Work items (token tile, channel block) are dealt out in contiguous runs, one run per CTA, so that the
//   e tile is reloaded only at tile changes.
constexpr int kDTok = 128;                      // tokens per tile (UMMA M)
constexpr int kDCh = 32;                        // channels per block and stream
constexpr int kDBox = 32 * 64;                  // one TMA box: 32 tokens x 32 channels of bf16
constexpr int kDWSlots = 8;                     // ring of W' k-steps ([n x 32 channels] x 16 columns each)
constexpr int kDMaxSlots = 6;                   // data slots
constexpr int kDMaxRing = 3;                    // dxhat buffers in tensor memory

// The full barriers belong to a quadrant (two in turn), the free barriers to a slot: a parity wait is only
// safe for a waiter that sees every phase of its barrier, and a slot serves all quadrants in turn.
struct DCtl {
    uint64_t e_full, e_empty, w_full[kDWSlots], w_empty[kDWSlots], d_full[4][2], s_free[kDMaxSlots], q_done[4],
        acc_full[kDMaxRing], acc_empty[kDMaxRing];
    uint32_t tmem_base;
    int abort[3];
};

struct DxArgs {
    int64_t T;
    int C, Kp, ncb;                 // channels per stream, padded projection columns, channel blocks per stream
    int64_t items, per_cta;         // work items = token tiles x channel blocks
    int tmem_cols, ring, dslots;
    const __nv_bfloat16* ehi;       // tiled
    const __nv_bfloat16* Wb;        // [ncb][Kp/8][n x 32][8]
    const float *kappa, *H_res, *H_pre;
    int* status;
};

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tc_ld8_nowait(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Ties the registers of an earlier tcgen05.ld to a point after the wait, so that no use is scheduled before it.
__device__ __forceinline__ void tc_ld_settle(uint32_t (&r)[8]) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]) :: "memory");
}

constexpr int kDThreads = 96 + 256;              // operand producer, MMA issuer, data producer, 8 epilogue warps

template <int N_, int MODE>
__global__ void __launch_bounds__(kDThreads, 1)
tail_dx_tc_k(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmg,
             const __grid_constant__ CUtensorMap tmdu, const __grid_constant__ CUtensorMap tmdx, const DxArgs a) {
    constexpr int kBoxes = MODE == 1 ? 2 * N_ + 1 : (MODE == 2 ? 2 * N_ : N_);
    constexpr int kOut = MODE == 0 ? 0 : N_;                   // dx takes the place of g (of the old dx; of x in MODE 0)
    constexpr int kDSlot = kBoxes * kDBox;
    constexpr int kDW = N_ * kDCh;                             // tensor-memory columns of one dxhat buffer = UMMA N
    constexpr int kWChunk = kDW * 32;                          // bytes of one k-step of W'
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int e_bytes = a.Kp * kDTok * 2;
    unsigned char* e_s = smem;
    unsigned char* w_s = e_s + e_bytes;                        // e_bytes is a multiple of 4096
    unsigned char* d_s = w_s + kDWSlots * kWChunk;             // a multiple of 1024
    DCtl* ctl = reinterpret_cast<DCtl*>(d_s + a.dslots * kDSlot);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t it_begin = (int64_t)blockIdx.x * a.per_cta;
    const int64_t it_end = (it_begin + a.per_cta < a.items) ? it_begin + a.per_cta : a.items;
    const int nit = it_end > it_begin ? (int)(it_end - it_begin) : 0;
    const int ksteps = a.Kp >> 4;
    volatile int* abort = ctl->abort;

    if (tid == 0) {
        mbar_init(smem_u32(&ctl->e_full), 1); mbar_init(smem_u32(&ctl->e_empty), 1);
        for (int s = 0; s < kDWSlots; ++s) { mbar_init(smem_u32(&ctl->w_full[s]), 1); mbar_init(smem_u32(&ctl->w_empty[s]), 1); }
        for (int q = 0; q < 4; ++q) {
            mbar_init(smem_u32(&ctl->d_full[q][0]), 1); mbar_init(smem_u32(&ctl->d_full[q][1]), 1);
            mbar_init(smem_u32(&ctl->q_done[q]), 2);
        }
        for (int s = 0; s < kDMaxSlots; ++s) mbar_init(smem_u32(&ctl->s_free[s]), 1);
        for (int s = 0; s < kDMaxRing; ++s) { mbar_init(smem_u32(&ctl->acc_full[s]), 1); mbar_init(smem_u32(&ctl->acc_empty[s]), 8); }
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
        // ---- producer of the MMA operands: e tile at tile changes, W' one k-step at a time ----------------
        if (lane == 0) {
            int64_t cur_tile = -1;
            int ec = 0;
            bool ok = true;
            for (int li = 0; li < nit && ok; ++li) {
                const int64_t item = it_begin + li;
                const int64_t tile = item / a.ncb;
                const int cb = (int)(item - tile * a.ncb);
                if (tile != cur_tile) {
                    ok = mbar_wait(smem_u32(&ctl->e_empty), (ec & 1) ^ 1, abort, 1, li);
                    if (!ok) break;
                    mbar_expect_tx(smem_u32(&ctl->e_full), e_bytes);
                    bulk_load(smem_u32(e_s), a.ehi + tile * (int64_t)a.Kp * kDTok, e_bytes, smem_u32(&ctl->e_full));
                    cur_tile = tile;
                    ++ec;
                }
                const __nv_bfloat16* wsrc = a.Wb + (int64_t)cb * (a.Kp >> 3) * (kDW * 8);
                for (int ks = 0; ks < ksteps && ok; ++ks) {
                    const int wi = li * ksteps + ks, ws = wi % kDWSlots;
                    ok = mbar_wait(smem_u32(&ctl->w_empty[ws]), ((wi / kDWSlots) & 1) ^ 1, abort, 2, wi);
                    if (!ok) break;
                    mbar_expect_tx(smem_u32(&ctl->w_full[ws]), kWChunk);
                    bulk_load(smem_u32(w_s + ws * kWChunk), wsrc + (int64_t)ks * (kDW * 16), kWChunk, smem_u32(&ctl->w_full[ws]));
                }
            }
        }
    } else if (warp == 2) {
        // ---- producer of the epilogue's data: x, g, du per 32-token quadrant, as far ahead as the ring allows.
        //      Lane b issues the copy of box b (issuing a TMA instruction keeps a thread busy for ~100 cycles: eleven in
        //      a row from one thread would hold back the slots behind it); lane 0 waits for the slot and arms the barrier.
        const CUtensorMap* mp = lane < N_ ? &tmx : (lane < 2 * N_ ? &tmg : &tmdu);
        const int jj = lane < N_ ? lane : (lane < 2 * N_ ? lane - N_ : 0);
        bool ok = true;
        for (int li = 0; li < nit && ok; ++li) {
            const int64_t item = it_begin + li;
            const int64_t tile = item / a.ncb;
            const int cb = (int)(item - tile * a.ncb);
            for (int q = 0; q < 4 && ok; ++q) {
                const int l = li * 4 + q, sl = l % a.dslots;
                if (lane == 0) ok = mbar_wait(smem_u32(&ctl->s_free[sl]), ((l / a.dslots) & 1) ^ 1, abort, 3, l);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t full = smem_u32(&ctl->d_full[q][li & 1]);
                if (lane == 0) mbar_expect_tx(full, kDSlot);
                __syncwarp();
                // (no L2 prefetch of the next item here: the tensor maps promote L2 fills to 256 bytes, so three of four
                //  channel blocks already hit, and the TMA unit is what this kernel keeps busiest: a prefetch per box
                //  made it 1.4 x slower)
                if (lane < kBoxes)
                    tma_load_3d(smem_u32(d_s + sl * kDSlot) + lane * kDBox, mp, full, cb * kDCh, jj, (int)(tile * kDTok + q * 32));
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -----------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_mn(128, kDW, 0, 0);
            int64_t cur_tile = -1;
            int ec = 0;
            bool ok = true;
            for (int li = 0; li < nit && ok; ++li) {
                const int64_t item = it_begin + li;
                const int64_t tile = item / a.ncb;
                const int rr = li % a.ring;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[rr]), ((li / a.ring) & 1) ^ 1, abort, 4, li);
                if (!ok) break;
                if (tile != cur_tile) {
                    ok = mbar_wait(smem_u32(&ctl->e_full), ec & 1, abort, 5, li);
                    if (!ok) break;
                    cur_tile = tile;
                    ++ec;
                }
                const uint32_t ea = smem_u32(e_s);
                for (int ks = 0; ks < ksteps && ok; ++ks) {
                    const int wi = li * ksteps + ks, ws = wi % kDWSlots;
                    ok = mbar_wait(smem_u32(&ctl->w_full[ws]), (wi / kDWSlots) & 1, abort, 6, wi);
                    if (!ok) break;
                    tc_fence_after();
                    // A: tokens x columns, K-major, no swizzle: column groups 2 KB apart, 8-token groups 128 B apart
                    // B: channels x columns, K-major, no swizzle: column groups n x 512 B apart, 8-channel groups 128 B apart
                    tc_mma(tmem + rr * kDW, smem_desc(ea + ks * 4096, 2048, 128, 0),
                           smem_desc(smem_u32(w_s + ws * kWChunk), kDW * 16, 128, 0), idesc, ks > 0 ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->w_empty[ws]));
                }
                if (!ok) break;
                tc_commit(smem_u32(&ctl->acc_full[rr]));
                const bool last_of_tile = (li + 1 == nit) || ((item + 1) / a.ncb != tile);
                if (last_of_tile) tc_commit(smem_u32(&ctl->e_empty));
            }
        }
    } else {
        // ---- epilogue: thread = token; the two warps of a lane quadrant take 16 channels each ---------
        const int quad = warp & 3;
        const int hw = (warp - 3) >> 2;
        uint64_t nkap2 = pack2f(0.f, 0.f);
        float hp[MODE == 1 ? N_ : 1], hr[MODE == 1 ? N_ : 1][MODE == 1 ? N_ : 1];
        int64_t cur_tile = -1;
        bool ok = true;
        for (int li = 0; li < nit; ++li) {
            const int64_t item = it_begin + li;
            const int64_t tile = item / a.ncb;
            const int cb = (int)(item - tile * a.ncb);
            const int64_t row0 = tile * kDTok + quad * 32;
            const int64_t t = row0 + lane;
            const bool live = t < a.T;
            if (tile != cur_tile) {
                cur_tile = tile;
                const float kap = live ? -__ldg(a.kappa + t) : 0.f;
                nkap2 = pack2f(kap, kap);
                if (MODE == 1) {
#pragma unroll
                    for (int j = 0; j < N_; ++j) hp[j] = live ? __ldg(a.H_pre + t * N_ + j) : 0.f;
#pragma unroll
                    for (int i = 0; i < N_; ++i)
#pragma unroll
                        for (int j = 0; j < N_; ++j) hr[i][j] = live ? __ldg(a.H_res + t * N_ * N_ + i * N_ + j) : 0.f;
                }
            }
            const int rr = li % a.ring;
            const int sl = (li * 4 + quad) % a.dslots;
            ok = mbar_wait(smem_u32(&ctl->acc_full[rr]), (li / a.ring) & 1, abort, 7, li);
            if (ok) ok = mbar_wait(smem_u32(&ctl->d_full[quad][li & 1]), (li >> 1) & 1, abort, 8, li);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t slot = smem_u32(d_s + sl * kDSlot);
            const int rsw = (lane >> 1) & 3;                    // 64-byte swizzle: piece ^= (row / 2) % 4
            const uint32_t tbase = tmem + ((uint32_t)(quad * 32) << 16) + rr * kDW;
#pragma unroll
            for (int pp = 0; pp < 2; ++pp) {
                const int pc = hw * 2 + pp;
                const uint32_t po = lane * 64 + ((pc ^ rsw) << 4);
                uint32_t acc[N_][8];
#pragma unroll
                for (int j = 0; j < N_; ++j) tc_ld8_nowait(tbase + j * kDCh + pc * 8, acc[j]);
                uint64_t gf[MODE == 1 ? N_ : 1][4], df[4];
                if (MODE == 1) {
#pragma unroll
                    for (int i = 0; i < N_; ++i) unpack8x2(lds128(slot + (N_ + i) * kDBox + po), gf[i]);
                    unpack8x2(lds128(slot + 2 * N_ * kDBox + po), df);
                }
                tc_ld_wait();
#pragma unroll
                for (int j = 0; j < N_; ++j) tc_ld_settle(acc[j]);
#pragma unroll
                for (int j = 0; j < N_; ++j) {
                    uint64_t xf[4], o[4];
                    unpack8x2(lds128(slot + j * kDBox + po), xf);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        o[k] = fma2(xf[k], nkap2, pack2f(__uint_as_float(acc[j][2 * k]), __uint_as_float(acc[j][2 * k + 1])));
                    if (MODE == 1) {
                        const uint64_t hp2 = pack2f(hp[j], hp[j]);
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[k] = fma2(hp2, df[k], o[k]);
#pragma unroll
                        for (int i = 0; i < N_; ++i) {
                            const uint64_t h2 = pack2f(hr[i][j], hr[i][j]);
#pragma unroll
                            for (int k = 0; k < 4; ++k) o[k] = fma2(h2, gf[i][k], o[k]);
                        }
                    }
                    if (MODE == 2) {
                        uint64_t old[4];
                        unpack8x2(lds128(slot + (N_ + j) * kDBox + po), old);
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[k] = fma2(old[k], pack2f(1.f, 1.f), o[k]);
                    }
                    sts128(slot + (kOut + j) * kDBox + po, pack8x2(o));
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[rr]));
            // the slot now holds dx: make the writes visible to the TMA unit and meet the quadrant's other warp (both
            // wait for the phase, so neither runs ahead of the other); then lane j of the first warp stores box j
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->q_done[quad]));
            ok = mbar_wait(smem_u32(&ctl->q_done[quad]), li & 1, abort, 9, li);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (hw == 0) {
                if (lane < N_ && row0 < a.T) {
                    tma_store_3d(&tmdx, slot + (kOut + lane) * kDBox, cb * kDCh, lane, (int)row0);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->s_free[sl]));
            }
        }
        if (hw == 0 && lane < N_) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    if (ctl->abort[0]) report_abort(abort, a.status, 3);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(a.tmem_cols) : "memory");
    }
}

// W' = diag(gain) W in bf16 as the B operand of tail_dx_tc_k: per channel block cb a block
// [Kp/8 column groups][n x 32 channels (stream-major)][8 columns]; zero beyond N columns and beyond C channels.
__global__ void __launch_bounds__(256) pack_wb_k(int n, int C, int N, int Kp, int ncb, const float* __restrict__ W,
                                                 const float* __restrict__ gain, __nv_bfloat16* __restrict__ Wb) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t total = (int64_t)n * ncb * Kp * kDCh;
    if (idx >= total) return;
    const int c8 = (int)(idx & 7);
    const int64_t rowi = idx >> 3;                             // (cb * (Kp / 8) + cg) * (n * 32) + j * 32 + channel
    const int rw = (int)(rowi % (n * kDCh));
    const int64_t rest = rowi / (n * kDCh);
    const int cg = (int)(rest % (Kp >> 3)), cb = (int)(rest / (Kp >> 3));
    const int j = rw / kDCh, ch = cb * kDCh + rw % kDCh, col = cg * 8 + c8;
    float w = 0.f;
    if (ch < C && col < N) {
        const int m = j * C + ch;
        w = __ldg(W + (int64_t)m * N + col) * __ldg(gain + m);
    }
    Wb[idx] = __float2bfloat16_rn(w);
}

// ---- host side -------------------------------------------------------------------------------------
template <int MT>
static bool launch_g_t(const TailPlan& p, const CUtensorMap& tmx, const void* ehi, const void* elo, int64_t T, int nC,
                       float* Gpart, int* status, cudaStream_t s) {
    const int stage_bytes = MT * 2 * kGXBox + 2 * (p.Kp >> 3) * (kGTok * 16);
    const int smem = kGStages * stage_bytes + (int)sizeof(GCtl) + 1024;
    int tmem_cols = 32;
    while (tmem_cols < MT * p.Kp) tmem_cols *= 2;
    cudaFuncSetAttribute(tail_g_tc_k<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    dim3 grid(p.g_groups, p.g_splits);
    // e_hi / e_lo as [granule x column group][16 groups of 8 tokens][8 tokens x 8 columns]: a box takes half a granule's
    // rows (64 tokens) of all column groups
    const uint64_t erows = (uint64_t)((T + kEGranule - 1) / kEGranule) * (uint64_t)(p.Kp >> 3);
    CUtensorMap tmeh, tmel;
    if (!make_tensor_map_3d(&tmeh, ehi, 64, 16, erows, 64, 1024, 64, 8, (uint32_t)(p.Kp >> 3), 0)) return false;
    if (!make_tensor_map_3d(&tmel, elo, 64, 16, erows, 64, 1024, 64, 8, (uint32_t)(p.Kp >> 3), 0)) return false;
    tail_g_tc_k<MT><<<grid, 192, smem, s>>>(tmx, tmeh, tmel, T,
                                            p.g_tok_per_split, nC, p.Kp, tmem_cols, Gpart, status);
    return true;
}

// G partials of every token range -> Gpart[g_splits][nC][Kp].  False when no tensor map could be made.
bool launch_tail_g_tc(const mhclite_ctx* c, int64_t T, const TailPlan& p, const void* x, const void* ehi,
                      const void* elo, float* Gpart, int* status, cudaStream_t s) {
    const int nC = c->n * c->C;
    CUtensorMap tmx;
    if (!make_tensor_map_2d(&tmx, x, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, 64, kGTok, 128)) return false;
    bool ok;
    switch (p.g_mt) {
        case 1: ok = launch_g_t<1>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
        case 2: ok = launch_g_t<2>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
        default: ok = launch_g_t<3>(p, tmx, ehi, elo, T, nC, Gpart, status, s); break;
    }
    if (ok) c->launches += 1;
    return ok;
}

size_t tail_wb_bytes(int n, int C, int Kp) { return (size_t)n * ((C + kDCh - 1) / kDCh) * Kp * kDCh * 2; }

template <int N_>
static void launch_dx_t(int grid, int smem, const CUtensorMap& tmx, const CUtensorMap& tmg, const CUtensorMap& tmdu,
                        const CUtensorMap& tmdx, const DxArgs& a, int mode, cudaStream_t s) {
#define MHCL_DX(M)                                                                                           \
    do {                                                                                                     \
        cudaFuncSetAttribute(tail_dx_tc_k<N_, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);        \
        tail_dx_tc_k<N_, M><<<grid, kDThreads, smem, s>>>(tmx, tmg, tmdu, tmdx, a);                          \
    } while (0)
    if (mode == 1) MHCL_DX(1);
    else if (mode == 2) MHCL_DX(2);
    else MHCL_DX(0);
#undef MHCL_DX
}

// dx of the projection / RMSNorm backward, fused with H_res^T g + H_pre du when g is given.  Packs W' first.
// False (nothing launched) when the shape does not fit shared memory or no tensor map could be made.
bool launch_tail_dx_tc(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                       const void* du, const void* ehi, const float* kappa, const float* H_res, const float* H_pre,
                       const float* W, const float* gain, void* Wb, void* dx, int acc_dx, int* status, cudaStream_t s) {
    const int n = c->n, C = c->C;
    const int mode = g != nullptr ? 1 : (acc_dx ? 2 : 0);
    const int boxes = mode == 1 ? 2 * n + 1 : (mode == 2 ? 2 * n : n);
    const int e_bytes = p.Kp * kDTok * 2;
    const int fixed = e_bytes + kDWSlots * n * kDCh * 32 + (int)sizeof(DCtl) + 1024;
    int dslots = (227 * 1024 - fixed) / (boxes * kDBox);
    if (dslots > kDMaxSlots) dslots = kDMaxSlots;
    if (dslots < 4) return false;
    const int smem = fixed + dslots * boxes * kDBox;
    if (n * kDCh > 256 || T > (int64_t)0x7fffffff - kDTok) return false;   // one instruction's N; 32-bit TMA coordinates
    // [token][stream][channel] maps with boxes of 32 tokens x 1 stream x 32 channels
    CUtensorMap tmx, tmg, tmdu, tmdx;
    if (!make_tensor_map_3d(&tmx, x, (uint64_t)C, (uint64_t)n, (uint64_t)T, (uint64_t)C, (uint64_t)n * C, kDCh, 1, 32, 64)) return false;
    if (!make_tensor_map_3d(&tmdx, dx, (uint64_t)C, (uint64_t)n, (uint64_t)T, (uint64_t)C, (uint64_t)n * C, kDCh, 1, 32, 64)) return false;
    tmg = mode == 2 ? tmdx : tmx; tmdu = tmx;
    if (mode == 1) {
        if (!make_tensor_map_3d(&tmg, g, (uint64_t)C, (uint64_t)n, (uint64_t)T, (uint64_t)C, (uint64_t)n * C, kDCh, 1, 32, 64)) return false;
        if (!make_tensor_map_3d(&tmdu, du, (uint64_t)C, 1, (uint64_t)T, (uint64_t)C, (uint64_t)C, kDCh, 1, 32, 64)) return false;
    }
    DxArgs a;
    a.T = T; a.C = C; a.Kp = p.Kp; a.ncb = (C + kDCh - 1) / kDCh;
    a.items = ((T + kDTok - 1) / kDTok) * a.ncb;
    int grid = c->sm_count;
    if ((int64_t)grid > a.items) grid = (int)a.items;
    if (grid < 1) return false;
    a.per_cta = (a.items + grid - 1) / grid;
    grid = (int)((a.items + a.per_cta - 1) / a.per_cta);
    a.ring = 512 / (n * kDCh) >= kDMaxRing ? kDMaxRing : 2;
    a.dslots = dslots;
    a.tmem_cols = 32;
    while (a.tmem_cols < a.ring * n * kDCh) a.tmem_cols *= 2;
    a.ehi = (const __nv_bfloat16*)ehi; a.Wb = (const __nv_bfloat16*)Wb;
    a.kappa = kappa; a.H_res = H_res; a.H_pre = H_pre; a.status = status;
    c->launches += 2;
    const int64_t total = (int64_t)n * a.ncb * p.Kp * kDCh;
    pack_wb_k<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(n, C, N, p.Kp, a.ncb, W, gain, (__nv_bfloat16*)Wb);
    KernelTimer timer_(c, MHCLITE_KERNEL_TAIL_DX, s);
    MHCL_DISPATCH_N(n, (launch_dx_t<N_>(grid, smem, tmx, tmg, tmdu, tmdx, a, mode, s)));
    return true;
}

}  // namespace mhcl
