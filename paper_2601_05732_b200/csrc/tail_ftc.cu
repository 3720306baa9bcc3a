// Blackwell tensor-core backward tail for narrow projections (n <= 4: at most 32 columns): the projection /
// RMSNorm backward of paper Eq. (4) fused with the gradient of Eq. (1), one pass over x, g and du.
//
//   dxhat[t,m] = sum_c e[t,c] W'[m,c] - x[t,m] kappa_t            (W' = diag(gain) W, e = rstd alpha (.) dz)
//   dx[t,j,c]  = sum_i H_res[t,i,j] g[t,i,c] + H_pre[t,j] du[t,c] + dxhat[t,j*C+c]
//   G[m,c]     = sum_t x[t,m] e[t,c]                              (dW = gain (.) G, dgain = sum_c W G)
//
// A CTA owns a slice of 64 channels of all n streams and walks over a range of 128-token tiles.
//   * x, g and du arrive by TMA (128-byte swizzle) per 32-token quadrant into five slots: one per lane
//     quadrant of the tensor memory plus one that goes round, so that the load of a quadrant's next tile is
//     under way while the quadrant still works on its current one (load number l goes to slot l mod 5).  The
//     tiled e buffers (hi, lo) of a tile arrive as two bulk copies; the CTA's rows of W' stay in shared memory.
//   * One thread issues tcgen05.mma: dxhat of a tile half (M = 128 tokens, N = n x 32 channels, K = Kp) into a
//     ring of tensor-memory buffers, and per arrived quadrant G += x^T e (M = 128 rows of the slice, N = Kp,
//     K = 32 tokens, x as the MN-major operand straight from its slot, e as hi | lo side by side in N) into
//     accumulators that stay in tensor memory over the whole token range.
//   * Eight epilogue warps (thread = token, two warps per quadrant) combine dxhat with x, g, du and the
//     token's H_res, H_pre and kappa, write dx over the g boxes of the slot (a thread has read all of g at
//     its position before it writes there), and one thread per quadrant sends the boxes to global memory
//     with a TMA store before it hands the slot back.
//   * At the end the G accumulators go to this token range's partial (no atomics).
// Every mbarrier wait is bounded; on a time-out the CTA raises its abort flag, records MHCLITE_ERR_TIMEOUT in
// the status word, lets copies in flight land, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"
#include "tc.cuh"

namespace mhcl {

constexpr int kFTok = 128;                      // tokens per tile (UMMA M)
constexpr int kFCs = 64;                        // channels per slice = one 128-byte swizzle row
constexpr int kFBox = 32 * 128;                 // one TMA box: 32 tokens x 64 channels of bf16
constexpr int kFEpiWarps = 8;
constexpr int kFThreads = 96 + 32 * kFEpiWarps; // operand producer, MMA issuer, data producer, epilogue
constexpr int kFMaxRing = 3;
constexpr int kFSlots = 5;                      // data slots: one per lane quadrant plus one that goes round
constexpr int kFMaxSplits = 64;                 // most token ranges per slice (bounds the G partials)

struct FCtl {
    uint64_t w_full, e_full[2], e_empty[2], elo_full, elo_empty, d_full[4][2], g_done[4][2], q_done[4],
        s_free[kFSlots], acc_full[kFMaxRing],
        acc_empty[kFMaxRing], g_final;
    uint32_t tmem_base;
    int abort[3];
};

struct FArgs {
    int64_t T;
    int C, Kp;
    int ntiles, splits;             // 128-token tiles in all, token ranges (grid y)
    int ring, tmem_cols;            // dxhat buffers in tensor memory, columns allocated
    const __nv_bfloat16 *ehi, *elo; // tiled (see e_tiled_index)
    const __nv_bfloat16* Wf;        // [slice][half][Kp/8][n][32][8]
    const float *kappa, *H_res, *H_pre;
    float* Gpart;                   // [splits][nC][Kp]
    int* status;
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
}
// Asks the L2 cache for a box ahead of the TMA load that will bring it to shared memory.
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void ftc_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}
__device__ __forceinline__ void ftc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Ties the registers of an earlier tcgen05.ld to a point after the wait, so that no use is scheduled before it.
__device__ __forceinline__ void ftc_settle(uint32_t (&r)[8]) {
    asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]) :: "memory");
}

// MODE 0: dx = dxhat (x only);  1: fused with H_res^T g + H_pre du;  2: dx += dxhat (x and the old dx).
template <int N_, int MODE>
__global__ void __launch_bounds__(kFThreads, 1)
tail_ftc_k(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmg,
           const __grid_constant__ CUtensorMap tmdu, const __grid_constant__ CUtensorMap tmdx, const FArgs a) {
    constexpr int kBoxes = MODE == 1 ? 2 * N_ + 1 : (MODE == 2 ? 2 * N_ : N_);
    constexpr int kSlot = kBoxes * kFBox;
    constexpr int kOut = MODE == 0 ? 0 : N_;                   // first of the boxes that dx is written over
    constexpr int kNA = (N_ + 1) / 2;                          // G accumulators: 128 rows = two streams' 64 channels
    constexpr int kDW = N_ * 32;                               // tensor-memory columns of one dxhat buffer
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int e_bytes = a.Kp * kFTok * 2;                      // one of hi / lo of a tile; a multiple of 4096
    const int w_bytes = a.Kp * N_ * kFCs * 2;
    unsigned char* slots = smem;
    unsigned char* e_s = slots + kFSlots * kSlot;              // e_hi of even tiles | e_hi of odd tiles | e_lo
    unsigned char* w_s = e_s + 3 * e_bytes;
    FCtl* ctl = reinterpret_cast<FCtl*>(w_s + ((w_bytes + 1023) & ~1023));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c0 = blockIdx.x * kFCs;
    // Token range blockIdx.y takes the tiles ntiles - 1 - (blockIdx.y + splits * ti), ti = 0, 1, ...: all ranges walk
    // down the token axis together, starting where the kernel before this one (it read x and du in ascending
    // order) left its last lines in the L2 cache.
    const int nt = (a.ntiles - (int)blockIdx.y + a.splits - 1) / a.splits;
    auto tile_of = [&](int ti) { return a.ntiles - 1 - ((int)blockIdx.y + a.splits * ti); };
    volatile int* abort = ctl->abort;

    if (tid == 0) {
        mbar_init(smem_u32(&ctl->w_full), 1);
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->e_full[s]), 1); mbar_init(smem_u32(&ctl->e_empty[s]), 1); }
        mbar_init(smem_u32(&ctl->elo_full), 1); mbar_init(smem_u32(&ctl->elo_empty), 1);
        for (int s = 0; s < kFSlots; ++s) mbar_init(smem_u32(&ctl->s_free[s]), 1);
        for (int s = 0; s < 4; ++s) {
            for (int b2 = 0; b2 < 2; ++b2) { mbar_init(smem_u32(&ctl->d_full[s][b2]), 1); mbar_init(smem_u32(&ctl->g_done[s][b2]), 1); }
            mbar_init(smem_u32(&ctl->q_done[s]), 2);
        }
        for (int s = 0; s < kFMaxRing; ++s) { mbar_init(smem_u32(&ctl->acc_full[s]), 1); mbar_init(smem_u32(&ctl->acc_empty[s]), kFEpiWarps); }
        mbar_init(smem_u32(&ctl->g_final), 1);
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
    const uint32_t tmem_g = tmem;                              // kNA accumulators of 2 Kp columns (hi | lo parts)
    const uint32_t tmem_d = tmem + kNA * 2 * a.Kp;             // ring of dxhat buffers

    if (warp == 0) {
        // ---- producer of the MMA operands: W' rows of the slice once, then the e tiles ------------------
        if (lane == 0 && nt > 0) {
            mbar_expect_tx(smem_u32(&ctl->w_full), w_bytes);
            bulk_load(smem_u32(w_s), a.Wf + (int64_t)blockIdx.x * (w_bytes / 2), w_bytes, smem_u32(&ctl->w_full));
            for (int ti = 0; ti < nt; ++ti) {
                const int buf = ti & 1;
                // e_hi (dxhat and G) is double-buffered, e_lo (G only) is not: shared memory goes to the data slots
                if (!mbar_wait(smem_u32(&ctl->e_empty[buf]), ((ti >> 1) & 1) ^ 1, abort, 1, ti)) break;
                const int64_t off = (int64_t)tile_of(ti) * a.Kp * kFTok;             // elements
                mbar_expect_tx(smem_u32(&ctl->e_full[buf]), e_bytes);
                bulk_load(smem_u32(e_s + buf * e_bytes), a.ehi + off, e_bytes, smem_u32(&ctl->e_full[buf]));
                if (!mbar_wait(smem_u32(&ctl->elo_empty), (ti & 1) ^ 1, abort, 12, ti)) break;
                mbar_expect_tx(smem_u32(&ctl->elo_full), e_bytes);
                bulk_load(smem_u32(e_s + 2 * e_bytes), a.elo + off, e_bytes, smem_u32(&ctl->elo_full));
            }
        }
    } else if (warp == 2) {
        // ---- producer of the data: x (and g, du, or the old dx) per 32-token quadrant.  Lane b issues the
        //      loads of box b (issuing a TMA instruction keeps a thread busy for ~100 cycles: nine in a row
        //      from one thread would delay the slots behind it), lane 0 arms the barrier.
        {
            const int b = lane < kBoxes ? lane : 0;
            const CUtensorMap* mp = b < N_ ? &tmx : (b < 2 * N_ ? &tmg : &tmdu);
            if (MODE == 2 && b >= N_) mp = &tmg;
            const int col = (b < N_ ? b * a.C : (b < 2 * N_ ? (b - N_) * a.C : 0)) + c0;
            bool ok = true;
            for (int ti = 0; ti < nt && ok; ++ti) {
                for (int q = 0; q < 4 && ok; ++q) {
                    // load number li goes to slot li % kFSlots: the slot that quadrant q - 1 hands back, so that the
                    // load of a quadrant's next tile is on its way while the quadrant still works on this one
                    const int li = ti * 4 + q, sl = li % kFSlots;
                    if (lane == 0) ok = mbar_wait(smem_u32(&ctl->s_free[sl]), ((li / kFSlots) & 1) ^ 1, abort, 2, li);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctl->d_full[q][ti & 1]);
                    if (lane == 0) mbar_expect_tx(full, kSlot);
                    __syncwarp();
                    const int row = tile_of(ti) * kFTok + q * 32;
                    const int next_row = tile_of(ti + 1) * kFTok + q * 32;
                    if (lane < kBoxes) {
                        tma_load_2d(smem_u32(slots + sl * kSlot) + b * kFBox, mp, full, col, row);
                        // the quadrant's next boxes start their way from HBM to L2 now: a slot is busy for a
                        // whole load + compute + store round, too long to hide the HBM latency with so few slots
                        // (every other tile only: the tensor maps promote L2 fills to 256 bytes, so the neighbouring
                        //  slice's CTA, which walks the same tiles at the same time, brings this slice's lines along
                        //  on the tiles in between; a prefetch costs the TMA unit as much as the load itself)
                        if (ti + 1 < nt && (((ti + (int)blockIdx.x) & 1) == 0)) tma_prefetch_2d(mp, col, next_row);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------------------
        if (lane == 0 && nt > 0) {
            const uint32_t idesc_d = umma_idesc_mn(128, kDW, 0, 0);
            const uint32_t idesc_g = umma_idesc_mn(128, a.Kp, 1, 1);
            const int ksteps = a.Kp >> 4;
            const uint32_t w_half = (uint32_t)(a.Kp >> 3) * (kDW * 16);          // bytes of one channel half of W'
            bool ok = mbar_wait(smem_u32(&ctl->w_full), 0, abort, 3, 0);
            bool g_started = false;
            for (int ti = 0; ti < nt && ok; ++ti) {
                const int buf = ti & 1;
                ok = mbar_wait(smem_u32(&ctl->e_full[buf]), (ti >> 1) & 1, abort, 4, ti);
                if (!ok) break;
                const uint32_t eh = smem_u32(e_s + buf * e_bytes), el = smem_u32(e_s + 2 * e_bytes);
                bool lo_ready = false;
                for (int half = 0; half < 2 && ok; ++half) {
                    const int u = 2 * ti + half, rr = u % a.ring;
                    ok = mbar_wait(smem_u32(&ctl->acc_empty[rr]), ((u / a.ring) & 1) ^ 1, abort, 5, u);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t wa = smem_u32(w_s) + half * w_half;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        // A: tokens x columns, K-major, no swizzle: column groups 2 KB apart, 8-token groups 128 B apart
                        // B: channels x columns, K-major, no swizzle: column groups kDW * 16 B apart, 8-channel groups 128 B apart
                        tc_mma(tmem_d + rr * kDW, smem_desc(eh + ks * 4096, 2048, 128, 0),
                               smem_desc(wa + ks * 2 * (kDW * 16), kDW * 16, 128, 0), idesc_d, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&ctl->acc_full[rr]));
                }
                // G += x^T e per quadrant, in the order in which the quadrants' data arrive
                uint32_t pending = 0xFu;
                for (uint32_t polls = 0; pending && ok; ++polls) {
                    if (polls > kWaitLimit || abort[0]) {
                        if (abort[0] == 0) { abort[1] = 6; abort[2] = ti; }
                        abort[0] = 1;
                        ok = false;
                        break;
                    }
                    for (int q = 0; q < 4; ++q) {
                        if (!(pending & (1u << q)) || !mbar_try_wait(smem_u32(&ctl->d_full[q][ti & 1]), (ti >> 1) & 1)) continue;
                        if (!lo_ready) {
                            ok = mbar_wait(smem_u32(&ctl->elo_full), ti & 1, abort, 13, ti);
                            if (!ok) break;
                            lo_ready = true;
                        }
                        pending &= ~(1u << q);
                        tc_fence_after();
                        const uint32_t xs = smem_u32(slots + ((ti * 4 + q) % kFSlots) * kSlot);
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks) {
                            // B: columns of e_hi, of e_lo = N (8-column groups 2 KB apart), tokens = K (8-token groups
                            // 128 B apart); the two products go to the two halves of the accumulator's columns
                            const uint32_t eo = (uint32_t)(q * 32 + ks * 16) * 16;
                            const uint64_t bh = smem_desc(eh + eo, 128, 2048, 0), bl = smem_desc(el + eo, 128, 2048, 0);
#pragma unroll
                            for (int ac = 0; ac < kNA; ++ac) {
                                // A: 128 rows = the 64 channels of two streams (boxes 4 KB apart), 8-token groups 1 KB apart
                                const uint64_t ad = smem_desc(xs + ac * 2 * kFBox + ks * 2048, kFBox, 1024, 2);
                                tc_mma(tmem_g + ac * 2 * a.Kp, ad, bh, idesc_g, g_started ? 1u : 0u);
                                tc_mma(tmem_g + ac * 2 * a.Kp + a.Kp, ad, bl, idesc_g, g_started ? 1u : 0u);
                            }
                            g_started = true;
                        }
                        tc_commit(smem_u32(&ctl->g_done[q][ti & 1]));
                    }
                }
                if (!ok) break;
                tc_commit(smem_u32(&ctl->e_empty[buf]));
                tc_commit(smem_u32(&ctl->elo_empty));
            }
            if (ok) tc_commit(smem_u32(&ctl->g_final));
        }
    } else {
        // ---- epilogue: thread = token; the two warps of a lane quadrant take 16 channels of each half ----
        const int quad = warp & 3;
        const int hw = (warp - 3) >> 2;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        // the token's coefficients, each twice in a 64-bit register for the packed FMAs (fma.rn.f32x2)
        uint64_t nkap2 = 0, hp2[N_], hr2[N_][N_];
        bool ok = true;
        for (int ti = 0; ti < nt; ++ti) {
            const int64_t row0 = (int64_t)tile_of(ti) * kFTok + quad * 32;
            const int64_t t = row0 + lane;
            const bool live = t < a.T;
            {
                const float kap = live ? -__ldg(a.kappa + t) : 0.f;
                nkap2 = pack2f(kap, kap);
            }
            if (MODE == 1) {
#pragma unroll
                for (int j = 0; j < N_; ++j) { const float h = live ? __ldg(a.H_pre + t * N_ + j) : 0.f; hp2[j] = pack2f(h, h); }
#pragma unroll
                for (int i = 0; i < N_; ++i)
#pragma unroll
                    for (int j = 0; j < N_; ++j) {
                        const float h = live ? __ldg(a.H_res + t * N_ * N_ + i * N_ + j) : 0.f;
                        hr2[i][j] = pack2f(h, h);
                    }
            }
            const uint32_t slot = smem_u32(slots + ((ti * 4 + quad) % kFSlots) * kSlot);
            ok = mbar_wait(smem_u32(&ctl->d_full[quad][ti & 1]), (ti >> 1) & 1, abort, 7, ti);
            // MODE 0 writes dx over x itself: the G MMAs must have read the boxes
            if (MODE == 0 && ok) ok = mbar_wait(smem_u32(&ctl->g_done[quad][ti & 1]), (ti >> 1) & 1, abort, 8, ti);
            for (int half = 0; half < 2; ++half) {
                const int u = 2 * ti + half, rr = u % a.ring;
                if (ok) ok = mbar_wait(smem_u32(&ctl->acc_full[rr]), (u / a.ring) & 1, abort, 9, u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t tbase = tmem_d + lane_base + rr * kDW;
#pragma unroll
                for (int pp = 0; pp < 2; ++pp) {
                    const int pcl = hw * 2 + pp;                       // 8-channel group within the half
                    const int pc = half * 4 + pcl;                     // 16-byte piece within the 128-byte row
                    const int po = lane * 128 + ((pc ^ (lane & 7)) << 4);
                    uint32_t acc[N_][8];
#pragma unroll
                    for (int j = 0; j < N_; ++j) ftc_ld8(tbase + j * 32 + pcl * 8, acc[j]);
                    uint64_t gf[MODE == 1 ? N_ : 1][4], df[4];
                    if (MODE == 1) {
#pragma unroll
                        for (int i = 0; i < N_; ++i) unpack8x2(lds128(slot + (N_ + i) * kFBox + po), gf[i]);
                        unpack8x2(lds128(slot + 2 * N_ * kFBox + po), df);
                    }
                    ftc_ld_wait();
#pragma unroll
                    for (int j = 0; j < N_; ++j) ftc_settle(acc[j]);
#pragma unroll
                    for (int j = 0; j < N_; ++j) {
                        uint64_t xf[4], o[4];
                        unpack8x2(lds128(slot + j * kFBox + po), xf);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            o[k] = fma2(xf[k], nkap2, pack2f(__uint_as_float(acc[j][2 * k]), __uint_as_float(acc[j][2 * k + 1])));
                        if (MODE == 1) {
#pragma unroll
                            for (int k = 0; k < 4; ++k) o[k] = fma2(hp2[j], df[k], o[k]);
#pragma unroll
                            for (int i = 0; i < N_; ++i)
#pragma unroll
                                for (int k = 0; k < 4; ++k) o[k] = fma2(hr2[i][j], gf[i][k], o[k]);
                        }
                        if (MODE == 2) {
                            uint64_t old[4];
                            unpack8x2(lds128(slot + (N_ + j) * kFBox + po), old);
#pragma unroll
                            for (int k = 0; k < 4; ++k) o[k] = fma2(old[k], pack2f(1.f, 1.f), o[k]);
                        }
                        // dx takes the place of g (of the old dx; of x itself in MODE 0) in the slot
                        sts128(slot + (kOut + j) * kFBox + po, pack8x2(o));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[rr]));
            }
            if (!ok) break;
            // the slot now holds dx: make the writes visible to the TMA unit, then one thread stores the boxes
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctl->q_done[quad]));
            }
            if (hw == 0) {
                // lane j stores box j once both warps of the quadrant have written their part
                bool oks = lane >= N_ || mbar_wait(smem_u32(&ctl->q_done[quad]), ti & 1, abort, 10, ti);
                if (oks && lane < N_ && row0 < a.T) {
                    tma_store_2d(&tmdx, slot + (kOut + lane) * kFBox, lane * a.C + c0, (int)row0);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                // the slot goes back once the G MMAs have read its x boxes as well (long done by now)
                if (MODE != 0 && lane == 0 && oks) oks = mbar_wait(smem_u32(&ctl->g_done[quad][ti & 1]), (ti >> 1) & 1, abort, 8, ti);
                oks = __all_sync(0xffffffffu, oks);
                if (oks && lane == 0) mbar_arrive(smem_u32(&ctl->s_free[(ti * 4 + quad) % kFSlots]));
            }
            __syncwarp();
        }
        if (hw == 0 && lane < N_) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        // ---- G of this token range -> its partial -----------------------------------------------------
        if (nt > 0) {
            if (ok) ok = mbar_wait(smem_u32(&ctl->g_final), 0, abort, 11, 0);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                float* Gp = a.Gpart + (int64_t)blockIdx.y * (N_ * a.C) * a.Kp;
                for (int ac = hw; ac < kNA; ac += 2) {
                    const int j = 2 * ac + (quad >> 1);
                    const int ch = c0 + (quad & 1) * 32 + lane;
                    for (int cc = 0; cc < a.Kp; cc += 16) {
                        float v[16], lo[16];
                        tc_ld16(tmem_g + lane_base + ac * 2 * a.Kp + cc, v);
                        tc_ld16(tmem_g + lane_base + ac * 2 * a.Kp + a.Kp + cc, lo);
#pragma unroll
                        for (int e = 0; e < 16; ++e) v[e] += lo[e];
                        if (j < N_) {
                            float* rowp = Gp + ((int64_t)j * a.C + ch) * a.Kp + cc;
#pragma unroll
                            for (int e = 0; e < 16; e += 4)
                                *reinterpret_cast<float4*>(rowp + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ctl->abort[0]) report_abort(abort, a.status, 4);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(a.tmem_cols) : "memory");
    }
}

// W' = diag(gain) W in bf16 as the B operand of tail_ftc_k: per slice of 64 channels and per half of it a
// block [Kp/8 column groups][n streams][32 channels][8 columns]; zero beyond the N columns.  The same launch
// clears the accumulators db[N] and dalpha[3] when they are given (the backward's kernels add into them).
__global__ void __launch_bounds__(256) pack_wf_k(int n, int C, int N, int Kp, const float* __restrict__ W,
                                                 const float* __restrict__ gain, __nv_bfloat16* __restrict__ Wf,
                                                 float* zero_db, float* zero_dalpha) {
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (zero_db && idx < N) zero_db[idx] = 0.f;
    if (zero_dalpha && idx < 3) zero_dalpha[idx] = 0.f;
    const int64_t total = (int64_t)n * C * Kp;
    if (idx >= total) return;
    const int c8 = (int)(idx & 7), chl = (int)((idx >> 3) & 31);
    int64_t rest = idx >> 8;
    const int j = (int)(rest % n); rest /= n;
    const int cg = (int)(rest % (Kp >> 3)); rest /= (Kp >> 3);
    const int half = (int)(rest & 1);
    const int slice = (int)(rest >> 1);
    const int ch = slice * kFCs + half * 32 + chl, col = cg * 8 + c8;
    float w = 0.f;
    if (col < N) {
        const int m = j * C + ch;
        w = __ldg(W + (int64_t)m * N + col) * __ldg(gain + m);
    }
    Wf[idx] = __float2bfloat16_rn(w);
}

// ---- host side -------------------------------------------------------------------------------------
static int ftc_smem_bytes(int n, int Kp, int mode) {
    const int boxes = mode == 1 ? 2 * n + 1 : (mode == 2 ? 2 * n : n);
    const int w_bytes = Kp * n * kFCs * 2;
    return kFSlots * boxes * kFBox + 3 * (Kp * kFTok * 2) + ((w_bytes + 1023) & ~1023) + (int)sizeof(FCtl) + 1024;
}

// Fills the plan's fields of this kernel: usable when the slices are whole (C a multiple of 64), the G
// accumulators (hi | lo parts) and two dxhat buffers fit the 512 columns of tensor memory, and the slots fit
// shared memory.
void plan_tail_ftc(int n, int C, int64_t T, int sm_count, TailPlan* p) {
    const int na = (n + 1) / 2;
    p->ftc = p->supported && (C % kFCs) == 0 && na * 2 * p->Kp + 2 * n * 32 <= 512 && ftc_smem_bytes(n, p->Kp, 1) <= 227 * 1024;
    p->f_slices = C / kFCs;
    const int64_t ntiles = (T + kFTok - 1) / kFTok;
    // Token ranges per slice.  One CTA fits an SM, so slices x ranges CTAs run in ceil(slices * ranges / SMs)
    // rounds of ceil(ntiles / ranges) tiles each (plus about two tiles' worth of start-up and G write-out per
    // CTA): take the count with the shortest total.  Several rounds of short CTAs beat one round that leaves SMs
    // idle (64 slices: 2 ranges use 128 of 148 SMs, 16 ranges run 6.9 rounds' worth of work in 7).
    int64_t best = 1, best_cost = INT64_MAX;
    const int64_t rmax = ntiles < kFMaxSplits ? ntiles : kFMaxSplits;
    for (int64_t r = 1; r <= rmax && p->f_slices > 0; ++r) {
        const int64_t rounds = (p->f_slices * r + sm_count - 1) / sm_count;
        const int64_t cost = rounds * ((ntiles + r - 1) / r + 2);
        if (cost < best_cost) { best_cost = cost; best = r; }
    }
    p->f_splits = (int)best;
    int ring = (512 - na * 2 * p->Kp) / (n * 32);
    p->f_ring = ring > kFMaxRing ? kFMaxRing : ring;
}

template <int N_>
static void launch_ftc_t(dim3 grid, int smem, const CUtensorMap& tmx, const CUtensorMap& tmg, const CUtensorMap& tmdu,
                         const CUtensorMap& tmdx, const FArgs& a, int mode, cudaStream_t s) {
#define MHCL_FTC(M)                                                                                      \
    do {                                                                                                 \
        cudaFuncSetAttribute(tail_ftc_k<N_, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);      \
        tail_ftc_k<N_, M><<<grid, kFThreads, smem, s>>>(tmx, tmg, tmdu, tmdx, a);                         \
    } while (0)
    if (mode == 1) MHCL_FTC(1);
    else if (mode == 2) MHCL_FTC(2);
    else MHCL_FTC(0);
#undef MHCL_FTC
}

// First launch of a backward whose tail is tail_ftc_k: packs W' and clears db / dalpha (null: left alone) in one
// kernel.  False (nothing launched) when that tail is not available for the plan.
bool launch_tail_ftc_prep(const mhclite_ctx* c, int N, const TailPlan& p, const float* W, const float* gain, void* Wf,
                          float* zero_db, float* zero_dalpha, cudaStream_t s) {
    if (c->n > 4 || !p.ftc || !tensor_maps_available()) return false;
    c->launches += 1;
    const int64_t total = (int64_t)c->n * c->C * p.Kp;
    pack_wf_k<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(c->n, c->C, N, p.Kp, W, gain, (__nv_bfloat16*)Wf, zero_db,
                                                              zero_dalpha);
    return true;
}

// dx and the G partials [f_splits][nC][Kp] in one pass; packs W' first unless launch_tail_ftc_prep has done so.
// False (nothing launched) when no tensor map could be made.
bool launch_tail_ftc(const mhclite_ctx* c, int64_t T, int N, const TailPlan& p, const void* x, const void* g,
                     const void* du, const void* ehi, const void* elo, const float* kappa, const float* H_res,
                     const float* H_pre, const float* W, const float* gain, void* Wf, bool wf_packed, void* dx,
                     int acc_dx, float* Gpart, int* status, cudaStream_t s) {
    const int n = c->n, C = c->C, nC = n * C;
    if (n > 4 || !p.ftc) return false;
    const int mode = g ? 1 : (acc_dx ? 2 : 0);
    CUtensorMap tmx, tmg, tmdu, tmdx;
    if (!make_tensor_map_2d(&tmx, x, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, kFCs, 32, 128)) return false;
    if (!make_tensor_map_2d(&tmdx, dx, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, kFCs, 32, 128)) return false;
    tmg = mode == 2 ? tmdx : tmx; tmdu = tmx;
    if (mode == 1) {
        if (!make_tensor_map_2d(&tmg, g, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, kFCs, 32, 128)) return false;
        if (!make_tensor_map_2d(&tmdu, du, (uint64_t)C, (uint64_t)T, (uint64_t)C, kFCs, 32, 128)) return false;
    }
    FArgs a;
    a.T = T; a.C = C; a.Kp = p.Kp;
    a.ntiles = (int)((T + kFTok - 1) / kFTok); a.splits = p.f_splits; a.ring = p.f_ring;
    const int smem = ftc_smem_bytes(n, p.Kp, mode);
    const int cols = ((n + 1) / 2) * 2 * p.Kp + a.ring * n * 32;
    a.tmem_cols = 32;
    while (a.tmem_cols < cols) a.tmem_cols *= 2;
    if (2 * smem <= 227 * 1024 && a.tmem_cols > 256) {        // two CTAs may share an SM: halve the claim
        a.ring = 2;
        a.tmem_cols = 256;
        if (((n + 1) / 2) * 2 * p.Kp + 2 * n * 32 > 256) return false;
    }
    a.ehi = (const __nv_bfloat16*)ehi; a.elo = (const __nv_bfloat16*)elo; a.Wf = (const __nv_bfloat16*)Wf;
    a.kappa = kappa; a.H_res = H_res; a.H_pre = H_pre; a.Gpart = Gpart; a.status = status;
    c->launches += 1;
    if (!wf_packed) {
        c->launches += 1;
        const int64_t total = (int64_t)nC * p.Kp;
        pack_wf_k<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(n, C, N, p.Kp, W, gain, (__nv_bfloat16*)Wf, nullptr,
                                                                  nullptr);
    }
    KernelTimer timer_(c, MHCLITE_KERNEL_TAIL_DX, s);
    dim3 grid(p.f_slices, p.f_splits);
    switch (n) {
        case 2: launch_ftc_t<2>(grid, smem, tmx, tmg, tmdu, tmdx, a, mode, s); break;
        case 3: launch_ftc_t<3>(grid, smem, tmx, tmg, tmdu, tmdx, a, mode, s); break;
        default: launch_ftc_t<4>(grid, smem, tmx, tmg, tmdu, tmdx, a, mode, s); break;
    }
    return true;
}

}  // namespace mhcl
