// Blackwell-native forward projection of paper Eq. (4): q = x W' (W' = diag(gain) W) and the RMSNorm sum of
// squares, in one pass over x, on the 5th-generation tensor cores.
//
//   TMA (cp.async.bulk.tensor, 128-byte swizzle) streams x tiles [128 tokens x 64 k] and W' tiles
//   [2 Nq x 64 k] into a shared-memory ring; one thread issues tcgen05.mma (M = 128 tokens, N = 2 Nq,
//   K = 16 per instruction) with the fp32 accumulator [128 x 2 Nq] in tensor memory; the bf16 pair
//   hi | lo of W' sits side by side in N, so x is read from shared memory once per k-step and the two
//   partial products are added in the epilogue.  When 2 Nq exceeds the 256 columns of one instruction
//   (n = 5: 130 columns) the hi and lo halves run as two instructions of N = Nq that accumulate into the
//   same [128 x Nq] accumulator.  Four warps read the same x tiles from shared memory for
//   the sum of squares, then fetch the accumulator with tcgen05.ld (thread = token) and store the K slice's
//   partial result.  The tensor work is a small fraction of the time the bytes take to arrive: the
//   kernel is bound by HBM.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (owns the tensor-memory
// allocation), warps 2..5 = sum of squares + epilogue (TMEM lane quadrant = warp % 4).
// Every wait on an mbarrier is bounded: when the bound is hit the CTA raises an abort flag, records a status
// word in global memory, lets in-flight copies land, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.h"
#include "mma.cuh"
#include "tc.cuh"

namespace mhcl {

constexpr int kTcTok = 128;                 // tokens per CTA = UMMA M
constexpr int kTcK = 64;                    // k per stage = one 128-byte swizzle row of bf16
constexpr int kTcXBytes = kTcTok * kTcK * 2;

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) with the 128-byte
// swizzle: 8-row groups 1024 bytes apart; descriptor version 1 (Blackwell), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);          // start address
    d |= (uint64_t)1 << 16;                          // leading byte offset (16 B units; fixed for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version
    d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
    return d;
}
// Instruction descriptor: D f32, A and B bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTcTok >> 4) << 24);
}

struct TcSmem {                       // control block placed after the stage ring
    uint64_t full[8], empty[8], accum;
    uint32_t tmem_base;
    int abort[3];
};

__global__ void __launch_bounds__(192, 1)
proj_fwd_tc_k(const __grid_constant__ CUtensorMap tmx, const __grid_constant__ CUtensorMap tmw, int64_t T, int nchunks,
              int chunks_per_split, int nq, int two_pass, int mt, int n_out, int stages, int tmem_cols,
              float* __restrict__ qpart, float* __restrict__ ssq, int* __restrict__ status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // the ring must start on a 1024-byte boundary (swizzle atoms)
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int w_bytes = 2 * nq * 128;                       // hi rows then lo rows
    const int umma_n = two_pass ? nq : 2 * nq;
    const int x_bytes = mt * kTcXBytes;                     // mt token tiles of 128 share one W' stage
    const int acc_cols = (umma_n + 31) & ~31;               // tensor-memory columns between the tiles' accumulators
    const int stage_bytes = x_bytes + w_bytes;
    TcSmem* ctl = reinterpret_cast<TcSmem*>(smem + stages * stage_bytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t t0 = (int64_t)blockIdx.x * kTcTok * mt;
    const int split = blockIdx.y;
    const int c_begin = split * chunks_per_split;
    const int c_end = (c_begin + chunks_per_split < nchunks) ? c_begin + chunks_per_split : nchunks;
    const int nloc = c_end - c_begin;
    volatile int* abort = ctl->abort;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 5); }
        mbar_init(smem_u32(&ctl->accum), 1);
        ctl->abort[0] = ctl->abort[1] = ctl->abort[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {      // tensor-memory allocation (whole warp), address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < nloc; ++i) {
                const int s = i % stages;
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ((i / stages) & 1) ^ 1, abort)) break;
                const uint32_t full = smem_u32(&ctl->full[s]);
                mbar_expect_tx(full, stage_bytes);
                const uint32_t dst = smem_u32(smem + s * stage_bytes);
                const int k = (c_begin + i) * kTcK;
                for (int m = 0; m < mt; ++m) tma_load_2d(dst + m * kTcXBytes, &tmx, full, k, (int)t0 + m * kTcTok);
                tma_load_2d(dst + x_bytes, &tmw, full, k, 0);
                if (two_pass) tma_load_2d(dst + x_bytes + nq * 128, &tmw, full, k, nq);     // box = Nq rows
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(umma_n);
            bool ok = true;
            for (int i = 0; i < nloc && ok; ++i) {
                const int s = i % stages;
                ok = mbar_wait(smem_u32(&ctl->full[s]), (i / stages) & 1, abort);
                if (!ok) break;
                tc_fence_after();
                const uint32_t xa = smem_u32(smem + s * stage_bytes);
                const uint64_t bd = smem_desc_k128(xa + x_bytes), bl = smem_desc_k128(xa + x_bytes + nq * 128);
                for (int m = 0; m < mt; ++m) {
                    const uint64_t ad = smem_desc_k128(xa + m * kTcXBytes);
#pragma unroll
                    for (int kk = 0; kk < kTcK / 16; ++kk) {    // 32 bytes further along the swizzled row per k-step
                        tc_mma(tmem + m * acc_cols, ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 2), idesc, (i > 0 || kk > 0) ? 1u : 0u);
                        if (two_pass) tc_mma(tmem + m * acc_cols, ad + (uint64_t)(kk * 2), bl + (uint64_t)(kk * 2), idesc, 1u);
                    }
                }
                tc_commit(smem_u32(&ctl->empty[s]));        // frees the stage when these MMAs have read it
            }
            if (ok) tc_commit(smem_u32(&ctl->accum));       // accumulator complete
        }
    } else {
        const int quad = warp & 3;
        const int row = quad * 32 + lane;                   // this thread's token within the tile
        float sqs[2] = {0.f, 0.f};                          // mt <= 2
        bool ok = true;
        for (int i = 0; i < nloc && ok; ++i) {
            const int s = i % stages;
            ok = mbar_wait(smem_u32(&ctl->full[s]), (i / stages) & 1, abort);
            if (!ok) break;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                if (m < mt) {
                    const uint32_t xr = smem_u32(smem + s * stage_bytes + m * kTcXBytes + row * 128);
                    float part = 0.f;                       // per 64-element chunk, then added: short chains round less
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float f[8];
                        unpack8(lds128(xr + ((c ^ (row & 7)) << 4)), f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) part = fmaf(f[e], f[e], part);
                    }
                    sqs[m] += part;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->empty[s]));
        }
        if (ok) ok = mbar_wait(smem_u32(&ctl->accum), 0, abort);
        ok = __all_sync(0xffffffffu, ok);                   // the tensor-memory loads below are warp-wide
        if (ok) {
            tc_fence_after();
            // hi columns [0, nq), lo columns [nq, 2 nq) (already added when the two halves share the accumulator)
#pragma unroll
            for (int m = 0; m < 2; ++m) {
            if (m >= mt) break;
            const int64_t t = t0 + m * kTcTok + row;
            const float sq = sqs[m];
            float* qrow = qpart + ((int64_t)split * T + t) * n_out;
            const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16) + m * acc_cols;
            for (int c0 = 0; c0 < nq; c0 += 16) {
                float hi[16], lo[16];
                tc_ld16(lane_base + c0, hi);
                if (two_pass) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) lo[e] = 0.f;
                } else {
                    tc_ld16(lane_base + nq + c0, lo);
                }
                if (t < T) {
#pragma unroll
                    for (int e = 0; e < 16; e += 4)
                        if (c0 + e < nq)
                            *reinterpret_cast<float4*>(qrow + c0 + e) =
                                make_float4(hi[e] + lo[e], hi[e + 1] + lo[e + 1], hi[e + 2] + lo[e + 2], hi[e + 3] + lo[e + 3]);
                }
            }
            if (t < T) ssq[(int64_t)split * T + t] = sq;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (ctl->abort[0]) report_abort(abort, status, 1);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    }
}

// ---- W' as two stacked K-major bf16 matrices: rows [0, nq) = hi, rows [nq, 2 nq) = lo, row length Kpad ----
__global__ void __launch_bounds__(256) pack_wt_k(int nC, int N, int nq, int Kpad, const float* __restrict__ W,
                                                 const float* __restrict__ gain, __nv_bfloat16* __restrict__ Wt) {
    // a 32 (k) x 32 (column) tile through shared memory: W is read along its rows, Wt written along k
    __shared__ float tile[32][33];
    const int k0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int r = ty; r < 32; r += 8) {
        const int k = k0 + r, c = c0 + tx;
        tile[r][tx] = (k < nC && c < N) ? __ldg(W + (int64_t)k * N + c) * __ldg(gain + k) : 0.f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int c = c0 + r, k = k0 + tx;
        if (c < nq && k < Kpad) {
            __nv_bfloat16 hi, lo;
            split_bf16(tile[tx][r], hi, lo);
            Wt[(int64_t)c * Kpad + k] = hi;
            Wt[(int64_t)(nq + c) * Kpad + k] = lo;
        }
    }
}

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

bool tensor_maps_available() { return encode_tiled_fn() != nullptr; }

// 2-D bf16 tensor map: `rows` rows of `cols` elements (row pitch `pitch_elems`), box = box_cols x box_rows,
// swizzle_bytes = 0 / 32 / 64 / 128 (the box's row must not be wider than the swizzle span).
bool make_tensor_map_2d(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_elems,
                        uint32_t box_cols, uint32_t box_rows, int swizzle_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch_elems * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                  : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D bf16 tensor map: d2 x d1 x d0 elements, d0 innermost, pitches in elements; box = box0 x box1 x box2.
bool make_tensor_map_3d(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch1_elems,
                        uint64_t pitch2_elems, uint32_t box0, uint32_t box1, uint32_t box2, int swizzle_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {d0, d1, d2};
    const cuuint64_t strides[2] = {pitch1_elems * 2, pitch2_elems * 2};
    const cuuint32_t box[3] = {box0, box1, box2};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                  : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool make_map(CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_elems, uint32_t box_rows) {
    return make_tensor_map_2d(m, base, cols, rows, pitch_elems, (uint32_t)kTcK, box_rows, 128);
}

// Columns of one half of W' in the packed operand: a multiple of 8 while both halves fit one instruction
// (2 Nq <= 256), else a multiple of 16 (the instruction's N granularity at M = 128).
int proj_tc_nq(int N) { return 2 * round_up(N, 8) <= 256 ? round_up(N, 8) : round_up(N, 16); }

bool proj_tc_supported(int n, int C, int N) {
    return proj_tc_nq(N) <= 256 && ((n * C) % 8) == 0 && encode_tiled_fn() != nullptr;
}

void launch_pack_wt(const mhclite_ctx* c, const ProjPlan& p, int N, const float* W, const float* gain, void* Wt,
                    cudaStream_t s) {
    c->launches += 1;
    const int nq = proj_tc_nq(N), Kpad = p.nchunks * kTcK;
    dim3 grid((unsigned)((Kpad + 31) / 32), (unsigned)((nq + 31) / 32));
    pack_wt_k<<<grid, 256, 0, s>>>(c->n * c->C, N, nq, Kpad, W, gain, (__nv_bfloat16*)Wt);
}

// Returns false when the tensor maps could not be built (the caller then uses the mma.sync kernel).
bool launch_proj_fwd_tc(const mhclite_ctx* c, int64_t T, int N, const ProjPlan& p, const void* x, const void* Wt,
                        float* qpart, float* ssq, int* status, cudaStream_t s) {
    const int nC = c->n * c->C, nq = proj_tc_nq(N), Kpad = p.nchunks * kTcK;
    const int two_pass = 2 * nq > 256;
    const int umma_n = two_pass ? nq : 2 * nq;
    if (nq > p.Npad) return false;                            // the rows of qpart hold Npad columns
    CUtensorMap tmx, tmw;
    if (!make_map(&tmx, x, (uint64_t)nC, (uint64_t)T, (uint64_t)nC, kTcTok)) return false;
    if (!make_map(&tmw, Wt, (uint64_t)Kpad, (uint64_t)(2 * nq), (uint64_t)Kpad, (uint32_t)umma_n)) return false;
    // wide projections (two instructions per k-step) stream more bytes of W' than of x per 128 tokens: two token
    // tiles then share each W' stage
    const int mt = (two_pass && T > kTcTok) ? 2 : 1;
    const int stage_bytes = mt * kTcXBytes + 2 * nq * 128;
    int stages = 100 * 1024 / stage_bytes;                   // two CTAs per SM when the stages are small enough
    if (stages > 6) stages = 6;
    if (stages < 3) stages = (220 * 1024 / stage_bytes < 4) ? 220 * 1024 / stage_bytes : 4;   // one CTA per SM
    if (stages > 8) stages = 8;
    const int smem = stages * stage_bytes + (int)sizeof(TcSmem) + 1024;
    int tmem_cols = 32;
    while (tmem_cols < (mt - 1) * ((umma_n + 31) & ~31) + umma_n) tmem_cols *= 2;
    c->launches += 1;
    KernelTimer timer_(c, MHCLITE_KERNEL_PROJ_FWD, s);
    cudaFuncSetAttribute(proj_fwd_tc_k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    dim3 grid((unsigned)((T + kTcTok * mt - 1) / (kTcTok * mt)), p.ksplit);
    proj_fwd_tc_k<<<grid, 192, smem, s>>>(tmx, tmw, T, p.nchunks, p.chunks_per_split, nq, two_pass, mt, p.Npad, stages,
                                          tmem_cols, qpart, ssq, status);
    return true;
}

}  // namespace mhcl
