// Shared device/host helpers of the mHC-lite library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "../../include/mhclite.h"

namespace mhcl {

constexpr int kMaxN = 5;          // residual streams supported: 2..5
#define MHCLITE_STEP_CHUNKS 8      // token chunks that mhclite_step_host keeps in flight
constexpr int kMaxFact = 120;     // 5!
constexpr int kWarp = 32;

// ---- context -------------------------------------------------------------------------------------
}  // namespace mhcl

struct mhclite_ctx {
    int n, C, device;
    int nfact;                    // residual weights per token: n!, or K with a subset of the permutations attached
    const uint8_t* table_dev;     // caller-owned device table [K][n] of that subset (null: all n! permutations)
    uint8_t table_host[120 * 5];  // validated host copy of the subset
    int sm_count;
    void* ws;
    size_t ws_bytes;
    mutable int64_t launches;     // kernels launched through this context
    int* status_word;             // device status word inside the attached workspace (null until first used)
    bool timing;                  // record CUDA events around the main kernels (mhclite_set_kernel_timing)
    cudaEvent_t ev[MHCLITE_KERNEL_COUNT][2];
    mutable bool ev_recorded[MHCLITE_KERNEL_COUNT];   // the pair has bracketed at least one launch
    // mhclite_step_host: copy-in and copy-out streams and the events that chain its token chunks (made on first use)
    cudaStream_t copy_in, copy_out;
    cudaEvent_t ev_fork, ev_join, ev_in[MHCLITE_STEP_CHUNKS], ev_cmp[MHCLITE_STEP_CHUNKS];
    // projection partials left in the workspace by mhclite_postres_fwd_next_proj for mhclite_pre_fwd_resume
    int64_t pending_T;            // tokens they cover (-1: none)
    const void* pending_x;        // the x_next they were computed from
    int pending_ksplit;           // K slices they come in
    char err[256];
};

namespace mhcl {

inline int ipow_fact(int n) { int f = 1; for (int i = 2; i <= n; ++i) f *= i; return f; }
inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline int64_t round_up64(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

// Layout of e = rstd * alpha (.) dz as a bf16 pair (hi, lo) for the tensor-core backward, Kp columns per
// token (a multiple of 16).  Tokens are grouped in granules of 128; inside a granule the columns are
// grouped by 8, and inside a column group the 16-byte pieces of the 128 tokens lie back to back:
//   element (t, c)  ->  ((t / 128) * (Kp / 8) + c / 8) * 1024 + (t % 128) * 8 + c % 8.
// A granule is then a ready-made shared-memory operand without swizzle (8 x 16-byte core matrices) both
// with tokens as the M dimension and columns as K, and with columns as N and tokens as K.
// db / dalpha as per-block partials (deterministic, and nothing has to be cleared first): a kernel that gets a null
// dalpha writes its block's sums to db[block * kPartStride + c], c < N for db and N..N+2 for dalpha; tail_finish_k
// adds the blocks up in a fixed order.
constexpr int kPartStride = 136;
constexpr int kMaxParts = 148 * 16;

constexpr int kEGranule = 128;
__host__ __device__ inline int64_t e_tiled_index(int Kp, int64_t t, int c) {
    return ((t >> 7) * (Kp >> 3) + (c >> 3)) * 1024 + (t & 127) * 8 + (c & 7);
}

// Grid of a warp-per-token kernel (8 warps per block) whose warps stride over the tokens: at most cap_blocks
// blocks, and no more warps than give every warp the same number of tokens (a warp with one token less than
// its neighbours only idles at the end).
inline int balanced_warp_blocks(int64_t T, int64_t cap_blocks) {
    if (T < 1) return 1;
    const int64_t per_warp = (T + cap_blocks * 8 - 1) / (cap_blocks * 8);
    const int64_t warps = (T + per_warp - 1) / per_warp;
    return (int)((warps + 7) / 8);
}

// Number of projection columns. kind 0: n!+2n (mHC-lite); kind 1: n*n+2n (SK path).
inline int n_res_cols(int n, int kind) { return kind == 0 ? ipow_fact(n) : n * n; }
inline int n_cols(int n, int kind) { return n_res_cols(n, kind) + 2 * n; }
// Projection columns of a context: a subset of K permutations (paper Section 5) narrows the residual group to K.
inline int ctx_cols(const mhclite_ctx* c, int kind) { return (kind == 0 ? c->nfact : c->n * c->n) + 2 * c->n; }

// Brackets one kernel launch with the context's events when kernel timing is switched on.
struct KernelTimer {
    const mhclite_ctx* c; int id; cudaStream_t s;
    KernelTimer(const mhclite_ctx* c_, int id_, cudaStream_t s_) : c(c_), id(id_), s(s_) {
        if (c->timing) cudaEventRecord(c->ev[id][0], s);
    }
    ~KernelTimer() { if (c->timing) { cudaEventRecord(c->ev[id][1], s); c->ev_recorded[id] = true; } }
};

int fail(mhclite_ctx* ctx, int status, const char* fmt, ...);
int check_cuda(mhclite_ctx* ctx, cudaError_t e, const char* what);

// Launch plan of the tensor-core projection for one problem size (proj_mma.cu).
constexpr int kMaxKSplit = 4;
struct ProjPlan {
    int NT;                 // 8-column tiles of the padded projection (1..5, or 20)
    int Npad;               // NT * 8: row length of qpart
    int nchunks;            // 64-wide K chunks covering nC
    int ksteps;             // 16-wide MMA k-steps in the packed weights (4 per chunk)
    int ksplit;             // K slices whose partial results the activation kernel adds
    int chunks_per_split;
};
ProjPlan plan_proj(int n, int C, int64_t T, int N, int sm_count);

// Launch plan of the tensor-core backward tail (tail_mma.cu).
struct TailPlan {
    int Kp, KS;             // projection columns padded to 16, and Kp / 16
    int slices, splits;     // 64-channel slices x token ranges = the grid
    int64_t tok_per_split;  // multiple of 32
    bool supported;         // KS <= 3 (N <= 48) and n <= 4: the fused mma.sync kernel
    // wider projections: tcgen05 kernels (tail_tc.cu) when the shape allows, else the CUDA-core kernels
    bool tc;                // Kp <= 256 and rows of x a multiple of 16 bytes
    int g_mt;               // G kernel: 128-row accumulators per CTA (g_mt * Kp <= 512 tensor-memory columns)
    int g_groups, g_splits; // its grid: row groups of 128 * g_mt x token ranges
    int64_t g_tok_per_split;   // multiple of 128
    // narrow projections: the fused tcgen05 kernel (tail_ftc.cu) when C is a multiple of 64
    bool ftc;
    int f_slices, f_splits;  // its grid: 64-channel slices x ranges of 128-token tiles
    int f_ring;              // dxhat buffers in tensor memory
};
TailPlan plan_tail(int n, int C, int64_t T, int N, int sm_count);

// Workspace layout (all offsets 256-byte aligned), see plan_workspace.
struct Workspace {
    float* e;        // [T][Npad]   rstd * alpha (.) dz, fp32
    float* kappa;    // [T]         rstd^2 * sum_c (alpha dz)_c p_c / (nC)
    float* G;        // [nC][Npad]  sum_t x[t,m] e[t,c] (before the gain factor)
    float* dH_pre;   // [T][n]      <du, x_j> of the fused backward tail
    void* Wp;        // packed bf16 hi/lo weights in MMA fragment order
    float* qpart;    // [kMaxKSplit][T][NTpad*8] partial x W' of each K slice
    float* ssq;      // [kMaxKSplit][T]          partial sums of squares
    void *ehi, *elo; // [T rounded up to 32][Kp] bf16 pair hi + lo = e
    float* Gpart;    // [splits or g_splits][nC][Kp] partial G of each token range
    void* Wb;        // bf16 W' blocks of the tcgen05 dx kernels
    void* Wt;        // [2 nq][Kpad] bf16: W' hi rows then lo rows, K-major (tcgen05 projection)
    float* dpart;    // [kMaxParts][kPartStride] per-block partials of db and dalpha
    int* status;     // device status word (0, or a negative mhclite_status raised by a kernel)
    size_t bytes;
    int Npad;
};
// (sm_count: SMs of the device the plan is for; the B200's 148 where no context is at hand)
Workspace plan_workspace(int n, int C, int64_t T, int N, void* base, int sm_count = 148);

// Permutation tables in constant memory (perm_table.cu).
struct PermTables {
    uint8_t sigma[kMaxFact * kMaxN];         // sigma[k*n + i] = sigma_k(i)
    uint8_t klist[kMaxN * kMaxN * 24];       // klist[(i*n+j)*(n-1)! + r] = r-th k with sigma_k(i) = j
};
void host_perm_tables(int n, PermTables* out);
cudaError_t upload_perm_tables(int n);       // to the current device
cudaError_t download_perm_sigma(int n, uint8_t* sigma_host);

// Instantiates a statement for the compile-time stream count N_ = n (2..5).
#define MHCL_DISPATCH_N(n, ...)                               \
    switch (n) {                                              \
        case 2: { constexpr int N_ = 2; __VA_ARGS__; } break; \
        case 3: { constexpr int N_ = 3; __VA_ARGS__; } break; \
        case 4: { constexpr int N_ = 4; __VA_ARGS__; } break; \
        case 5: { constexpr int N_ = 5; __VA_ARGS__; } break; \
        default: break;                                       \
    }

// ---- device helpers ------------------------------------------------------------------------------
#ifdef __CUDACC__
extern __constant__ PermTables c_perm[kMaxN + 1];   // indexed by n

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

// 8 bf16 (one 16-byte vector) -> 8 floats
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    f[0] = bf16lo(v.x); f[1] = bf16hi(v.x); f[2] = bf16lo(v.y); f[3] = bf16hi(v.y);
    f[4] = bf16lo(v.z); f[5] = bf16hi(v.z); f[6] = bf16lo(v.w); f[7] = bf16hi(v.w);
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);      // .x = a (low half), .y = b
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    uint4 v;
    v.x = pack2(f[0], f[1]); v.y = pack2(f[2], f[3]); v.z = pack2(f[4], f[5]); v.w = pack2(f[6], f[7]);
    return v;
}
// Two fp32 in one 64-bit register and the packed fused multiply-add of sm_100 (two FMAs per instruction).
__device__ __forceinline__ uint64_t pack2f(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2f(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// 8 bf16 (one 16-byte vector) -> 4 packed pairs of floats
__device__ __forceinline__ void unpack8x2(const uint4& v, uint64_t* f) {
    f[0] = pack2f(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u));
    f[1] = pack2f(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
    f[2] = pack2f(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u));
    f[3] = pack2f(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
}
__device__ __forceinline__ uint4 pack8x2(const uint64_t* f) {
    float a[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) unpack2f(f[k], a[2 * k], a[2 * k + 1]);
    uint4 v;
    v.x = pack2(a[0], a[1]); v.y = pack2(a[2], a[3]); v.z = pack2(a[4], a[5]); v.w = pack2(a[6], a[7]);
    return v;
}
// streaming 16-byte accesses: activations are touched once per kernel
__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
#endif

}  // namespace mhcl
