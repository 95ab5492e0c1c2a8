// Shared device/host helpers for the LLA kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lla.h"

namespace lla {

// ---------------------------------------------------------------------------------------------
// Launch arguments handed from the C-ABI layer to the kernel launchers (plain pointers + sizes).
// ---------------------------------------------------------------------------------------------
// Debug build (-DLLA_DEBUG_BOUNDS, liblla_debug.so): the kernels' global stores check their row or record index
// against the extent that the launch geometry implies; a failed check counts in LLA_STATUS_BOUNDS, leaves the id
// of the first failing site in LLA_STATUS_BOUNDS_SITE and skips the store (no trap, the context stays usable).
// In the product build the macro is the constant `true`.
// ---------------------------------------------------------------------------------------------
#ifdef LLA_DEBUG_BOUNDS
__device__ __forceinline__ bool in_bounds(unsigned long long idx, unsigned long long limit, int* status, int site) {
    if (idx < limit) return true;
    if (status) {
        atomicAdd(status + LLA_STATUS_BOUNDS, 1);
        atomicCAS(status + LLA_STATUS_BOUNDS_SITE, 0, site);
    }
    return false;
}
#define LLA_IN_BOUNDS(idx, limit, status, site) \
    ::lla::in_bounds((unsigned long long)(idx), (unsigned long long)(limit), (status), (site))
#else
#define LLA_IN_BOUNDS(idx, limit, status, site) true
#endif

// ---------------------------------------------------------------------------------------------
// (batch, query head) unit -> (batch, key/value head) unit when `group` query heads share one K/V head
__host__ __device__ __forceinline__ int kv_unit(int bh, int H, int group) {
    return group <= 1 ? bh : (bh / H) * (H / group) + (bh % H) / group;
}

// Paged key/value cache of the decode entry points: pages of page_size keys laid out
// [num_pages][kv heads][page_size][d]; sequence b's keys j live in page table[b * max_pages + j / page_size].
// table == nullptr: the contiguous [B][kv heads][Lmax][d] cache.
struct PagedKv {
    const int* table;
    int page_size, max_pages, num_pages;
};
// row (in units of d elements) of key j of (sequence b, key/value head kvl of hkv) -- j's page must hold it
__device__ __forceinline__ size_t kv_row(const PagedKv& pg, int b, int kvl, int hkv, int Lmax, int j) {
    if (!pg.table) return ((size_t)b * hkv + kvl) * Lmax + j;
    int page = pg.table[(size_t)b * pg.max_pages + j / pg.page_size];
    page = min(max(page, 0), pg.num_pages - 1);      // a bad table entry reads the wrong page, never outside the cache
    return ((size_t)page * hkv + kvl) * pg.page_size + j % pg.page_size;
}

// Keys a decode unit sees: all len cached keys, or with a sliding window the last `window` of them
// (positions len - window .. len - 1).
__host__ __device__ __forceinline__ int visible_keys(int len, int Lmax, int window) {
    const int L = len < 1 ? 1 : (len > Lmax ? Lmax : len);
    return window > 0 && window < L ? window : L;
}
__host__ __device__ __forceinline__ int first_visible_key(int len, int Lmax, int window) {
    const int L = len < 1 ? 1 : (len > Lmax ? Lmax : len);
    return L - visible_keys(len, Lmax, window);
}

// Element strides (batch, head, row) of a [B, heads, rows, width] tensor whose innermost index has stride 1.
struct Strides {
    long long b, h, r;
    __host__ __device__ __forceinline__ size_t at(int batch, int head, long long row) const {
        return (size_t)((long long)batch * b + (long long)head * h + row * r);
    }
};
__host__ __device__ __forceinline__ Strides contiguous_strides(int heads, long long rows, int width) {
    return Strides{(long long)heads * rows * width, rows * width, (long long)width};
}

struct ForwardArgs {
    const void* q;
    const void* k;
    const void* v;
    void* out;
    int B, H, n, d, dv;
    int in_dtype, out_dtype;
    float scale, lambda;
    int causal;
    int max_iters;
    float tol;
    int head_rows;   // rows seeing fewer keys than this are solved directly (fp64)
    float* rho;      // optional
    float* stats;    // optional
    int* iters;      // optional
    int* status;     // optional device status words
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    const float* lambda_rows;   // optional per-row ridge [B, H, nq]
    int ridge_mode;             // lla_ridge_mode
    int nq;                     // query rows per head (the last nq of the n positions); nq == n: plain prefill
    int kv_group = 1;           // query heads per key/value head: k, v are [B, H / kv_group, n, d]
    int window = 0;             // causal sliding window: a row sees its last `window` positions (0: all)
    const float* rhs = nullptr; // tensor-core kernel only: solve C_i x_i = rhs_i (centred system) for the
    float* sol = nullptr;       // iterative rows and write x_i [B, H, nq, d] instead of the output
    const float* kbar_in = nullptr;     // with rhs / sol, optional: kbar_i [B, H, nq, d] and the saved stats [B, H, nq, 3] of
    const float* stats_in = nullptr;    // the forward; given both, the kernel skips the sweep that recomputes them
    // layouts of q [B, H, nq, d], k [B, H / kv_group, n, d], v [.., dv] and out [B, H, nq, dv]; zero = not set: the
    // launchers that build a ForwardArgs themselves call set_contiguous()
    Strides sq = {0, 0, 0}, sk = {0, 0, 0}, sv = {0, 0, 0}, so = {0, 0, 0};
    void set_contiguous() {
        const int hk = H / (kv_group > 0 ? kv_group : 1);
        sq = contiguous_strides(H, nq, d); sk = contiguous_strides(hk, n, d);
        sv = contiguous_strides(hk, n, dv); so = contiguous_strides(H, nq, dv);
    }
    const unsigned char* block_mask = nullptr;   // tensor-core kernel: block sparsity (lla_forward_params.block_mask)
    long long block_mask_stride = 0;
    long long wait_clocks = 0;  // tensor-core kernel: cap of its bounded waits in SM clocks (0: default) and a test
    int no_loads = 0;           // aid: issue no copy at all (lla_forward_params.debug_*)
    const void* minv = nullptr; // CG preconditioner matrices (fp16), set by forward_tensor_prepass when enabled
    int precondition = 0;       // 1: preconditioned CG when the workspace has room for the matrices
    const void* k16 = nullptr;  // fp16 copy of k and its validity word, set by forward_tensor_prepass
    const int* f16_ok = nullptr;
    int precise_iters = 1;      // tensor-core kernel: CG iterations run with bf16 hi + lo operand pairs before the
    int precise_iters_early = 4;   // switch to single fp16 operands (see lla_forward_params.cg_precise_iters); the
                                // second value is for row tiles that end within the first 8 d positions
};

struct DecodeArgs {
    const void* q;
    const void* kcache;
    const void* vcache;
    const int* lens;
    void* out;
    int B, H, Lmax, d, dv;
    int in_dtype, out_dtype;
    float scale, lambda;
    int splits;
    int head_rows;   // caches shorter than this are solved directly (fp64)
    int impl;        // lla_impl
    int* status;
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    const float* lambda_units;  // optional per-(sequence, head) ridge [B, H]
    int ridge_mode;             // lla_ridge_mode
    int kv_group = 1;           // query heads per key/value head: caches are [B, H / kv_group, Lmax, d]
    PagedKv paged = {nullptr, 0, 0, 0};
    int window = 0;             // sliding window: only the last `window` cached keys are visible (0: all)
    long long wait_clocks = 0;  // tensor-core kernel: cap of its bounded waits in SM clocks (0: default) and a test aid:
    int no_loads = 0;           // issue no copy at all (lla_decode_params.debug_*)
};

// Backward pass (backward appendix): gradients of a scalar loss with respect to q, k, v given
// g = dL/d(out) and the tensors the forward saved.
struct BackwardArgs {
    const void* q;
    const void* k;
    const void* v;
    const void* out;      // forward output [B, H, n, d] (out_dtype)
    const void* dout;     // upstream gradient g [B, H, n, d] (dout_dtype)
    const float* rho;     // saved by the forward [B, H, n, d]
    const float* stats;   // saved by the forward [B, H, n, 3]
    float* dq;            // [B, H, n, d] fp32
    float* dk;
    float* dv;
    int B, H, n, d;
    int out_dtype, dout_dtype;
    float scale, lambda;
    int max_iters;
    float tol;
    int head_rows;
    int* status;
    float* dlambda;       // optional [B, H, n]: dL/d(lambda_i) for a ridge of its own per query row
    int* iters;           // optional [B, H, n]: CG iterations of the extra solve (rows solved directly: untouched)
    void* workspace;
    size_t workspace_bytes;
    cudaStream_t stream;
    int kv_group;               // query heads per key/value head (k, v, dk, dv are [B, H / kv_group, n, d])
    int cuda_core_pairs;        // 1: pair kernel on the CUDA cores even where the tensor-core one exists
    int nq;                     // query rows of the forward being differentiated (0 = n): q, out, dout, rho, stats, dq are
                                // [B, H, nq, ..] for the positions n - nq .. n - 1
    int window;                 // causal sliding window of the forward being differentiated (0: none)
    int precondition;           // 1: the extra solve runs the preconditioned CG (as ForwardArgs::precondition)
    long long wait_clocks;      // as ForwardArgs::wait_clocks / no_loads, for the solve and the tensor-core kernels
    int no_loads;
    const unsigned char* block_mask;    // block sparsity of the forward being differentiated (as ForwardArgs::block_mask)
    long long block_mask_stride;
    cudaStream_t side_stream;   // optional: the directly-solved rows run here, forked from and joined to `stream`
    cudaEvent_t fork, join;
};
// The tensor-core kernels of the backward pass (lla_backward_tensor.cu).  Every array is contiguous [B, H (or the
// key/value heads), n, d]; gh/gl, yh/yl, tnh/tnl are the upstream gradient, y and -t as bf16 pairs hi + lo (gl may
// be null: a bf16 gradient has no lo half); rowsc is the per-row record of the CUDA-core kernels, of which the
// moments kernel fills gbar (slot 2); pairsc [heads][ceil(n / 2)][8] holds the scalars of two consecutive rows a, b
// per record: (nm2_a, nm2_b, ky_a, ky_b, gk_a, gk_b, kk_a, kk_b) with nm2 = -(m log2 e + log2 omega) (-1e30: the row
// is not handled by these kernels), ky = kbar.y, gk = gbar - kbar.t, kk = kbar.t - kappa.
struct BwdTensorArgs {
    const void *q, *k, *v;
    const void *gh, *gl, *yh, *yl, *tnh, *tnl;
    float* rowsc;
    const float* pairsc;
    const float* stats;
    const float* yvec;
    const float* tvec;
    float *kbar, *hvec, *dq, *dk, *dv;
    int B, H, n, d, first, kv_group;
    int nq;         // query rows (the positions n - nq .. n - 1); the row arrays are [B, H, nq, ..]
    int window;     // causal sliding window (0: none)
    long long wait_clocks;  // cap of the kernels' bounded waits in SM clocks (0: default) and a test aid: issue no copy at
    int no_loads;           // all (lla_backward_params.debug_*)
    int head_rows;  // with block_mask: key blocks that start below this position are always attended
    const unsigned char* block_mask;    // optional, as ForwardArgs::block_mask
    long long block_mask_stride;
    float scale;
    int* status;
    cudaStream_t stream;
};
int launch_backward_tensor(const BwdTensorArgs& a, int which);   // which: 0 = kbar, gbar, h; 1 = dQ; 2 = dK and dV
size_t backward_workspace_bytes(int B, int H, int n, int d);
int launch_backward(const BackwardArgs& a);

// Launchers implemented in the other translation units; each returns an lla_status.
int head_rows_count(const ForwardArgs& a);   // leading query rows per head solved directly
int launch_head_rows(const ForwardArgs& a);
int launch_forward_simt(const ForwardArgs& a);
int launch_forward_tensor(const ForwardArgs& a);
bool forward_tensor_supported(const ForwardArgs& a);
int forward_tensor_prepass(ForwardArgs& a);    // fp16 copy of k into the workspace (no-op without room)
size_t forward_tensor_scratch_bytes();         // d = 128 row-state scratch (0 if the device cannot be queried)
size_t forward_tensor_workspace_bytes(int B, int H, int n, int d);   // that scratch + the fp16 copy of k (upper bound: kv heads = H)
// CG preconditioner of the tensor-core forward (lla_precond.cu): one d x d fp16 matrix per block of 128 keys
int precond_blocks(int n);
// Beyond the first 16 blocks (2048 keys) the covariance changes little from one block of 128 keys to the next: only
// every fourth block gets a matrix of its own there, and a tile takes the last one at or before its key block.
__host__ __device__ __forceinline__ int precond_block_used(int g) { return g < 16 ? g : ((g + 1) / 4) * 4 - 1; }
size_t precond_gram_bytes(int units, int n, int d);     // fp32 running Gram sums (scratch of the pre-pass)
size_t precond_minv_bytes(int units, int n, int d);     // the fp16 matrices [units][blocks][d][d]
int launch_precond(const void* k, int B, int Hk, Strides sk, int n, int d, float lambda, int window, void* gram, void* minv,
                   cudaStream_t st);
int launch_decode(const DecodeArgs& a);
int launch_head_rows_decode(const DecodeArgs& a);
bool decode_tensor_supported(const DecodeArgs& a);
int launch_decode_tensor_moments(const DecodeArgs& a);
size_t decode_workspace_bytes(int B, int H, int d, int dv, int splits);   // required bytes (0 when unsplit)
size_t decode_record_bytes(int B, int H, int d, int dv, int splits);      // moment records of all parts

// ---------------------------------------------------------------------------------------------
// Element access
// ---------------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements (16-byte aligned for float, 8-byte for bf16) as floats.
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    float4 r;
    r.x = __uint_as_float(raw.x << 16);
    r.y = __uint_as_float(raw.x & 0xFFFF0000u);
    r.z = __uint_as_float(raw.y << 16);
    r.w = __uint_as_float(raw.y & 0xFFFF0000u);
    return r;
}

// Load 8 consecutive bf16 (16-byte aligned) as floats.
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float* dst) {
    const uint4 raw = *reinterpret_cast<const uint4*>(p);
    dst[0] = __uint_as_float(raw.x << 16); dst[1] = __uint_as_float(raw.x & 0xFFFF0000u);
    dst[2] = __uint_as_float(raw.y << 16); dst[3] = __uint_as_float(raw.y & 0xFFFF0000u);
    dst[4] = __uint_as_float(raw.z << 16); dst[5] = __uint_as_float(raw.z & 0xFFFF0000u);
    dst[6] = __uint_as_float(raw.w << 16); dst[7] = __uint_as_float(raw.w & 0xFFFF0000u);
}

__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// ---------------------------------------------------------------------------------------------
// Dense symmetric positive-definite solve in shared memory, double precision, by a whole block.
//   S   : D x D, row stride lds doubles, lower triangle filled; destroyed (LDL^T in place)
//   rhs : D doubles; replaced by the solution
//   n   : active size, a multiple of 8 and at most D (D only sizes the register arrays)
// Returns false if a pivot was not positive.  Every thread of the block must call it; blockDim.x
// must be a multiple of 32.
//
// Blocked right-looking LDL^T with panels of NB = 8 columns.  After a column is eliminated it holds
// L[r][c] * D_c (left unscaled) and the diagonal holds D_c.  The right-hand side rides along as
// matrix row D, so the forward substitution happens inside the elimination.  Per panel:
//   (i)   the 8 x 8 diagonal block is factorised by warp 0 in registers (one row per lane, pivot row
//         and pivot column passed by shuffles: no block barrier inside the eight column steps);
//   (ii)  every row below it (and the right-hand side) eliminates its eight panel entries against
//         the finished diagonal block, one thread per row;
//   (iii) one rank-8 update of everything to the right, all threads.
// The backward substitution is blocked the same way and runs in warp 0: eight unknowns at a time
// by shuffles, then their contribution to all earlier unknowns (held in registers, lane-strided).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double fast_rcp(double x) {
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
    r = r * (2.0 - x * r);
    r = r * (2.0 - x * r);
    return r;
}
// One Newton step on the 20-bit seed: relative error ~1e-12, enough for elimination multipliers
// (the error only perturbs the factorised matrix at that level) and one dependent pair shorter.
__device__ __forceinline__ double fast_rcp1(double x) {
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
    r = r * (2.0 - x * r);
    return r;
}


// (i): factorise the NB x NB diagonal block at c0 (called by one full warp).  The reciprocal of
// pivot c is left in S[c][c + 1], an element of the unused upper triangle (lds >= D + 1).
template <int NB>
__device__ __forceinline__ void ldlt_diag_block(double* S, int lds, int c0) {
    constexpr unsigned FULL = 0xffffffffu;
    const int tx = threadIdx.x & 31;
    const int i = tx & (NB - 1);   // lanes NB..31 mirror lanes 0..NB-1: every shuffle source is live
    double a[NB];
#pragma unroll
    for (int k = 0; k < NB; ++k) a[k] = k <= i ? S[(c0 + i) * lds + c0 + k] : 0.0;
#pragma unroll
    for (int k = 0; k < NB; ++k) {
        const double piv = __shfl_sync(FULL, a[k], k);
        const double inv = fast_rcp1(piv);
        if (tx == 0) S[(c0 + k) * lds + c0 + k + 1] = inv;
        const double l = a[k] * inv;
#pragma unroll
        for (int c2 = k + 1; c2 < NB; ++c2) {
            const double colv = __shfl_sync(FULL, a[k], c2);
            if (i >= c2) a[c2] -= l * colv;
        }
    }
    if (tx < NB) {
#pragma unroll
        for (int k = 1; k < NB; ++k)
            if (k <= i) S[(c0 + i) * lds + c0 + k] = a[k];
    }
}

template <int D>
__device__ __forceinline__ bool block_ldlt_solve(double* S, int lds, double* rhs, int n = D,
                                                 int nrhs = 1, int rhs_stride = 0) {
    // nrhs right-hand sides at rhs + q * rhs_stride, each replaced by its solution
    const int nend = n + nrhs;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int ty = tid >> 5, tx = tid & 31, ny = nt >> 5;
    constexpr int NB = 8;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int SLOTS = (D - NB + 31) / 32 > 0 ? (D - NB + 31) / 32 : 1;   // trailing columns per lane
    static_assert(D % NB == 0, "head size must be a multiple of the panel width");
    __syncthreads();
    if (ty == 0) ldlt_diag_block<NB>(S, lds, 0);
    __syncthreads();
    for (int c0 = 0; c0 < n; c0 += NB) {
        double dinv[NB];
#pragma unroll
        for (int k = 0; k < NB; ++k) dinv[k] = S[(c0 + k) * lds + c0 + k + 1];
        // (ii)
        for (int r = c0 + NB + tid; r < nend; r += nt) {
            double* rowp = r < n ? S + r * lds : rhs + (r - n) * rhs_stride;
            double x[NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) x[k] = rowp[c0 + k];
#pragma unroll
            for (int k = 0; k < NB - 1; ++k) {
                const double l = x[k] * dinv[k];
#pragma unroll
                for (int c2 = k + 1; c2 < NB; ++c2) x[c2] -= l * S[(c0 + c2) * lds + c0 + k];
            }
#pragma unroll
            for (int k = 1; k < NB; ++k) rowp[c0 + k] = x[k];
        }
        __syncthreads();
        // (iii) element (r, c2) -= sum_k S[r][c0+k] * S[c2][c0+k] / D_k.  A lane keeps the scaled
        // panel entries of its columns c2 in registers for the whole update and walks down the rows;
        // a row's eight panel entries are the same address for every lane (broadcast loads), so
        // shared-memory traffic is one load and one store per updated element.
        if (c0 + NB < n) {
            double u[SLOTS][NB];
#pragma unroll
            for (int sl = 0; sl < SLOTS; ++sl) {
                const int c2 = c0 + NB + tx + 32 * sl;
#pragma unroll
                for (int k = 0; k < NB; ++k) u[sl][k] = c2 < n ? S[c2 * lds + c0 + k] * dinv[k] : 0.0;
            }
            auto update_row = [&](int r) {
                double* rowp = r < n ? S + r * lds : rhs + (r - n) * rhs_stride;
                double a[NB];
#pragma unroll
                for (int k = 0; k < NB; ++k) a[k] = rowp[c0 + k];
                const int cmax = r < n ? r : n - 1;
#pragma unroll
                for (int sl = 0; sl < SLOTS; ++sl) {
                    const int c2 = c0 + NB + tx + 32 * sl;
                    if (c2 <= cmax) {
                        double acc = 0.0;
#pragma unroll
                        for (int k = 0; k < NB; ++k) acc += a[k] * u[sl][k];
                        rowp[c2] -= acc;
                    }
                }
            };
            if (ty == 0) {
                // warp 0 brings the next diagonal block up to date and factorises it at once, while
                // the other warps update the rows below it
                // (a lane per element of the block, two passes)
#pragma unroll
                for (int pass = 0; pass < NB * NB / 32; ++pass) {
                    const int e = tx + 32 * pass, ro = e / NB, co = e % NB;
                    if (co <= ro) {
                        const double* ra = S + (c0 + NB + ro) * lds + c0;
                        const double* rb = S + (c0 + NB + co) * lds + c0;
                        double acc = 0.0;
#pragma unroll
                        for (int k = 0; k < NB; ++k) acc += ra[k] * (rb[k] * dinv[k]);
                        S[(c0 + NB + ro) * lds + c0 + NB + co] -= acc;
                    }
                }
                __syncwarp();
                ldlt_diag_block<NB>(S, lds, c0 + NB);
                if (ny == 1)
                    for (int r = c0 + 2 * NB; r < nend; ++r) update_row(r);
            } else {
                for (int r = c0 + 2 * NB + ty - 1; r < nend; r += ny - 1) update_row(r);
            }
            __syncthreads();
        }
    }
    bool ok = true;
    for (int k = 0; k < n; ++k)
        if (!(S[k * lds + k] > 0.0)) ok = false;
    // rhs now holds y with L y = b.  Backward: x_t = (y_t - sum_{r>t} S[r][t] x_r) / D_t.
    // (one warp per right-hand side: warp ty takes the sides ty, ty + ny, ...)
    for (int q = ty; q < nrhs; q += ny) {
        double* rhs_q = rhs + q * rhs_stride;
        constexpr int PER = (D + 31) / 32;
        const int i = tx & 7;
        double part[PER], yv[PER];
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int t = tx + 32 * u;
            part[u] = 0.0;
            yv[u] = t < n ? rhs_q[t] : 0.0;
        }
        for (int c0 = n - NB; c0 >= 0; c0 -= NB) {
            // y - (contributions of later panels) for the eight unknowns c0 + i of this panel
            double mine = 0.0;
#pragma unroll
            for (int u = 0; u < PER; ++u)
                if (u == (c0 >> 5)) mine = yv[u] - part[u];
            double val = __shfl_sync(FULL, mine, (c0 & 31) + i);
            double sc[NB];   // column c0 + i of the diagonal block, below the diagonal
#pragma unroll
            for (int r = 0; r < NB; ++r) sc[r] = r > i ? S[(c0 + r) * lds + c0 + i] : 0.0;
            const double di = S[(c0 + i) * lds + c0 + i + 1];
            double xb[NB];
#pragma unroll
            for (int t = NB - 1; t >= 0; --t) {
                xb[t] = __shfl_sync(FULL, val * di, t);
                val -= sc[t] * xb[t];
            }
            if (tx < NB) {
                double xm = 0.0;
#pragma unroll
                for (int t = 0; t < NB; ++t)
                    if (t == tx) xm = xb[t];
                rhs_q[c0 + tx] = xm;
            }
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int t = tx + 32 * u;
                if (t < c0) {
#pragma unroll
                    for (int r = 0; r < NB; ++r) part[u] += S[(c0 + r) * lds + t] * xb[r];
                }
            }
        }
    }
    __syncthreads();
    return ok;
}

#define LLA_CUDA_TRY(expr)                         \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess) return LLA_ERR_CUDA; \
    } while (0)

}  // namespace lla
