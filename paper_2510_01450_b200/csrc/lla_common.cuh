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
};

// Launchers implemented in the other translation units; each returns an lla_status.
int head_rows_count(const ForwardArgs& a);   // leading rows per head solved directly
int launch_head_rows(const ForwardArgs& a);
int launch_forward_simt(const ForwardArgs& a);
int launch_forward_tensor(const ForwardArgs& a);
bool forward_tensor_supported(const ForwardArgs& a);
int launch_decode(const DecodeArgs& a);
int launch_head_rows_decode(const DecodeArgs& a);
bool decode_tensor_supported(const DecodeArgs& a);
int launch_decode_tensor_moments(const DecodeArgs& a);
size_t decode_workspace_bytes(int B, int H, int d, int dv, int splits);

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
// Returns false if a pivot was not positive.  Every thread of the block must call it; blockDim.x
// must be a multiple of 32 with at least two warps.
//
// The right-hand side rides along as an extra matrix row, so the forward substitution happens
// inside the elimination; the backward substitution is a column sweep by warp 0 with the partial
// sums of each unknown held in registers.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double fast_rcp(double x) {
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
    r = r * (2.0 - x * r);
    r = r * (2.0 - x * r);
    return r;
}

template <int D>
__device__ __forceinline__ bool block_ldlt_solve(double* S, int lds, double* rhs) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int ty = tid >> 5, tx = tid & 31, ny = nt >> 5;
    bool ok = true;
    __syncthreads();
    // Blocked right-looking LDL^T, panels of NB columns.  After a column is eliminated it holds
    // L[r][c] * D_c (left unscaled) and the diagonal holds D_c.  The right-hand side is carried as
    // row index D.  Per panel: (a) eliminate inside the panel, one thread per row; (b) one rank-NB
    // update of everything to the right (4 multiply-adds per element loaded and stored).
    constexpr int NB = 8;
    static_assert(D % NB == 0, "head size must be a multiple of the panel width");
    for (int c0 = 0; c0 < D; c0 += NB) {
        for (int k = 0; k < NB; ++k) {
            const int c = c0 + k;
            const double piv = S[c * lds + c];
            if (!(piv > 0.0)) ok = false;
            const double inv = fast_rcp(piv);
            for (int r = c + 1 + tid; r <= D; r += nt) {
                double* rowp = r < D ? S + r * lds : rhs;
                const double l = rowp[c] * inv;
                for (int c2 = c + 1; c2 < c0 + NB; ++c2)
                    if (r == D || c2 <= r) rowp[c2] -= l * S[c2 * lds + c];
            }
            __syncthreads();
        }
        if (c0 + NB < D) {
            double dinv[NB];
#pragma unroll
            for (int k = 0; k < NB; ++k) dinv[k] = fast_rcp(S[(c0 + k) * lds + c0 + k]);
            for (int r = c0 + NB + ty; r <= D; r += ny) {
                double* rowp = r < D ? S + r * lds : rhs;
                double ls[NB];
#pragma unroll
                for (int k = 0; k < NB; ++k) ls[k] = rowp[c0 + k] * dinv[k];
                const int cmax = r < D ? r : D - 1;
                for (int c2 = c0 + NB + tx; c2 <= cmax; c2 += 32) {
                    const double* u = S + c2 * lds + c0;
                    double acc = 0.0;
#pragma unroll
                    for (int k = 0; k < NB; ++k) acc += ls[k] * u[k];
                    rowp[c2] -= acc;
                }
            }
            __syncthreads();
        }
    }
    if (!(S[(D - 1) * lds + (D - 1)] > 0.0)) ok = false;
    // rhs now holds y with L y = b.  Backward: x_r = (y_r - sum_{t>r} S[t][r] x_t) / D_r.
    if (tid < 32) {
        constexpr int PER = (D + 31) / 32;
        double part[PER], dinv[PER], yv[PER];
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int t = tx + 32 * u;
            part[u] = 0.0;
            dinv[u] = t < D ? fast_rcp(S[t * lds + t]) : 0.0;
            yv[u] = t < D ? rhs[t] : 0.0;
        }
        for (int r = D - 1; r >= 0; --r) {
            const int owner = r & 31, slot = r >> 5;
            double xr = 0.0;
#pragma unroll
            for (int u = 0; u < PER; ++u)
                if (u == slot) xr = (yv[u] - part[u]) * dinv[u];
            xr = __shfl_sync(0xffffffffu, xr, owner);
            if (tx == owner) rhs[r] = xr;
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int t = tx + 32 * u;
                if (t < r) part[u] += S[r * lds + t] * xr;
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
