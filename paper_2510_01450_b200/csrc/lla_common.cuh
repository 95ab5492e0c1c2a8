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
//   S   : d x d, row stride lds doubles, lower triangle filled; destroyed (LDL^T in place)
//   rhs : d doubles; replaced by the solution
// Returns false if a pivot was not positive.  Every thread of the block must call it.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ bool block_ldlt_solve(double* S, int lds, double* rhs, int d) {
    const int tid = threadIdx.x, nt = blockDim.x;
    bool ok = true;
    __syncthreads();
    // after step c, column c holds L[r][c] * D_c (left unscaled), diagonal holds D_c
    for (int c = 0; c < d - 1; ++c) {
        const double piv = S[c * lds + c];
        if (!(piv > 0.0)) ok = false;
        const double inv = 1.0 / piv;
        const int rem = d - 1 - c;
        for (int e = tid; e < rem * rem; e += nt) {
            const int rr = e / rem, cc = e - rr * rem;
            if (cc <= rr) {
                const int r = c + 1 + rr, c2 = c + 1 + cc;
                S[r * lds + c2] -= S[r * lds + c] * S[c2 * lds + c] * inv;
            }
        }
        __syncthreads();
    }
    if (!(S[(d - 1) * lds + (d - 1)] > 0.0)) ok = false;
    if (tid < 32) {
        const int lane = tid;
        for (int r = 0; r < d; ++r) {   // forward with the unit lower factor L[t][r] = S[t][r] / S[r][r]
            const double yr = rhs[r] / S[r * lds + r];
            for (int t = r + 1 + lane; t < d; t += 32) rhs[t] -= S[t * lds + r] * yr;
            __syncwarp();
        }
        for (int r = lane; r < d; r += 32) rhs[r] /= S[r * lds + r];
        __syncwarp();
        for (int r = d - 1; r > 0; --r) {   // backward with L^T
            const double xr = rhs[r];
            for (int t = lane; t < r; t += 32) rhs[t] -= S[r * lds + t] / S[t * lds + t] * xr;
            __syncwarp();
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
