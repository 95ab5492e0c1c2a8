// Preconditioner for the conjugate-gradient solve of the tensor-core forward kernel (Algorithm 2 with a
// preconditioner; the paper runs plain CG).
//
// The system of query row i is C_i = sum_j p_ij (k_j - kbar_i)(k_j - kbar_i)^T + ridge_i I with weights
// p_ij = w_ij / omega_i over the visible keys.  With all weights equal it is the covariance of those keys,
// which is the same matrix for every row that sees the same keys and changes slowly from row to row.  Its
// inverse, formed once per block of 128 keys for the keys up to the end of that block, is a good
// preconditioner wherever the weights are not far from uniform: on the synthetic workloads it halves the
// iteration count.  It never changes the solution, only the path to it, so it is built in fp32 and stored
// in fp16; a block whose inversion breaks down gets the identity.
//
// Three kernels, all on the caller's stream ahead of the forward kernel:
//   gram_blocks_kernel   G_b = sum_j k_j k_j^T and s_b = sum_j k_j over the keys of block b
//   gram_scan_kernel     running sums over b (in place)
//   precond_invert_kernel   M_g = (G / L - s s^T / L^2 + (lambda / L) I)^{-1} by Gauss-Jordan elimination in
//                        shared memory, scaled to a largest entry of one (conjugate gradients do not see the
//                        scale of a preconditioner), rounded to fp16
#include <cuda_fp16.h>

#include "lla_common.cuh"

namespace lla {
namespace {

constexpr int PC_THREADS = 256;
constexpr int PC_BLOCK = 128;      // keys per Gram block

template <int D>
__global__ void __launch_bounds__(PC_THREADS)
gram_blocks_kernel(const __nv_bfloat16* __restrict__ k, float* __restrict__ gram, int n, int nb, int Hk, Strides sk) {
    constexpr int LD = D + 1, TR = D / 16;
    extern __shared__ float pc_smem[];
    float* ks = pc_smem;                                   // [PC_BLOCK][LD]
    const int b = blockIdx.x, u = blockIdx.y, tid = threadIdx.x;
    const int j0 = b * PC_BLOCK, rows = min(PC_BLOCK, n - j0);
    const __nv_bfloat16* src = k + sk.at(u / Hk, u % Hk, j0);
    for (int idx = tid; idx < PC_BLOCK * (D / 8); idx += PC_THREADS) {
        const int r = idx / (D / 8), c = (idx % (D / 8)) * 8;
        float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (r < rows) load8(src + (size_t)r * sk.r + c, x);
#pragma unroll
        for (int e = 0; e < 8; ++e) ks[r * LD + c + e] = x[e];
    }
    __syncthreads();
    const int ti = tid >> 4, tj = tid & 15;
    float acc[TR][TR] = {};
    for (int r = 0; r < PC_BLOCK; ++r) {
        float a[TR], c[TR];
#pragma unroll
        for (int e = 0; e < TR; ++e) { a[e] = ks[r * LD + ti + 16 * e]; c[e] = ks[r * LD + tj + 16 * e]; }
#pragma unroll
        for (int x = 0; x < TR; ++x)
#pragma unroll
            for (int y = 0; y < TR; ++y) acc[x][y] = fmaf(a[x], c[y], acc[x][y]);
    }
    float* dst = gram + ((size_t)u * nb + b) * (D * D + D);
#pragma unroll
    for (int x = 0; x < TR; ++x)
#pragma unroll
        for (int y = 0; y < TR; ++y) dst[(ti + 16 * x) * D + tj + 16 * y] = acc[x][y];
    if (tid < D) {
        float s = 0.f;
        for (int r = 0; r < PC_BLOCK; ++r) s += ks[r * LD + tid];
        dst[D * D + tid] = s;
    }
}

// gram[u][b] += gram[u][b - 1], element by element
__global__ void __launch_bounds__(PC_THREADS)
gram_scan_kernel(float* __restrict__ gram, int nb, int rec) {
    const int e = blockIdx.x * PC_THREADS + threadIdx.x;
    if (e >= rec) return;
    float* p = gram + (size_t)blockIdx.y * nb * rec + e;
    float run = p[0];
    for (int b = 1; b < nb; ++b) {
        run += p[(size_t)b * rec];
        p[(size_t)b * rec] = run;
    }
}

// One preconditioner per key block g: the keys [lo, hi) with hi = min(n, 128 (g + 1)) and lo = 0, or with a
// sliding window the start of the block that holds position hi - window.
template <int D>
__global__ void __launch_bounds__(PC_THREADS)
precond_invert_kernel(const float* __restrict__ gram, __half* __restrict__ minv, int n, int nb, float lambda, int window) {
    constexpr int LD = D + 1;
    extern __shared__ float pc_smem[];
    float* A = pc_smem;                                    // [D][LD]
    float* sv = A + D * LD;                                // [D]
    __shared__ float s_red[PC_THREADS / 32];
    __shared__ int s_bad;
    const int g = blockIdx.x, u = blockIdx.y, tid = threadIdx.x;
    if (precond_block_used(g) != g) return;        // no tile asks for this block's matrix
    const int rec = D * D + D;
    const int hi = min(n, PC_BLOCK * (g + 1));
    const int glo = window > 0 ? max(0, hi - window) / PC_BLOCK : 0;     // first block that counts
    const float* Gh = gram + ((size_t)u * nb + g) * rec;
    const float* Gl = glo > 0 ? gram + ((size_t)u * nb + glo - 1) * rec : nullptr;
    const float L = (float)(hi - glo * PC_BLOCK), invL = 1.f / L;
    if (tid == 0) s_bad = 0;
    for (int e = tid; e < D; e += PC_THREADS) sv[e] = (Gh[D * D + e] - (Gl ? Gl[D * D + e] : 0.f)) * invL;
    __syncthreads();
    float tr_part = 0.f;
    for (int e = tid; e < D * D; e += PC_THREADS) {
        const int r = e / D, c = e % D;
        const float v = (Gh[e] - (Gl ? Gl[e] : 0.f)) * invL - sv[r] * sv[c];
        A[r * LD + c] = v;
        if (r == c) tr_part += v;
    }
    // ridge: lambda / L, but at least a millionth of the mean diagonal so that the elimination cannot stall
    for (int off = 16; off > 0; off >>= 1) tr_part += __shfl_xor_sync(0xffffffffu, tr_part, off);
    if ((tid & 31) == 0) s_red[tid >> 5] = tr_part;
    __syncthreads();
    float trace = 0.f;
    for (int w = 0; w < PC_THREADS / 32; ++w) trace += s_red[w];
    const float ridge = fmaxf(lambda * invL, 1e-6f * trace / D);
    for (int e = tid; e < D; e += PC_THREADS) A[e * LD + e] += ridge;
    __syncthreads();
    // In-place Gauss-Jordan inversion (no pivoting: the matrix is symmetric positive definite).  Thread (ty, tx)
    // of the 16 x 16 grid keeps the entries (ty + 16 i, tx + 16 j) in registers; per step the pivot row and the
    // pivot column go through shared memory (two buffers in turn: one barrier per step).
    constexpr int TR = D / 16;
    const int ty = tid >> 4, tx = tid & 15;
    float a[TR][TR];
#pragma unroll
    for (int i = 0; i < TR; ++i)
#pragma unroll
        for (int j = 0; j < TR; ++j) a[i][j] = A[(ty + 16 * i) * LD + tx + 16 * j];
    __shared__ float s_row[2][D], s_col[2][D];
    for (int kk = 0; kk < D; ++kk) {
        const int ki = kk >> 4, kr = kk & 15, bsel = kk & 1;
        if (ty == kr) {
#pragma unroll
            for (int i = 0; i < TR; ++i)
                if (i == ki) {
#pragma unroll
                    for (int j = 0; j < TR; ++j) s_row[bsel][tx + 16 * j] = a[i][j];
                }
        }
        if (tx == kr) {
#pragma unroll
            for (int j = 0; j < TR; ++j)
                if (j == ki) {
#pragma unroll
                    for (int i = 0; i < TR; ++i) s_col[bsel][ty + 16 * i] = a[i][j];
                }
        }
        __syncthreads();
        const float piv = s_row[bsel][kk];
        if (!(piv > 0.f) || !isfinite(piv)) { if (tid == 0) s_bad = 1; }
        const float ip = 1.f / piv;
        float rw[TR], cl[TR];
#pragma unroll
        for (int j = 0; j < TR; ++j) rw[j] = s_row[bsel][tx + 16 * j] * ip;
#pragma unroll
        for (int i = 0; i < TR; ++i) cl[i] = s_col[bsel][ty + 16 * i];
        // every entry as an ordinary one, then the owners of the pivot row and column put theirs right
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < TR; ++j) a[i][j] = fmaf(-cl[i], rw[j], a[i][j]);
        if (ty == kr) {
#pragma unroll
            for (int i = 0; i < TR; ++i)
                if (i == ki) {
#pragma unroll
                    for (int j = 0; j < TR; ++j) a[i][j] = rw[j];
                }
        }
        if (tx == kr) {
#pragma unroll
            for (int j = 0; j < TR; ++j)
                if (j == ki) {
#pragma unroll
                    for (int i = 0; i < TR; ++i) a[i][j] = (ty == kr && i == ki) ? ip : -cl[i] * ip;
                }
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < TR; ++i)
#pragma unroll
        for (int j = 0; j < TR; ++j) A[(ty + 16 * i) * LD + tx + 16 * j] = a[i][j];
    __syncthreads();
    // symmetrise, find the largest entry, store as fp16 scaled to a largest entry of one
    float mx = 0.f;
    bool bad = false;
    for (int e = tid; e < D * D; e += PC_THREADS) {
        const int r = e / D, c = e % D;
        const float v = 0.5f * (A[r * LD + c] + A[c * LD + r]);
        bad |= !isfinite(v);
        mx = fmaxf(mx, fabsf(v));
    }
    for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (bad) s_bad = 1;
    if ((tid & 31) == 0) s_red[tid >> 5] = mx;
    __syncthreads();
    mx = 0.f;
    for (int w = 0; w < PC_THREADS / 32; ++w) mx = fmaxf(mx, s_red[w]);
    const bool use_identity = s_bad != 0 || !(mx > 0.f);
    const float sc = use_identity ? 0.f : 1.f / mx;
    __half* dst = minv + ((size_t)u * nb + g) * D * D;
    for (int e = tid; e < D * D; e += PC_THREADS) {
        const int r = e / D, c = e % D;
        const float v = use_identity ? (r == c ? 1.f : 0.f) : 0.5f * (A[r * LD + c] + A[c * LD + r]) * sc;
        dst[e] = __float2half_rn(v);
    }
}

template <int D>
int launch_t(const __nv_bfloat16* k, int B, int Hk, Strides sk, int n, float lambda, int window, float* gram, __half* minv, cudaStream_t st) {
    const int units = B * Hk;
    const int nb = precond_blocks(n), rec = D * D + D;
    const size_t smem_g = sizeof(float) * PC_BLOCK * (D + 1), smem_i = sizeof(float) * (D * (D + 1) + D);
    LLA_CUDA_TRY(cudaFuncSetAttribute(gram_blocks_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_g));
    LLA_CUDA_TRY(cudaFuncSetAttribute(precond_invert_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_i));
    gram_blocks_kernel<D><<<dim3(nb, units), PC_THREADS, smem_g, st>>>(k, gram, n, nb, Hk, sk);
    LLA_CUDA_TRY(cudaGetLastError());
    if (nb > 1) {
        gram_scan_kernel<<<dim3((rec + PC_THREADS - 1) / PC_THREADS, units), PC_THREADS, 0, st>>>(gram, nb, rec);
        LLA_CUDA_TRY(cudaGetLastError());
    }
    precond_invert_kernel<D><<<dim3(nb, units), PC_THREADS, smem_i, st>>>(gram, minv, n, nb, lambda, window);
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

}  // namespace

int precond_blocks(int n) { return (n + PC_BLOCK - 1) / PC_BLOCK; }

size_t precond_gram_bytes(int units, int n, int d) {
    return ((size_t)units * precond_blocks(n) * ((size_t)d * d + d) * sizeof(float) + 255) & ~(size_t)255;
}
size_t precond_minv_bytes(int units, int n, int d) {
    return ((size_t)units * precond_blocks(n) * (size_t)d * d * sizeof(__half) + 255) & ~(size_t)255;
}

int launch_precond(const void* k, int B, int Hk, Strides sk, int n, int d, float lambda, int window, void* gram, void* minv,
                   cudaStream_t st) {
    if (d == 64) return launch_t<64>(static_cast<const __nv_bfloat16*>(k), B, Hk, sk, n, lambda, window, static_cast<float*>(gram),
                                     static_cast<__half*>(minv), st);
    if (d == 128) return launch_t<128>(static_cast<const __nv_bfloat16*>(k), B, Hk, sk, n, lambda, window, static_cast<float*>(gram),
                                       static_cast<__half*>(minv), st);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
