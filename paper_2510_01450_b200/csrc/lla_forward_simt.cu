// LLA forward on CUDA cores, fp32 arithmetic: the path for fp32 tensors and for every shape the
// tensor-core kernel is not compiled for.
//
// Structure follows Algorithm 1 (three sweeps over the key blocks per query block) with the
// solver of Algorithm 2 in between, in the weighted-mean-centred form of Eq. "lla_decomp":
//
//   sweep 1   m_i = max_j s_ij,  w_ij = exp(s_ij - m_i),  omega_i = sum_j w_ij,
//             kbar_i = sum_j w_ij k_j / omega_i                      (Algorithm 1, first loop)
//   solve     C_i y_i = kbar_i - q_i  by conjugate gradients, where
//             C_i x = (1/omega_i) sum_j w_ij (k_j.x - kbar_i.x) k_j + (lambda e^{-m_i}/omega_i) x
//             one sweep over the keys per iteration, weights recomputed on the fly, rows frozen
//             once |r| <= tol |b| (Algorithm 2: matrix-free product, active mask)
//   sweep 3   o_i = sum_j w_ij (1 - (k_j - kbar_i).y_i) v_j / sum_j w_ij (1 - (k_j - kbar_i).y_i)
//
// C_i is Sigma_i / omega_i with the rank-one term of the weighted key mean projected out
// (Sherman-Morrison): rho_i = y_i / g_i and delta_i = omega_i / g_i with g_i = 1 + (kbar_i-q_i).y_i,
// and 1 - z_ij.rho_i = (1 - (k_j - kbar_i).y_i) / g_i, so the output equals Eq. "lla" exactly while
// the solve loses the outlier eigenvalue omega_i (1/d + |q_i|^2) and the final coefficients are
// no longer a small difference of O(1) terms.  The ridge is lambda * exp(-m_i) because the weights
// carry the factor exp(-m_i): only the joint scaling of weights and ridge leaves Eq. "lla" unchanged.
//
// Thread mapping: TPR consecutive lanes share one query row, each owning D/TPR columns of every
// row vector (q, kbar, x, r, p, C p) in registers; dot products finish with TPR-wide xor shuffles.
// Key (and value) tiles are staged in shared memory as fp32 and read as broadcast float4s.
#include "lla_common.cuh"

namespace lla {
namespace {

constexpr int FS_THREADS = 256;
constexpr int FS_BC = 64;  // keys per shared-memory tile

template <int TPR>
__device__ __forceinline__ float row_sum(float x) {
#pragma unroll
    for (int off = 1; off < TPR; off <<= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
}

template <bool ACCURATE>
__device__ __forceinline__ float exp_w(float x) {
    return ACCURATE ? expf(x) : __expf(x);
}

template <int D, typename TIn>
__device__ __forceinline__ void load_tile(float* __restrict__ dst, const TIn* __restrict__ src,
                                          int j0, int n, long long row_stride) {
    // dst[FS_BC][D] <- src rows j0 .. j0+FS_BC-1 (zero beyond n); rows are row_stride elements apart
    constexpr int VEC = FS_BC * D / 4;
    for (int e = threadIdx.x; e < VEC; e += FS_THREADS) {
        const int jj = e / (D / 4), f = e - jj * (D / 4);
        float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j0 + jj < n) val = load4(src + (size_t)(j0 + jj) * row_stride + 4 * f);
        reinterpret_cast<float4*>(dst)[e] = val;
    }
}

template <int D, int DV, int TPR, typename TIn, typename TOut>
__global__ void __launch_bounds__(FS_THREADS)
forward_simt_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
                    TOut* __restrict__ out, int n, int causal, float scale, float lambda,
                    int head_rows, int max_iters, float tol, int first_tile,
                    float* __restrict__ rho_out, float* __restrict__ stats, int* __restrict__ iters_out,
                    int* __restrict__ status, const float* __restrict__ lambda_rows, int ridge_mode, int nq, int H, int kv_group, int window,
                    const Strides sq, const Strides sk, const Strides sv, const Strides so) {
    constexpr int ROWS = FS_THREADS / TPR;
    constexpr int NG = D / (4 * TPR);    // float4 groups per thread (keys)
    constexpr int NGV = DV / (4 * TPR);  // float4 groups per thread (values)
    constexpr bool ACCURATE = sizeof(TIn) == 4;
    extern __shared__ float4 smem_f4[];
    float* Ks = reinterpret_cast<float*>(smem_f4);
    float* Vs = Ks + FS_BC * D;

    const int bh = blockIdx.y;
    // heaviest (latest) query tiles first
    const int tile = first_tile + (gridDim.x - 1 - blockIdx.x);
    const int r0 = tile * ROWS;
    const int lr = threadIdx.x % TPR;
    const int row = r0 + threadIdx.x / TPR;
    const int off = n - nq;                             // query row r sits at position off + r
    const int L = causal ? off + row + 1 : n;           // visible keys of this row
    const bool row_ok = row < nq && L >= head_rows;     // other rows: out of range or solved directly
    const int jend = causal ? min(n, off + r0 + ROWS) : n;   // keys this block must sweep
    // sliding window (causal only): a row sees keys jlo .. L - 1, the block starts at its first row's window
    const int jlo = (causal && window > 0) ? max(0, L - window) : 0;
    const int jbeg = (causal && window > 0) ? max(0, off + r0 + 1 - window) / FS_BC * FS_BC : 0;
    const int hk = (bh % H) / max(kv_group, 1);             // key/value head of this query head
    const TIn* kb = k + sk.at(bh / H, hk, 0);
    const TIn* vb = v + sv.at(bh / H, hk, 0);

    float4 qv[NG], kbar[NG];
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        qv[g] = row < nq ? load4(q + sq.at(bh / H, bh % H, row) + 4 * (g * TPR + lr))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
        kbar[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    }

    // ---- sweep 1: running maximum, omega, weighted key sum (Algorithm 1, first loop) ----
    float m = -INFINITY, omega = 0.f;
    for (int j0 = jbeg; j0 < jend; j0 += FS_BC) {
        __syncthreads();
        load_tile<D>(Ks, kb, j0, n, sk.r);
        __syncthreads();
        const int lim = row_ok ? min(FS_BC, L - j0) : 0;
        const int wlim = __reduce_max_sync(0xffffffffu, lim);
        for (int jj = 0; jj < wlim; ++jj) {
            const float4* kr = reinterpret_cast<const float4*>(Ks + jj * D);
            float4 kv[NG];
            float s = 0.f;
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                kv[g] = kr[g * TPR + lr];
                s += qv[g].x * kv[g].x + qv[g].y * kv[g].y + qv[g].z * kv[g].z + qv[g].w * kv[g].w;
            }
            s = row_sum<TPR>(s) * scale;
            if (jj < lim && jj >= jlo - j0) {
                if (s > m) {
                    const float c = exp_w<ACCURATE>(m - s);
                    omega *= c;
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        kbar[g].x *= c; kbar[g].y *= c; kbar[g].z *= c; kbar[g].w *= c;
                    }
                    m = s;
                }
                const float w = exp_w<ACCURATE>(s - m);
                omega += w;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    kbar[g].x += w * kv[g].x; kbar[g].y += w * kv[g].y;
                    kbar[g].z += w * kv[g].z; kbar[g].w += w * kv[g].w;
                }
            }
        }
    }
    const float inv_omega = row_ok ? 1.f / omega : 0.f;
    const float lam_i = (lambda_rows && row < nq) ? lambda_rows[(size_t)bh * nq + row] : lambda;
    const float ridge = row_ok ? (ridge_mode == LLA_RIDGE_PRINTED ? lam_i : lam_i * exp_w<ACCURATE>(-m)) * inv_omega : 0.f;

    // ---- conjugate gradients on C y = kbar - q (Algorithm 2) ----
    float4 x[NG], r[NG], p[NG];
    float rr = 0.f;
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        kbar[g].x *= inv_omega; kbar[g].y *= inv_omega; kbar[g].z *= inv_omega; kbar[g].w *= inv_omega;
        x[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        r[g] = make_float4(kbar[g].x - qv[g].x, kbar[g].y - qv[g].y, kbar[g].z - qv[g].z, kbar[g].w - qv[g].w);
        if (!row_ok) r[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        p[g] = r[g];
        rr += r[g].x * r[g].x + r[g].y * r[g].y + r[g].z * r[g].z + r[g].w * r[g].w;
    }
    rr = row_sum<TPR>(rr);
    const float stop = tol * tol * rr;
    bool active = row_ok && rr > 0.f;
    int its = 0;
    for (int t = 0; t < max_iters; ++t) {
        active = active && rr > stop;
        if (!__syncthreads_or(active)) break;
        float pk = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g)
            pk += kbar[g].x * p[g].x + kbar[g].y * p[g].y + kbar[g].z * p[g].z + kbar[g].w * p[g].w;
        const float abar = row_sum<TPR>(pk);
        float4 acc[NG];
#pragma unroll
        for (int g = 0; g < NG; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j0 = jbeg; j0 < jend; j0 += FS_BC) {
            __syncthreads();
            load_tile<D>(Ks, kb, j0, n, sk.r);
            __syncthreads();
            const int lim = active ? min(FS_BC, L - j0) : 0;
            const int wlim = __reduce_max_sync(0xffffffffu, lim);
            for (int jj = 0; jj < wlim; ++jj) {
                const float4* kr = reinterpret_cast<const float4*>(Ks + jj * D);
                float4 kv[NG];
                float s = 0.f, a = 0.f;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    kv[g] = kr[g * TPR + lr];
                    s += qv[g].x * kv[g].x + qv[g].y * kv[g].y + qv[g].z * kv[g].z + qv[g].w * kv[g].w;
                    a += p[g].x * kv[g].x + p[g].y * kv[g].y + p[g].z * kv[g].z + p[g].w * kv[g].w;
                }
                s = row_sum<TPR>(s) * scale;
                a = row_sum<TPR>(a);
                const float u = (jj < lim && jj >= jlo - j0) ? exp_w<ACCURATE>(s - m) * (a - abar) : 0.f;
#pragma unroll
                for (int g = 0; g < NG; ++g) {
                    acc[g].x += u * kv[g].x; acc[g].y += u * kv[g].y;
                    acc[g].z += u * kv[g].z; acc[g].w += u * kv[g].w;
                }
            }
        }
        float pAp = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            acc[g].x = acc[g].x * inv_omega + ridge * p[g].x;
            acc[g].y = acc[g].y * inv_omega + ridge * p[g].y;
            acc[g].z = acc[g].z * inv_omega + ridge * p[g].z;
            acc[g].w = acc[g].w * inv_omega + ridge * p[g].w;
            pAp += p[g].x * acc[g].x + p[g].y * acc[g].y + p[g].z * acc[g].z + p[g].w * acc[g].w;
        }
        pAp = row_sum<TPR>(pAp);
        if (active && !(pAp > 0.f)) active = false;   // breakdown guard: keep the current iterate
        const float alpha = active ? rr / pAp : 0.f;
        float rr2 = 0.f;
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            x[g].x += alpha * p[g].x; x[g].y += alpha * p[g].y; x[g].z += alpha * p[g].z; x[g].w += alpha * p[g].w;
            r[g].x -= alpha * acc[g].x; r[g].y -= alpha * acc[g].y; r[g].z -= alpha * acc[g].z; r[g].w -= alpha * acc[g].w;
            rr2 += r[g].x * r[g].x + r[g].y * r[g].y + r[g].z * r[g].z + r[g].w * r[g].w;
        }
        rr2 = row_sum<TPR>(rr2);
        if (active) {
            const float beta = rr2 / rr;
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                p[g].x = r[g].x + beta * p[g].x; p[g].y = r[g].y + beta * p[g].y;
                p[g].z = r[g].z + beta * p[g].z; p[g].w = r[g].w + beta * p[g].w;
            }
            rr = rr2;
            ++its;
        }
    }
    const bool at_cap = active && rr > stop;

    // ---- sweep 3: coefficients and output (Algorithm 1, last loop) ----
    float yk = 0.f, yb = 0.f;
#pragma unroll
    for (int g = 0; g < NG; ++g) {
        yk += kbar[g].x * x[g].x + kbar[g].y * x[g].y + kbar[g].z * x[g].z + kbar[g].w * x[g].w;
        yb += (kbar[g].x - qv[g].x) * x[g].x + (kbar[g].y - qv[g].y) * x[g].y +
              (kbar[g].z - qv[g].z) * x[g].z + (kbar[g].w - qv[g].w) * x[g].w;
    }
    const float ybar = row_sum<TPR>(yk);
    const float gfac = 1.f + row_sum<TPR>(yb);
    float4 o[NGV];
#pragma unroll
    for (int g = 0; g < NGV; ++g) o[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (int j0 = jbeg; j0 < jend; j0 += FS_BC) {
        __syncthreads();
        load_tile<D>(Ks, kb, j0, n, sk.r);
        load_tile<DV>(Vs, vb, j0, n, sv.r);
        __syncthreads();
        const int lim = row_ok ? min(FS_BC, L - j0) : 0;
        const int wlim = __reduce_max_sync(0xffffffffu, lim);
        for (int jj = 0; jj < wlim; ++jj) {
            const float4* kr = reinterpret_cast<const float4*>(Ks + jj * D);
            const float4* vr = reinterpret_cast<const float4*>(Vs + jj * DV);
            float s = 0.f, a = 0.f;
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                const float4 kv = kr[g * TPR + lr];
                s += qv[g].x * kv.x + qv[g].y * kv.y + qv[g].z * kv.z + qv[g].w * kv.w;
                a += x[g].x * kv.x + x[g].y * kv.y + x[g].z * kv.z + x[g].w * kv.w;
            }
            s = row_sum<TPR>(s) * scale;
            a = row_sum<TPR>(a);
            const float c = (jj < lim && jj >= jlo - j0) ? exp_w<ACCURATE>(s - m) * (1.f - (a - ybar)) : 0.f;
            den += c;
#pragma unroll
            for (int g = 0; g < NGV; ++g) {
                const float4 vv = vr[g * TPR + lr];
                o[g].x += c * vv.x; o[g].y += c * vv.y; o[g].z += c * vv.z; o[g].w += c * vv.w;
            }
        }
    }
    if (row_ok) {
        const float inv_den = 1.f / den;
        const size_t rowi = (size_t)bh * nq + row;
        if (!LLA_IN_BOUNDS(rowi, (size_t)gridDim.x * nq, status, 301)) return;
        TOut* orow = out + so.at(bh / H, bh % H, row);
#pragma unroll
        for (int g = 0; g < NGV; ++g) {
            const int c0 = 4 * (g * TPR + lr);
            store_out(orow + c0 + 0, o[g].x * inv_den);
            store_out(orow + c0 + 1, o[g].y * inv_den);
            store_out(orow + c0 + 2, o[g].z * inv_den);
            store_out(orow + c0 + 3, o[g].w * inv_den);
        }
        if (rho_out) {
            const float ig = 1.f / gfac;
#pragma unroll
            for (int g = 0; g < NG; ++g)
                reinterpret_cast<float4*>(rho_out + rowi * D)[g * TPR + lr] =
                    make_float4(x[g].x * ig, x[g].y * ig, x[g].z * ig, x[g].w * ig);
        }
        if (lr == 0) {
            if (stats) {
                stats[rowi * 3 + 0] = m;
                stats[rowi * 3 + 1] = omega;
                stats[rowi * 3 + 2] = omega / gfac;
            }
            if (iters_out) iters_out[rowi] = its;
            if (status) {
                if (at_cap) atomicAdd(status + LLA_STATUS_ROWS_AT_CAP, 1);
                atomicAdd(status + LLA_STATUS_ITER_SUM, its);
            }
        }
    }
}

template <int D, int TPR, typename TIn, typename TOut>
int launch_t(const ForwardArgs& a) {
    constexpr int ROWS = FS_THREADS / TPR;
    const int hr = head_rows_count(a);
    if (!a.causal && hr >= a.nq) return LLA_OK;  // every row was solved directly
    // causal: rows 0..hr-1 are done elsewhere; skip query tiles that hold only such rows
    const int first_tile = a.causal ? hr / ROWS : 0;
    const int tiles = (a.nq + ROWS - 1) / ROWS - first_tile;
    if (tiles <= 0) return LLA_OK;
    const size_t smem = sizeof(float) * (size_t)FS_BC * (D + D);
    auto kern = forward_simt_kernel<D, D, TPR, TIn, TOut>;
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid(tiles, a.B * a.H);
    kern<<<grid, FS_THREADS, smem, a.stream>>>(
        (const TIn*)a.q, (const TIn*)a.k, (const TIn*)a.v, (TOut*)a.out, a.n, a.causal, a.scale,
        a.lambda, a.head_rows > 0 ? a.head_rows : 0, a.max_iters, a.tol, first_tile, a.rho, a.stats,
        a.iters, a.status, a.lambda_rows, a.ridge_mode, a.nq, a.H, a.kv_group, a.window, a.sq, a.sk, a.sv, a.so);
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

template <int D, int TPR>
int launch_d(const ForwardArgs& a) {
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_BF16)
        return launch_t<D, TPR, __nv_bfloat16, __nv_bfloat16>(a);
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_F32)
        return launch_t<D, TPR, __nv_bfloat16, float>(a);
    if (a.in_dtype == LLA_F32 && a.out_dtype == LLA_F32)
        return launch_t<D, TPR, float, float>(a);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace

int launch_forward_simt(const ForwardArgs& a) {
    if (a.d != a.dv) return LLA_ERR_UNSUPPORTED;
    switch (a.d) {
        case 16: return launch_d<16, 4>(a);
        case 64: return launch_d<64, 4>(a);
        case 128: return launch_d<128, 8>(a);
        default: return LLA_ERR_UNSUPPORTED;
    }
}

}  // namespace lla
