// Direct fp64 solve for the rows that see only a few keys.
//
// For a row with L visible keys and L < head_rows (default 2d) the system Sigma_i rho_i = mu_i of
// Eq. "query_specific" has condition numbers of 1e4..1e5 at the paper's ridge sizes (Sigma_i is
// low rank plus lambda*I while L < d).  fp32 conjugate gradients cannot resolve that, so these few
// rows are computed exactly as Section 2.3 writes them: explicit moments, an LDL^T factorisation
// of the d x d matrix in shared memory, and the intercept of Eq. "lla".  They are 2d/n of the
// rows and about (2d/n)^2 of the pair work.
//
// One thread block per (batch*head, row).  All arithmetic is double precision.
#include "lla_common.cuh"

namespace lla {
namespace {

constexpr int HR_CHUNK = 32;  // keys staged per step of the moment build

template <int D>
struct HrCfg {
    static constexpr int TILES_1D = D / 4;                           // 4x4 register tiles
    static constexpr int TILES = TILES_1D * (TILES_1D + 1) / 2;      // lower triangle incl. diagonal
    // One thread per tile where that fits (136 tiles for D = 64 -> 5 warps).  The factorisation
    // that follows has little parallelism, so small blocks, and more of them per SM, is what
    // keeps the double-precision pipe busy.
    static constexpr int THREADS = D <= 64 ? 160 : 256;
    static constexpr int BLOCKS_PER_SM = D <= 64 ? 6 : 1;
    static constexpr int TILES_PER_THREAD = (TILES + THREADS - 1) / THREADS;
    // shared memory (doubles): the Sigma matrix; the staged keys of the moment build lie over it
    // (the matrix is written only after the build)
    static constexpr int S_DOUBLES = D * (D + 1) > HR_CHUNK * D ? D * (D + 1) : HR_CHUNK * D;
    static constexpr size_t smem_doubles(int lcap) { return (size_t)S_DOUBLES + 2 * D + ((lcap + 1) & ~1) + THREADS / 32 + 1; }
    static constexpr int LDS = D + 1;                                // padded row stride (doubles)
};

template <int HR_THREADS>
__device__ __forceinline__ double block_reduce(double x, bool is_max, double* scratch) {
    // scratch: HR_THREADS/32 + 1 doubles
    for (int off = 16; off > 0; off >>= 1) {
        const double y = __shfl_xor_sync(0xffffffffu, x, off);
        x = is_max ? fmax(x, y) : x + y;
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    if (warp == 0) {
        double t = lane < HR_THREADS / 32 ? scratch[lane] : (is_max ? -INFINITY : 0.0);
        for (int off = 16; off > 0; off >>= 1) {
            const double y = __shfl_xor_sync(0xffffffffu, t, off);
            t = is_max ? fmax(t, y) : t + y;
        }
        if (lane == 0) scratch[HR_THREADS / 32] = t;
    }
    __syncthreads();
    return scratch[HR_THREADS / 32];
}

// dot product of a double vector in shared memory with one row of keys (vector loads, 8 at a time)
template <int D>
__device__ __forceinline__ double dot_row(const double* __restrict__ a, const __nv_bfloat16* __restrict__ kr) {
    double s = 0.0;
#pragma unroll 1
    for (int c = 0; c < D; c += 8) {
        float f[8];
        load8(kr + c, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) s += a[c + e] * (double)f[e];
    }
    return s;
}
template <int D>
__device__ __forceinline__ double dot_row(const double* __restrict__ a, const float* __restrict__ kr) {
    double s = 0.0;
#pragma unroll 1
    for (int c = 0; c < D; c += 4) {
        const float4 f = load4(kr + c);
        s += a[c] * (double)f.x + a[c + 1] * (double)f.y + a[c + 2] * (double)f.z + a[c + 3] * (double)f.w;
    }
    return s;
}


// two consecutive elements (4- or 8-byte aligned) as floats
__device__ __forceinline__ void load2(const __nv_bfloat16* p, float& a, float& b) {
    const uint32_t raw = *reinterpret_cast<const uint32_t*>(p);
    a = __uint_as_float(raw << 16);
    b = __uint_as_float(raw & 0xFFFF0000u);
}
__device__ __forceinline__ void load2(const float* p, float& a, float& b) {
    const float2 f = *reinterpret_cast<const float2*>(p);
    a = f.x;
    b = f.y;
}

template <int D, int DV, typename TIn, typename TOut>
__global__ void __launch_bounds__(HrCfg<D>::THREADS, HrCfg<D>::BLOCKS_PER_SM)
head_rows_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
                 TOut* __restrict__ out, int n, int rows_per_head, int causal, double scale,
                 double lambda, int lcap, float* __restrict__ rho_out, float* __restrict__ stats,
                 int* __restrict__ iters, int* __restrict__ status, const int* __restrict__ lens, int H,
                 const float* __restrict__ lambda_rows, int ridge_mode, int nq, int kv_group,
                 const PagedKv paged, int window, const Strides sq, const Strides sk, const Strides sv, const Strides so) {
    // Prefill (lens == nullptr): block (i, bh) solves row i of head bh; n is the sequence length.
    // Decode (lens != nullptr): block (0, bh) solves the single query of (sequence, head) bh over
    // lens[bh / H] cached keys, but only when that is at most lcap; n is the cache stride Lmax.
    using C = HrCfg<D>;
    constexpr int HR_THREADS = C::THREADS;
    extern __shared__ __align__(16) double smem[];
    double* S = smem;                       // D * LDS (S_DOUBLES reserved)
    double* qd = S + C::S_DOUBLES;          // D
    double* rhs = qd + D;                   // D  (mu, then rho)
    double* w = rhs + D;                    // lcap (scores -> weights -> coefficients)
    double* red = w + ((lcap + 1) & ~1);    // HR_THREADS/32 + 1
    double* zc = S;                         // HR_CHUNK * D  centred keys of the current chunk (over S)

    const int tid = threadIdx.x;
    // blockIdx.x (fastest in launch order) is the head, blockIdx.y counts rows from the last one down:
    // rows with the most keys are the longest blocks and start first, so the tail of the launch is short
    const int bh = blockIdx.x;
    const int i = rows_per_head - 1 - blockIdx.y;   // row index inside the head
    if (i >= rows_per_head) return;
    int L = causal ? (n - nq) + i + 1 : n;    // query row i sits at position n - nq + i
    if (lens) {
        L = visible_keys(lens[bh / H], n, window);
        if (L > lcap) return;               // long caches go through the moment kernel
    }
    const size_t row = lens ? (size_t)bh : (size_t)bh * nq + i;      // row of the contiguous per-row outputs (rho, stats, ...)
    // (debug build: the keys must fit the shared-memory arrays sized for lcap, the row the per-row outputs)
    if (!LLA_IN_BOUNDS(L, lcap + 1, status, 201) || !LLA_IN_BOUNDS(row, (size_t)gridDim.x * (lens ? 1 : nq), status, 202)) return;
    // prefill: q, k, v and out are addressed through their strides; decode keeps its contiguous / paged layout
    const TIn* qrow = lens ? q + row * D : q + sq.at(bh / H, bh % H, i);
    // (decode over a paged cache: the at most lcap <= page_size keys of a directly-solved unit sit in its first page)
    const int kstart = lens ? first_visible_key(lens[bh / H], n, window) : 0;      // sliding-window decode
    const size_t kvrow = kv_row(paged, bh / H, (bh % H) / max(kv_group, 1), H / max(kv_group, 1), n, kstart);
    const int hk = (bh % H) / max(kv_group, 1);
    const TIn* kb = lens ? k + kvrow * D : k + sk.at(bh / H, hk, 0);
    const TIn* vb = lens ? v + kvrow * DV : v + sv.at(bh / H, hk, 0);
    const size_t krs = lens ? (size_t)D : (size_t)sk.r, vrs = lens ? (size_t)DV : (size_t)sv.r;      // row strides of k and v
    TOut* orow = lens ? out + row * DV : out + so.at(bh / H, bh % H, i);

    for (int c = tid; c < D; c += HR_THREADS) qd[c] = (double)to_f32(qrow[c]);
    __syncthreads();

    // scores, their maximum, weights exp(s - m), ridge lambda * exp(-m)
    double lmax = -INFINITY;
    for (int j = tid; j < L; j += HR_THREADS) {
        const double s = dot_row<D>(qd, kb + (size_t)j * krs) * scale;
        w[j] = s;
        lmax = fmax(lmax, s);
    }
    const double m = block_reduce<HR_THREADS>(lmax, true, red);
    double lsum = 0.0;
    for (int j = tid; j < L; j += HR_THREADS) {
        const double e = exp(w[j] - m);
        w[j] = e;
        lsum += e;
    }
    const double omega = block_reduce<HR_THREADS>(lsum, false, red);
    // per-row ridge if given (prefill: [B,H,n]; decode: [B,H]); see lla_ridge_mode for the two frames
    const double lam_i = lambda_rows ? (double)lambda_rows[row] : lambda;
    const double lambda_m = ridge_mode == LLA_RIDGE_PRINTED ? lam_i : lam_i * exp(-m);

    // Rows with at most d keys (and a positive ridge) go through the dual (Gram) form: with Z the
    // L x d matrix of centred keys, w_j (1 - z_j . rho) = lambda' alpha_j where
    // (Z Z^T + lambda' diag(1/w)) alpha = 1  --  an L x L system instead of d x d, free of the
    // cancellation in 1 - z . rho, and rho = Z^T alpha.  The system is padded to a multiple of 8 with
    // identity rows.
    double csum = 0.0, rho_val = 0.0;
    bool bad = false;
    const bool dual = L <= D && lambda_m > 0.0;          // block-uniform
    const int Lp = (L + 7) & ~7;                         // dual: system size padded to the panel width
    // lower-triangular 4x4 register tiles of the matrix being built (Sigma, or the Gram matrix):
    // tile index -> (row tile, column tile); interleaved: rows tr + T1 a, columns tc + T1 b
    const int T1 = dual ? Lp / 4 : C::TILES_1D, ntiles = T1 * (T1 + 1) / 2;
    double acc[C::TILES_PER_THREAD][4][4];
    int tr[C::TILES_PER_THREAD], tc[C::TILES_PER_THREAD];
#pragma unroll
    for (int t = 0; t < C::TILES_PER_THREAD; ++t) {
        const int tile = tid + t * HR_THREADS;
        int r = 0;
        if (tile < ntiles) {
            r = (int)((sqrt(8.0 * tile + 1.0) - 1.0) * 0.5);
            while ((r + 1) * (r + 2) / 2 <= tile) ++r;
            while (r * (r + 1) / 2 > tile) --r;
        }
        tr[t] = tile < ntiles ? r : -1;
        tc[t] = tile < ntiles ? tile - r * (r + 1) / 2 : 0;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[t][a][b] = 0.0;
    }
    if (dual) {
        const int LZ = Lp + 1;                            // odd row stride of the staged keys
        double* zt = S;                                   // zt[c * LZ + j] = k_j[c] - q[c]  (over S: D * LZ <= S_DOUBLES)
        for (int e = tid; e < Lp * D; e += HR_THREADS) {
            const int j = e / D, c = e - j * D;
            zt[c * LZ + j] = j < L ? (double)to_f32(kb[(size_t)j * krs + c]) - qd[c] : 0.0;
        }
        __syncthreads();
        // Gram matrix
#pragma unroll
        for (int t = 0; t < C::TILES_PER_THREAD; ++t) {
            if (tr[t] < 0) continue;
            for (int c = 0; c < D; ++c) {
                double zj[4], zl[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    zj[x] = zt[c * LZ + tr[t] + T1 * x];
                    zl[x] = zt[c * LZ + tc[t] + T1 * x];
                }
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) acc[t][x][y] += zj[x] * zl[y];
            }
        }
        __syncthreads();       // the staged keys (lying over S) are no longer read
#pragma unroll
        for (int t = 0; t < C::TILES_PER_THREAD; ++t) {
            if (tr[t] < 0) continue;
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const int r = tr[t] + T1 * x, c = tc[t] + T1 * y;
                    // diagonal: ridge / weight for live keys (weights clamped away from 0), 1 for padding
                    const double dg = r < L ? lambda_m / fmax(w[r], 1e-290) : 1.0;
                    if (c <= r) S[r * C::LDS + c] = acc[t][x][y] + (r == c ? dg : 0.0);
                    else if (tr[t] != tc[t]) S[c * C::LDS + r] = acc[t][x][y];
                }
        }
        for (int j = tid; j < Lp; j += HR_THREADS) rhs[j] = j < L ? 1.0 : 0.0;
        __syncthreads();
        bad = !block_ldlt_solve<D>(S, C::LDS, rhs, Lp);
        // coefficients c_j = lambda' alpha_j
        for (int j = tid; j < L; j += HR_THREADS) {
            const double cj = lambda_m * rhs[j];
            w[j] = cj;
            csum += cj;
        }
        if (rho_out && tid < D) {                         // rho = Z^T alpha
            double acc_r = 0.0;
            for (int j = 0; j < L; ++j) acc_r += rhs[j] * ((double)to_f32(kb[(size_t)j * krs + tid]) - qd[tid]);
            rho_val = acc_r;
        }
    } else {
        // moments: Sigma and mu
        double mu_acc = 0.0;  // thread tid < D owns mu[tid]
        // The keys of a chunk are fetched (element pairs, coalesced) one chunk ahead, so the global-load
        // latency hides behind the accumulation of the chunk before.
        constexpr int PAIRS = (HR_CHUNK * D / 2 + HR_THREADS - 1) / HR_THREADS;
        float pre[PAIRS][2];
        auto fetch = [&](int j0) {
            const int np = min(HR_CHUNK, L - j0) * (D / 2);
    #pragma unroll
            for (int u = 0; u < PAIRS; ++u) {
                const int pi = tid + HR_THREADS * u;
                if (pi < np) load2(kb + (size_t)(j0 + (2 * pi) / D) * krs + (2 * pi) % D, pre[u][0], pre[u][1]);
            }
        };
        fetch(0);
        for (int j0 = 0; j0 < L; j0 += HR_CHUNK) {
            const int jn = min(HR_CHUNK, L - j0);
            __syncthreads();
    #pragma unroll
            for (int u = 0; u < PAIRS; ++u) {
                const int pi = tid + HR_THREADS * u;
                if (pi < jn * (D / 2)) {
                    const int c = (2 * pi) % D;
                    *reinterpret_cast<double2*>(zc + 2 * pi) = make_double2((double)pre[u][0] - qd[c], (double)pre[u][1] - qd[c + 1]);
                }
            }
            __syncthreads();
            if (j0 + HR_CHUNK < L) fetch(j0 + HR_CHUNK);
            if (tid < D)
                for (int jj = 0; jj < jn; ++jj) mu_acc += w[j0 + jj] * zc[jj * D + tid];
    #pragma unroll
            for (int t = 0; t < C::TILES_PER_THREAD; ++t) {
                if (tr[t] < 0) continue;
                // interleaved 4x4 tile: rows tr + T1*a, columns tc + T1*b, so that neighbouring threads
                // read neighbouring doubles (no shared-memory bank conflicts)
                const int r0 = tr[t], c0 = tc[t];
                for (int jj = 0; jj < jn; ++jj) {
                    const double wj = w[j0 + jj];
                    double zr[4], zcv[4];
    #pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        zr[a] = wj * zc[jj * D + r0 + C::TILES_1D * a];
                        zcv[a] = zc[jj * D + c0 + C::TILES_1D * a];
                    }
    #pragma unroll
                    for (int a = 0; a < 4; ++a)
    #pragma unroll
                        for (int b = 0; b < 4; ++b) acc[t][a][b] += zr[a] * zcv[b];
                }
            }
        }
        __syncthreads();   // the staged keys (lying over S) are no longer read
    #pragma unroll
        for (int t = 0; t < C::TILES_PER_THREAD; ++t) {
            if (tr[t] < 0) continue;
    #pragma unroll
            for (int a = 0; a < 4; ++a)
    #pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int r = tr[t] + C::TILES_1D * a, c = tc[t] + C::TILES_1D * b;
                    if (c <= r) S[r * C::LDS + c] = acc[t][a][b] + (r == c ? lambda_m : 0.0);
                    else if (tr[t] != tc[t]) S[c * C::LDS + r] = acc[t][a][b];   // mirror of tile (tc, tr)
                }
        }
        if (tid < D) rhs[tid] = mu_acc;
        __syncthreads();

        // rhs <- Sigma^{-1} mu (LDL^T in shared memory)
        bad = !block_ldlt_solve<D>(S, C::LDS, rhs);

        // coefficients c_j = w_j (1 - z_j . rho) and their sum (= omega - mu . rho)
        double qrho = 0.0;
        for (int c = 0; c < D; ++c) qrho += qd[c] * rhs[c];
        for (int j = tid; j < L; j += HR_THREADS) {
            const double t = dot_row<D>(rhs, kb + (size_t)j * krs) - qrho;
            const double cj = w[j] * (1.0 - t);
            w[j] = cj;
            csum += cj;
        }
        if (tid < D) rho_val = rhs[tid];
    }
    const double denom = block_reduce<HR_THREADS>(csum, false, red);
    for (int c = tid; c < DV; c += HR_THREADS) {
        double o = 0.0;
        for (int j = 0; j < L; ++j) o += w[j] * (double)to_f32(vb[(size_t)j * vrs + c]);
        store_out(orow + c, (float)(o / denom));
    }
    if (rho_out && tid < D) rho_out[row * D + tid] = (float)rho_val;
    if (tid == 0) {
        if (stats) {
            stats[row * 3 + 0] = (float)m;
            stats[row * 3 + 1] = (float)omega;
            stats[row * 3 + 2] = (float)denom;
        }
        if (iters) iters[row] = -1;
        if (bad && status) atomicAdd(status + LLA_STATUS_BAD_PIVOT, 1);
    }
}

template <int D, typename TIn, typename TOut>
int launch_t(const ForwardArgs& a, int rows_per_head, int lcap) {
    using C = HrCfg<D>;
    const size_t smem = sizeof(double) * C::smem_doubles(lcap);
    auto kern = head_rows_kernel<D, D, TIn, TOut>;
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    dim3 grid(a.B * a.H, rows_per_head);
    kern<<<grid, C::THREADS, smem, a.stream>>>(
        (const TIn*)a.q, (const TIn*)a.k, (const TIn*)a.v, (TOut*)a.out, a.n, rows_per_head, a.causal,
        (double)a.scale, (double)a.lambda, lcap, a.rho, a.stats, a.iters, a.status, nullptr, a.H, a.lambda_rows,
        a.ridge_mode, a.nq, a.kv_group, PagedKv{nullptr, 0, 0, 0}, 0, a.sq, a.sk, a.sv, a.so);
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

template <int D, typename TIn, typename TOut>
int launch_decode_t(const DecodeArgs& a, int lcap) {
    using C = HrCfg<D>;
    const size_t smem = sizeof(double) * C::smem_doubles(lcap);
    auto kern = head_rows_kernel<D, D, TIn, TOut>;
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    dim3 grid(a.B * a.H, 1);
    kern<<<grid, C::THREADS, smem, a.stream>>>(
        (const TIn*)a.q, (const TIn*)a.kcache, (const TIn*)a.vcache, (TOut*)a.out, a.Lmax, 1, 0,
        (double)a.scale, (double)a.lambda, lcap, nullptr, nullptr, nullptr, a.status, a.lens, a.H, a.lambda_units,
        a.ridge_mode, 1, a.kv_group, a.paged, a.window, Strides{0, 0, 0}, Strides{0, 0, 0}, Strides{0, 0, 0}, Strides{0, 0, 0});
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

template <int D>
int launch_decode_d(const DecodeArgs& a, int lcap) {
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_BF16)
        return launch_decode_t<D, __nv_bfloat16, __nv_bfloat16>(a, lcap);
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_F32)
        return launch_decode_t<D, __nv_bfloat16, float>(a, lcap);
    if (a.in_dtype == LLA_F32 && a.out_dtype == LLA_F32)
        return launch_decode_t<D, float, float>(a, lcap);
    return LLA_ERR_UNSUPPORTED;
}

template <int D>
int launch_d(const ForwardArgs& a, int rows_per_head, int lcap) {
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_BF16)
        return launch_t<D, __nv_bfloat16, __nv_bfloat16>(a, rows_per_head, lcap);
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_F32)
        return launch_t<D, __nv_bfloat16, float>(a, rows_per_head, lcap);
    if (a.in_dtype == LLA_F32 && a.out_dtype == LLA_F32)
        return launch_t<D, float, float>(a, rows_per_head, lcap);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace

// Number of leading rows per head handled directly (causal), or n / 0 (non-causal).
int head_rows_count(const ForwardArgs& a) {
    if (a.head_rows <= 0) return 0;
    if (a.causal) {     // query row i sees n - nq + i + 1 keys
        const int rows = a.head_rows - 1 - (a.n - a.nq);
        return rows < 0 ? 0 : (rows > a.nq ? a.nq : rows);
    }
    return a.n < a.head_rows ? a.nq : 0;
}

int launch_head_rows(const ForwardArgs& a) {
    const int rows = head_rows_count(a);
    if (rows <= 0) return LLA_OK;
    const int lcap = a.causal ? (a.n - a.nq) + rows : a.n;
    if (a.d != a.dv) return LLA_ERR_UNSUPPORTED;
    switch (a.d) {
        case 16: return launch_d<16>(a, rows, lcap);
        case 64: return launch_d<64>(a, rows, lcap);
        case 128: return launch_d<128>(a, rows, lcap);
        default: return LLA_ERR_UNSUPPORTED;
    }
}

// Decode: (sequence, head) pairs whose cache holds at most head_rows - 1 keys.
int launch_head_rows_decode(const DecodeArgs& a) {
    if (a.head_rows <= 1) return LLA_OK;
    const int lcap = a.head_rows - 1;
    switch (a.d) {
        case 16: return launch_decode_d<16>(a, lcap);
        case 64: return launch_decode_d<64>(a, lcap);
        case 128: return launch_decode_d<128>(a, lcap);
        default: return LLA_ERR_UNSUPPORTED;
    }
}

}  // namespace lla
