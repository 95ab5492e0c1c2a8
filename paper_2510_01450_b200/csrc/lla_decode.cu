// LLA single-query decode over a KV cache (Eq. "lla" at one row per (sequence, head)).
//
// Decode is bound by reading the cache once, so the keys and values are streamed a single time
// and folded into weighted moments about the origin,
//     omega = sum_j w_j,  a = sum_j w_j k_j,  c = sum_j w_j v_j,
//     M = sum_j w_j k_j k_j^T (d x d),  N = sum_j w_j v_j k_j^T (dv x d),       w_j = exp(s_j - m),
// with a running maximum m (rescaling the accumulators when it grows, as in Algorithm 1's first
// loop).  The centred quantities of Eq. "lla_decomp" follow without touching the cache again:
//     kbar = a/omega, vbar = c/omega, C = M/omega - kbar kbar^T + (lambda e^{-m}/omega) I,
//     S_vk = N/omega - vbar kbar^T,   o = vbar + S_vk C^{-1} (q - kbar),
// which equals Eq. "lla" (optimal slope W = S_vk C^{-1}).  The d x d solve is done once per
// (sequence, head) in double precision.  Long caches can be cut into `splits` key ranges whose
// partial moments are merged by a second kernel (each part carries its own maximum).
#include "lla_common.cuh"

namespace lla {
namespace {

constexpr int DC_THREADS = 256;
constexpr int DC_BK = 32;  // keys per shared-memory tile

template <int D>
struct DcCfg {
    static constexpr int T1 = D / 4;                                  // 4x4 tiles per side
    static constexpr int TPT = (T1 * T1 + DC_THREADS - 1) / DC_THREADS;  // tiles per thread per matrix
    static constexpr int PART_FLOATS = 2 * D * D + 2 * D + 4;         // M, N, a, c, omega, m, 2 pad (16-byte rows)
};

// Solve and emit one output row from moments held in shared memory (doubles).
//   Md: M (becomes C), lower triangle used, row stride D+1;  Nd: N as float, row stride D
//   a, c: first moments; returns through out[dv]
template <int D, typename TOut>
__device__ void finalize_row(double* Md, const float* Nd, double* a, double* c, double omega, double m,
                             const double* qd, double lambda, int ridge_mode, TOut* out, int* status) {
    const int tid = threadIdx.x;
    constexpr int LDS = D + 1;
    const double inv = 1.0 / omega;
    const double ridge = (ridge_mode == LLA_RIDGE_PRINTED ? lambda : lambda * exp(-m)) * inv;
    __syncthreads();
    for (int e = tid; e < D * D; e += DC_THREADS) {
        const int r = e / D, cc = e - r * D;
        if (cc <= r) Md[r * LDS + cc] = Md[r * LDS + cc] * inv - (a[r] * inv) * (a[cc] * inv) + (r == cc ? ridge : 0.0);
    }
    __syncthreads();
    // a <- kbar, c <- vbar; the right-hand side q - kbar lives in the D doubles that follow c
    double* rhs = c + D;
    for (int e = tid; e < D; e += DC_THREADS) {
        a[e] *= inv;
        c[e] *= inv;
        rhs[e] = qd[e] - a[e];
    }
    const bool ok = block_ldlt_solve<D>(Md, LDS, rhs);
    for (int e = tid; e < D; e += DC_THREADS) {   // dv == d
        double o = c[e];
        for (int f = 0; f < D; ++f) o += ((double)Nd[e * D + f] * inv - c[e] * a[f]) * rhs[f];
        store_out(out + e, (float)o);
    }
    if (!ok && tid == 0 && status) atomicAdd(status + LLA_STATUS_BAD_PIVOT, 1);
}

template <int D, typename TIn, typename TOut>
__global__ void __launch_bounds__(DC_THREADS)
decode_moments_kernel(const TIn* __restrict__ q, const TIn* __restrict__ kcache, const TIn* __restrict__ vcache,
                      const int* __restrict__ lens, TOut* __restrict__ out, int H, int Lmax, float scale,
                      float lambda, int splits, int head_rows, float* __restrict__ parts, int* __restrict__ status,
                      const float* __restrict__ lambda_units, int ridge_mode, int kv_group, const PagedKv paged, int window) {
    using C = DcCfg<D>;
    constexpr bool ACCURATE = sizeof(TIn) == 4;
    extern __shared__ double smem_d[];
    // streaming phase: fp32 tiles; finalize phase (splits == 1): doubles over the same memory
    float* Ks = reinterpret_cast<float*>(smem_d);   // DC_BK * D
    float* Vs = Ks + DC_BK * D;                     // DC_BK * D
    float* sc = Vs + DC_BK * D;                     // DC_BK scores
    float* qs = sc + DC_BK;                         // D

    const int tid = threadIdx.x;
    const int bh = blockIdx.y, part = blockIdx.x;
    const int b = bh / H;
    const int start = first_visible_key(lens[b], Lmax, window);     // sliding window: keys start .. start + L - 1
    const int L = visible_keys(lens[b], Lmax, window);
    if (L < head_rows) return;   // short caches are solved directly by the fp64 kernel
    const int chunk = ((L + splits - 1) / splits + DC_BK - 1) / DC_BK * DC_BK;
    const int jbeg = part * chunk, jend = min(L, jbeg + chunk);
    const int hkv = H / max(kv_group, 1), kvl = (bh % H) / max(kv_group, 1);

    for (int e = tid; e < D; e += DC_THREADS) qs[e] = to_f32(q[(size_t)bh * D + e]);

    float accM[C::TPT][4][4], accN[C::TPT][4][4];
#pragma unroll
    for (int t = 0; t < C::TPT; ++t)
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) { accM[t][x][y] = 0.f; accN[t][x][y] = 0.f; }
    float first = 0.f;   // tid < D: a[tid];  D <= tid < 2D: c[tid-D]
    float omega = 0.f, m = -INFINITY;

    for (int j0 = jbeg; j0 < jend; j0 += DC_BK) {
        const int jn = min(DC_BK, jend - j0);
        // a tile never straddles a page (page_size is a multiple of the tile, j0 of the tile)
        const size_t row0 = kv_row(paged, b, kvl, hkv, Lmax, start + j0);
        const TIn* kb = kcache + row0 * D;
        const TIn* vb = vcache + row0 * D;
        __syncthreads();
        for (int e = tid; e < DC_BK * D / 4; e += DC_THREADS) {
            const int jj = e / (D / 4), f = e - jj * (D / 4);
            float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
            if (jj < jn) {
                kv = load4(kb + (size_t)jj * D + 4 * f);
                vv = load4(vb + (size_t)jj * D + 4 * f);
            }
            reinterpret_cast<float4*>(Ks)[e] = kv;
            reinterpret_cast<float4*>(Vs)[e] = vv;
        }
        __syncthreads();
        {   // scores: 8 lanes per key
            const int jj = tid >> 3, l8 = tid & 7;
            float s = 0.f;
            for (int cidx = l8; cidx < D; cidx += 8) s += qs[cidx] * Ks[jj * D + cidx];
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            s += __shfl_xor_sync(0xffffffffu, s, 4);
            if (l8 == 0) sc[jj] = jj < jn ? s * scale : -INFINITY;
        }
        __syncthreads();
        float tmax = m;
        for (int jj = 0; jj < DC_BK; ++jj) tmax = fmaxf(tmax, sc[jj]);
        if (tmax > m) {   // uniform across the block
            const float c = ACCURATE ? expf(m - tmax) : __expf(m - tmax);
            omega *= c;
            first *= c;
#pragma unroll
            for (int t = 0; t < C::TPT; ++t)
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int y = 0; y < 4; ++y) { accM[t][x][y] *= c; accN[t][x][y] *= c; }
            m = tmax;
        }
        for (int jj = 0; jj < jn; ++jj) {
            const float w = ACCURATE ? expf(sc[jj] - m) : __expf(sc[jj] - m);
            omega += w;
            if (tid < D) first += w * Ks[jj * D + tid];
            else if (tid < 2 * D) first += w * Vs[jj * D + tid - D];
#pragma unroll
            for (int t = 0; t < C::TPT; ++t) {
                const int tile = tid + t * DC_THREADS;
                if (tile < C::T1 * C::T1) {
                    const int r0 = (tile / C::T1) * 4, c0 = (tile % C::T1) * 4;
                    const float4 kr = *reinterpret_cast<const float4*>(Ks + jj * D + r0);
                    const float4 vr = *reinterpret_cast<const float4*>(Vs + jj * D + r0);
                    const float4 kc = *reinterpret_cast<const float4*>(Ks + jj * D + c0);
                    const float kw[4] = {w * kr.x, w * kr.y, w * kr.z, w * kr.w};
                    const float vw[4] = {w * vr.x, w * vr.y, w * vr.z, w * vr.w};
                    const float kk[4] = {kc.x, kc.y, kc.z, kc.w};
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int y = 0; y < 4; ++y) {
                            accM[t][x][y] += kw[x] * kk[y];
                            accN[t][x][y] += vw[x] * kk[y];
                        }
                }
            }
        }
    }
    __syncthreads();

    if (splits > 1) {
        float* dst = parts + ((size_t)bh * splits + part) * C::PART_FLOATS;
#pragma unroll
        for (int t = 0; t < C::TPT; ++t) {
            const int tile = tid + t * DC_THREADS;
            if (tile < C::T1 * C::T1) {
                const int r0 = (tile / C::T1) * 4, c0 = (tile % C::T1) * 4;
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    *reinterpret_cast<float4*>(dst + (r0 + x) * D + c0) =
                        make_float4(accM[t][x][0], accM[t][x][1], accM[t][x][2], accM[t][x][3]);
                    *reinterpret_cast<float4*>(dst + D * D + (r0 + x) * D + c0) =
                        make_float4(accN[t][x][0], accN[t][x][1], accN[t][x][2], accN[t][x][3]);
                }
            }
        }
        if (tid < 2 * D) dst[2 * D * D + tid] = first;
        if (tid == 0) {
            dst[2 * D * D + 2 * D] = omega;
            dst[2 * D * D + 2 * D + 1] = m;
        }
        return;
    }

    // single part: finalize here.  Shared memory is re-carved as doubles.
    __shared__ double qd_s[D];
    for (int e = tid; e < D; e += DC_THREADS) qd_s[e] = (double)qs[e];
    __syncthreads();
    double* Md = smem_d;                 // D * (D+1)
    double* a = Md + D * (D + 1);        // D
    double* c = a + D;                   // D, followed by rhs (D)
    float* Nd = reinterpret_cast<float*>(c + 2 * D);   // D * D
#pragma unroll
    for (int t = 0; t < C::TPT; ++t) {
        const int tile = tid + t * DC_THREADS;
        if (tile < C::T1 * C::T1) {
            const int r0 = (tile / C::T1) * 4, c0 = (tile % C::T1) * 4;
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    Md[(r0 + x) * (D + 1) + c0 + y] = (double)accM[t][x][y];
                    Nd[(r0 + x) * D + c0 + y] = accN[t][x][y];
                }
        }
    }
    if (tid < D) a[tid] = (double)first;
    else if (tid < 2 * D) c[tid - D] = (double)first;
    finalize_row<D>(Md, Nd, a, c, (double)omega, (double)m, qd_s, (double)(lambda_units ? lambda_units[bh] : lambda),
                    ridge_mode, out + (size_t)bh * D, status);
}

template <int D, typename TIn, typename TOut>
__global__ void __launch_bounds__(DC_THREADS)
decode_combine_kernel(const TIn* __restrict__ q, const float* __restrict__ parts, TOut* __restrict__ out,
                      const int* __restrict__ lens, int H, int Lmax, int head_rows, float lambda, int splits,
                      int* __restrict__ status, const float* __restrict__ lambda_units, int ridge_mode, int window) {
    using C = DcCfg<D>;
    extern __shared__ double smem_d[];
    double* Md = smem_d;
    double* a = Md + D * (D + 1);
    double* c = a + D;
    float* Nd = reinterpret_cast<float*>(c + 2 * D);
    __shared__ double qd_s[D];
    const int tid = threadIdx.x, bh = blockIdx.x;
    if (visible_keys(lens[bh / H], Lmax, window) < head_rows) return;
    const float* src = parts + (size_t)bh * splits * C::PART_FLOATS;
    for (int e = tid; e < D; e += DC_THREADS) qd_s[e] = (double)to_f32(q[(size_t)bh * D + e]);
    float m = -INFINITY;
    for (int p = 0; p < splits; ++p) m = fmaxf(m, src[(size_t)p * C::PART_FLOATS + 2 * D * D + 2 * D + 1]);
    double omega = 0.0;
    for (int e = tid; e < D * D; e += DC_THREADS) {
        const int r = e / D, cc = e - r * D;
        double sm = 0.0, sn = 0.0;
        for (int p = 0; p < splits; ++p) {
            const float* pp = src + (size_t)p * C::PART_FLOATS;
            const double f = exp((double)pp[2 * D * D + 2 * D + 1] - (double)m);   // 0 for empty parts
            sm += f * (double)pp[e];
            sn += f * (double)pp[D * D + e];
        }
        Md[r * (D + 1) + cc] = sm;
        Nd[e] = (float)sn;
    }
    for (int e = tid; e < 2 * D; e += DC_THREADS) {
        double s1 = 0.0;
        for (int p = 0; p < splits; ++p) {
            const float* pp = src + (size_t)p * C::PART_FLOATS;
            s1 += exp((double)pp[2 * D * D + 2 * D + 1] - (double)m) * (double)pp[2 * D * D + e];
        }
        if (e < D) a[e] = s1; else c[e - D] = s1;
    }
    for (int p = 0; p < splits; ++p) {
        const float* pp = src + (size_t)p * C::PART_FLOATS;
        omega += exp((double)pp[2 * D * D + 2 * D + 1] - (double)m) * (double)pp[2 * D * D + 2 * D];
    }
    finalize_row<D>(Md, Nd, a, c, omega, (double)m, qd_s, (double)(lambda_units ? lambda_units[bh] : lambda), ridge_mode,
                    out + (size_t)bh * D, status);
}

template <int D>
constexpr size_t decode_smem_bytes() {
    const size_t stream = sizeof(float) * (2 * (size_t)DC_BK * D + DC_BK + D);
    const size_t fin = sizeof(double) * ((size_t)D * (D + 1) + 3 * D) + sizeof(float) * (size_t)D * D;
    return stream > fin ? stream : fin;
}

template <int D, typename TIn, typename TOut>
int launch_t(const DecodeArgs& a) {
    const int splits = a.splits < 1 ? 1 : a.splits;
    const size_t smem = decode_smem_bytes<D>();
    if (splits > 1) {
        const size_t need = decode_workspace_bytes(a.B, a.H, a.d, a.dv, splits);
        if (!a.workspace || a.workspace_bytes < need) return LLA_ERR_WORKSPACE;
    }
    // The tensor-core path keeps its moments relative to the first tile's maximum, not the true one,
    // which the printed ridge variant is defined against: that variant runs on the kernels below.
    if (a.impl == LLA_IMPL_TENSOR && a.ridge_mode == LLA_RIDGE_PRINTED) return LLA_ERR_UNSUPPORTED;
    if (a.impl != LLA_IMPL_SIMT && a.ridge_mode == LLA_RIDGE_DEFINITION && decode_tensor_supported(a)) {
        // tensor-core path: streaming kernel plus its own solve kernel (or fused epilogue)
        return launch_decode_tensor_moments(a);
    } else {
        if (a.impl == LLA_IMPL_TENSOR) return LLA_ERR_UNSUPPORTED;
        auto k1 = decode_moments_kernel<D, TIn, TOut>;
        LLA_CUDA_TRY(cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        dim3 grid(splits, a.B * a.H);
        k1<<<grid, DC_THREADS, smem, a.stream>>>((const TIn*)a.q, (const TIn*)a.kcache, (const TIn*)a.vcache,
                                                 a.lens, (TOut*)a.out, a.H, a.Lmax, a.scale, a.lambda, splits,
                                                 a.head_rows, (float*)a.workspace, a.status, a.lambda_units, a.ridge_mode, a.kv_group, a.paged, a.window);
        LLA_CUDA_TRY(cudaGetLastError());
    }
    if (splits > 1) {
        auto k2 = decode_combine_kernel<D, TIn, TOut>;
        LLA_CUDA_TRY(cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        k2<<<a.B * a.H, DC_THREADS, smem, a.stream>>>((const TIn*)a.q, (const float*)a.workspace,
                                                      (TOut*)a.out, a.lens, a.H, a.Lmax, a.head_rows, a.lambda, splits, a.status,
                                                      a.lambda_units, a.ridge_mode, a.window);
        LLA_CUDA_TRY(cudaGetLastError());
    }
    return LLA_OK;
}

template <int D>
int launch_d(const DecodeArgs& a) {
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_BF16) return launch_t<D, __nv_bfloat16, __nv_bfloat16>(a);
    if (a.in_dtype == LLA_BF16 && a.out_dtype == LLA_F32) return launch_t<D, __nv_bfloat16, float>(a);
    if (a.in_dtype == LLA_F32 && a.out_dtype == LLA_F32) return launch_t<D, float, float>(a);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace

size_t decode_record_bytes(int B, int H, int d, int dv, int splits) {
    (void)dv;
    return sizeof(float) * (size_t)B * H * (splits < 1 ? 1 : splits) * (2 * (size_t)d * d + 2 * d + 4);
}

size_t decode_workspace_bytes(int B, int H, int d, int dv, int splits) {
    if (splits <= 1) return 0;
    (void)dv;
    return sizeof(float) * (size_t)B * H * splits * (2 * (size_t)d * d + 2 * d + 4);
}

int launch_decode(const DecodeArgs& a) {
    if (a.d != a.dv) return LLA_ERR_UNSUPPORTED;
    switch (a.d) {
        case 16: return launch_d<16>(a);
        case 64: return launch_d<64>(a);
        case 128: return launch_d<128>(a);
        default: return LLA_ERR_UNSUPPORTED;
    }
}

// ---------------------------------------------------------------------------------------------
// Decode without any allocation: the split-key decode above, with the partial-moment records kept
// in a fixed device array that is part of the library image.
// ---------------------------------------------------------------------------------------------
namespace {

// Scratch shared by every lla_decode_noalloc call on a device.  It lives in each device's copy of
// the module for as long as the library stays loaded.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LLA_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal

// The array's name is only a host-side handle in host code; kernels need its device address.
int noalloc_scratch_ptr(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LLA_ERR_CUDA;
    void* p = __atomic_load_n(&g_noalloc_ptr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return LLA_ERR_CUDA;
        __atomic_store_n(&g_noalloc_ptr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return LLA_OK;
}

}  // namespace
}  // namespace lla

extern "C" int lla_decode_noalloc(const void* q, const void* kcache, const void* vcache, const int* lens,
                                  void* out, int B, int H, int Lmax, int d, int dv, int in_dtype, int out_dtype,
                                  float scale, float lambda, int splits, void* stream) {
    if (!q || !kcache || !vcache || !lens || !out) return LLA_ERR_INVALID_ARG;
    if (B < 1 || H < 1 || Lmax < 1 || d < 1 || dv < 1 || splits < 0) return LLA_ERR_INVALID_ARG;
    if (!(lambda >= 0.f) || !isfinite(lambda) || !isfinite(scale)) return LLA_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)kcache | (uintptr_t)vcache | (uintptr_t)out) & 15u) return LLA_ERR_INVALID_ARG;
    if (d != dv || !(d == 16 || d == 64 || d == 128) || (long long)B * H > 65535) return LLA_ERR_UNSUPPORTED;
    const bool dt_ok = (in_dtype == LLA_BF16 && (out_dtype == LLA_BF16 || out_dtype == LLA_F32)) ||
                       (in_dtype == LLA_F32 && out_dtype == LLA_F32);
    if (!dt_ok) return LLA_ERR_UNSUPPORTED;
    lla::DecodeArgs a;
    a.q = q; a.kcache = kcache; a.vcache = vcache; a.lens = lens; a.out = out;
    a.B = B; a.H = H; a.Lmax = Lmax; a.d = d; a.dv = dv;
    a.in_dtype = in_dtype; a.out_dtype = out_dtype;
    a.scale = scale; a.lambda = lambda;
    a.lambda_units = nullptr; a.ridge_mode = LLA_RIDGE_DEFINITION;
    a.splits = splits > 0 ? splits : lla_decode_default_splits(B, H, Lmax);
    a.head_rows = 2 * d;
    a.impl = LLA_IMPL_AUTO;
    a.status = nullptr;
    a.workspace = nullptr; a.workspace_bytes = 0;
    a.stream = (cudaStream_t)stream;
    // records are required for a split decode and optional otherwise (they let the tensor-core path
    // run its solve as a separate kernel)
    size_t need = lla::decode_record_bytes(B, H, d, dv, a.splits);
    if (splits == 0 && a.splits > 1 && need > (size_t)LLA_NOALLOC_SCRATCH_BYTES) {
        a.splits = 1;      // the default split count does not fit the fixed array: run unsplit, as lla_decode_ex does
        need = lla::decode_record_bytes(B, H, d, dv, 1);
    }
    if (a.splits > 1 && need > (size_t)LLA_NOALLOC_SCRATCH_BYTES) return LLA_ERR_WORKSPACE;   // beyond the fixed array
    if (need <= (size_t)LLA_NOALLOC_SCRATCH_BYTES) {
        void* scratch = nullptr;
        const int rc = lla::noalloc_scratch_ptr(&scratch);
        if (rc != LLA_OK) return rc;
        a.workspace = scratch;
        a.workspace_bytes = LLA_NOALLOC_SCRATCH_BYTES;
    }
    const int st = lla::launch_decode(a);
    if (st != LLA_OK) return st;
    return lla::launch_head_rows_decode(a);
}
