// Backward pass of causal local linear attention (the paper's backward appendix), bf16 inputs, d = dv in
// {64, 128}, fp32 gradients.
//
// The gradient is taken in the weighted-mean-centred form the forward kernels use.  Per query row i with
// visible keys j <= i, p_j = w_ij / omega_i, kbar = sum_j p_j k_j, xi_j = k_j - kbar,
// C = sum_j p_j xi_j xi_j^T + (lambda e^{-m_i} / omega_i) I, mbar = kbar - q_i, the forward computes
//     y = C^{-1} mbar,  e_j = xi_j . y,  a_j = p_j (1 - e_j)  (the paper's s_ij),  o_i = sum_j a_j v_j.
// With g = dL/do_i and gamma_j = g . v_j (the appendix's gamma_ij), gbar = sum_j p_j gamma_j and
//     h = sum_j p_j gamma_j xi_j,   t = C^{-1} h   (the one extra solve; the appendix's u_i in this frame),
//     f_j = xi_j . t,   kappa = g . o_i + t . mbar,
// the chain rule through p (a softmax of the scores), k_j and q_i gives
//     dL/ds_ij = p_j [gamma_j (1 - e_j) + (gbar + f_j) e_j - f_j - kappa]
//     dV_j += a_j g
//     dK_j += scale dL/ds_ij q_i + p_j [(f_j - gamma_j + gbar) y + (e_j - 1) t]
//     dQ_i  = scale sum_j dL/ds_ij k_j + t.
// In exact arithmetic this is the appendix's Delta_Q, Delta_K, Delta_V (same function, same derivative);
// y follows from the saved rho and delta as y = rho omega / delta.
//
// Kernels (the direct rows run on a side stream beside the others, which run in this order):
//   bwd_split_kernel      an fp32 upstream gradient as bf16 pairs hi + lo
//   moments               per query tile: kbar_i, gbar_i, h_i
//   forward_tc_kernel     in solve mode: C_i t_i = h_i by conjugate gradients           (tcgen05 tensor cores)
//   bwd_rowprep_kernel    y_i, the per-row scalars, dL/dlambda_i; y and -t as bf16 pairs
//   pairs                 dQ per query tile, dK and dV per key tile
//   bwd_head_rows_kernel  rows with fewer than head_rows keys: everything in fp64 with a direct solve
// The moments and pair kernels are the tcgen05 kernels of lla_backward_tensor.cu (dQ by plain stores of the tile
// that owns the rows; dK and dV by atomic adds, which the direct rows and grouped heads also add into).  The fp32
// CUDA-core versions in this file (impl = LLA_IMPL_SIMT) are kept as an independent cross-check; their pair kernel
// adds dQ atomically.  With grouped heads (kv_group > 1) k, v, dk, dv are indexed by the key/value head.
#include "lla_common.cuh"

namespace lla {
namespace {

constexpr int BW_THREADS = 256;
constexpr int BW_BJ = 64;      // keys per tile
constexpr int BW_LDP = 68;     // row stride of the [query][key] pair matrices (floats)
constexpr int BW_ROWSC = 8;    // floats per row of the scalar record: m, 1/omega, gbar, kappa, kbar.y, kbar.t

template <int D>
struct BwCfg {
    static constexpr int BI = D <= 64 ? 64 : 32;   // query rows per tile
    static constexpr int LD = D + 4;               // row stride of the operand tiles (floats)
    static constexpr int RI = BI / 16;             // query rows per thread
    static constexpr int CU = D / 64;              // float4 column groups per thread
    static constexpr int LDT = BI + 4;             // row stride of the [key][query] matrices
    static constexpr size_t MOMENTS_SMEM = sizeof(float) * ((size_t)(2 * BI + 2 * BW_BJ) * LD + 2 * BW_BJ * LDT + BI);
    static constexpr size_t PAIRS_SMEM = sizeof(float) * ((size_t)(4 * BI + 2 * BW_BJ) * LD + 3 * BI * BW_LDP + BW_BJ * LDT);
};

// rows [row0, row0 + rows) of a row-major [.., D] array -> fp32 shared tile [rows][D + 4]; rows outside
// [lo, nvalid) are zero (never read: their memory may be uninitialised)
template <int D>
__device__ __forceinline__ void load_tile(float* dst, const void* src, int dtype, size_t row0, int rows, int nvalid, int lo = 0) {
    constexpr int LD = D + 4;
    for (int idx = threadIdx.x; idx < rows * (D / 4); idx += BW_THREADS) {
        const int r = idx / (D / 4), c = (idx % (D / 4)) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < nvalid && r >= lo) {
            if (dtype == LLA_F32) x = load4(static_cast<const float*>(src) + (row0 + r) * D + c);
            else x = load4(static_cast<const __nv_bfloat16*>(src) + (row0 + r) * D + c);
        }
        *reinterpret_cast<float4*>(dst + r * LD + c) = x;
    }
}

__device__ __forceinline__ float ld_any(const void* p, int dtype, size_t i) {
    return dtype == LLA_F32 ? static_cast<const float*>(p)[i] : __bfloat162float(static_cast<const __nv_bfloat16*>(p)[i]);
}

// acc[r][4u + x] += sum_l M[l][a0 + r] * X[l][4 tc + 64 u + x]   for l < len
template <int NR, int CU>
__device__ __forceinline__ void mac_tile(float (&acc)[NR][4 * CU], const float* M, int ldm, int a0, const float* X, int ldx,
                                         int tc, int len, float sign = 1.f) {
#pragma unroll 4
    for (int l = 0; l < len; ++l) {
        float mv[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) mv[r] = sign * M[l * ldm + a0 + r];
#pragma unroll
        for (int u = 0; u < CU; ++u) {
            const float4 x = *reinterpret_cast<const float4*>(X + l * ldx + 4 * tc + 64 * u);
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                acc[r][4 * u + 0] = fmaf(mv[r], x.x, acc[r][4 * u + 0]);
                acc[r][4 * u + 1] = fmaf(mv[r], x.y, acc[r][4 * u + 1]);
                acc[r][4 * u + 2] = fmaf(mv[r], x.z, acc[r][4 * u + 2]);
                acc[r][4 * u + 3] = fmaf(mv[r], x.w, acc[r][4 * u + 3]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// kbar_i = sum_j p_ij k_j,  gbar_i = sum_j p_ij gamma_ij,  h_i = sum_j p_ij gamma_ij k_j - gbar_i kbar_i
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(BW_THREADS)
bwd_moments_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, const void* __restrict__ dout, int dout_dtype,
                   const float* __restrict__ stats, float* __restrict__ kbar, float* __restrict__ hvec,
                   float* __restrict__ rowsc, int n, int first, float scale, int H, int kv_group) {
    using C = BwCfg<D>;
    constexpr int BI = C::BI, LD = C::LD, RI = C::RI, CU = C::CU, LDT = C::LDT;
    extern __shared__ __align__(16) float bw_smem[];
    float* Qs = bw_smem;
    float* Gs = Qs + BI * LD;
    float* Ks = Gs + BI * LD;
    float* Vs = Ks + BW_BJ * LD;
    float* Pt = Vs + BW_BJ * LD;          // [key][query]
    float* PGt = Pt + BW_BJ * LDT;
    float* gbs = PGt + BW_BJ * LDT;       // [BI]
    const int tid = threadIdx.x, ti = tid >> 4, tj = tid & 15;
    const int tile = gridDim.y - 1 - blockIdx.y;      // longest tiles first, heads fastest
    const int bh = blockIdx.x;
    const int i0 = tile * BI;
    if (i0 + BI <= first) return;                      // every row of the tile is solved directly
    const size_t base = (size_t)bh * n;
    const size_t kvbase = (size_t)kv_unit(bh, H, kv_group) * n;     // grouped heads: the key/value head's rows
    const int nrow = min(BI, n - i0);
    load_tile<D>(Qs, q, LLA_BF16, base + i0, BI, nrow);
    load_tile<D>(Gs, dout, dout_dtype, base + i0, BI, nrow);
    float mrow[RI], iom[RI], gb[RI];
#pragma unroll
    for (int r = 0; r < RI; ++r) {
        const int gi = i0 + ti + 16 * r;
        const bool okr = gi < n && gi >= first;
        mrow[r] = okr ? stats[(base + gi) * 3 + 0] : 0.f;
        iom[r] = okr ? 1.f / stats[(base + gi) * 3 + 1] : 0.f;
        gb[r] = 0.f;
    }
    float akb[RI][4 * CU] = {}, ah[RI][4 * CU] = {};
    const int jt_end = (min(n, i0 + BI) + BW_BJ - 1) / BW_BJ;
    for (int jt = 0; jt < jt_end; ++jt) {
        const int j0 = jt * BW_BJ;
        __syncthreads();
        load_tile<D>(Ks, k, LLA_BF16, kvbase + j0, BW_BJ, min(BW_BJ, n - j0));
        load_tile<D>(Vs, v, LLA_BF16, kvbase + j0, BW_BJ, min(BW_BJ, n - j0));
        __syncthreads();
        float s[RI][4] = {}, gm[RI][4] = {};
#pragma unroll 2
        for (int c = 0; c < D; c += 4) {
            float4 qv[RI], gv[RI];
#pragma unroll
            for (int r = 0; r < RI; ++r) {
                qv[r] = *reinterpret_cast<const float4*>(Qs + (ti + 16 * r) * LD + c);
                gv[r] = *reinterpret_cast<const float4*>(Gs + (ti + 16 * r) * LD + c);
            }
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float4 kv = *reinterpret_cast<const float4*>(Ks + (tj + 16 * x) * LD + c);
                const float4 vv = *reinterpret_cast<const float4*>(Vs + (tj + 16 * x) * LD + c);
#pragma unroll
                for (int r = 0; r < RI; ++r) {
                    s[r][x] = fmaf(qv[r].x, kv.x, fmaf(qv[r].y, kv.y, fmaf(qv[r].z, kv.z, fmaf(qv[r].w, kv.w, s[r][x]))));
                    gm[r][x] = fmaf(gv[r].x, vv.x, fmaf(gv[r].y, vv.y, fmaf(gv[r].z, vv.z, fmaf(gv[r].w, vv.w, gm[r][x]))));
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RI; ++r) {
            const int il = ti + 16 * r, gi = i0 + il;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int jl = tj + 16 * x, gj = j0 + jl;
                const float p = (gj <= gi && iom[r] > 0.f) ? __expf(fmaf(scale, s[r][x], -mrow[r])) * iom[r] : 0.f;
                const float pg = p * gm[r][x];
                Pt[jl * LDT + il] = p;
                PGt[jl * LDT + il] = pg;
                gb[r] += pg;
            }
        }
        __syncthreads();
        mac_tile<RI, CU>(akb, Pt, LDT, RI * ti, Ks, LD, tj, BW_BJ);
        mac_tile<RI, CU>(ah, PGt, LDT, RI * ti, Ks, LD, tj, BW_BJ);
    }
#pragma unroll
    for (int r = 0; r < RI; ++r) {
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) gb[r] += __shfl_xor_sync(0xffffffffu, gb[r], o);
        if (tj == 0) gbs[ti + 16 * r] = gb[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RI; ++r) {
        const int il = RI * ti + r, gi = i0 + il;
        if (gi >= n || gi < first) continue;
        const float gbar = gbs[il];
        if (tj == 0) rowsc[(base + gi) * BW_ROWSC + 2] = gbar;
#pragma unroll
        for (int u = 0; u < CU; ++u) {
            const int c = 4 * tj + 64 * u;
            float4 kb4 = make_float4(akb[r][4 * u], akb[r][4 * u + 1], akb[r][4 * u + 2], akb[r][4 * u + 3]);
            float4 h4 = make_float4(ah[r][4 * u] - gbar * kb4.x, ah[r][4 * u + 1] - gbar * kb4.y,
                                    ah[r][4 * u + 2] - gbar * kb4.z, ah[r][4 * u + 3] - gbar * kb4.w);
            *reinterpret_cast<float4*>(kbar + (base + gi) * D + c) = kb4;
            *reinterpret_cast<float4*>(hvec + (base + gi) * D + c) = h4;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Per iterative row: y = rho omega / delta and the scalars the pair kernels need.  One warp per row.
// CUDA-core pair kernel (pairs16 == nullptr): dQ_i = t_i, to which that kernel adds the rest with atomics.
// Tensor-core pair kernels: y and -t also as bf16 pairs hi + lo (pairs16 = yh, yl, tnh, tnl, each [rows][D]); the
// rows solved directly get zero operands and a zero record, which switches them off in those kernels.
// ------------------------------------------------------------------------------------------------
// (x0, x1) -> packed bf16 pairs hi and lo with x = hi + lo up to 2^-17 relative
__device__ __forceinline__ void split_pack(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
    hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}
struct Pairs16 {
    uint32_t *yh, *yl, *tnh, *tnl;      // two bf16 per word
    float* pairsc;                      // [heads][npair][8]: the scalars of two rows per record (BwdTensorArgs::pairsc)
    int npair;
};
// row i's four scalars go to slots s, 2 + s, 4 + s, 6 + s of record i / 2 (s = i & 1)
__device__ __forceinline__ void store_pair_record(const Pairs16& p16, long long head, int i, float nm2, float ky, float gk, float kk) {
    float* rp = p16.pairsc + ((size_t)head * p16.npair + (i >> 1)) * 8 + (i & 1);
    if (!LLA_IN_BOUNDS(i >> 1, p16.npair, nullptr, 601)) return;
    rp[0] = nm2; rp[2] = ky; rp[4] = gk; rp[6] = kk;
}
template <int D>
__global__ void __launch_bounds__(BW_THREADS)
bwd_rowprep_kernel(const __nv_bfloat16* __restrict__ q, const void* __restrict__ out, int out_dtype,
                   const void* __restrict__ dout, int dout_dtype, const float* __restrict__ rho,
                   const float* __restrict__ stats, const float* __restrict__ kbar, const float* __restrict__ tvec,
                   float* __restrict__ yvec, float* __restrict__ rowsc, float* __restrict__ dq, int n, int first,
                   long long rows, float* __restrict__ dlambda, Pairs16 p16) {
    const long long row = (long long)blockIdx.x * (BW_THREADS / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int i = (int)(row % n);
    if (i < first) {
        if (p16.yh) {
            for (int c = 2 * lane; c < D; c += 64) {
                const size_t w = ((size_t)row * D + c) >> 1;
                p16.yh[w] = 0; p16.yl[w] = 0; p16.tnh[w] = 0; p16.tnl[w] = 0;
            }
            if (lane == 0) store_pair_record(p16, row / n, i, -1e30f, 0.f, 0.f, 0.f);
        }
        return;
    }
    const float m = stats[row * 3 + 0], omega = stats[row * 3 + 1], delta = stats[row * 3 + 2];
    const float fac = omega / delta;
    float ky = 0.f, kt = 0.f, qt = 0.f, go = 0.f, ty = 0.f;
#pragma unroll
    for (int c = 2 * lane; c < D; c += 64) {
        const size_t e = (size_t)row * D + c;
        const float2 r2 = *reinterpret_cast<const float2*>(rho + e), t2 = *reinterpret_cast<const float2*>(tvec + e);
        const float2 kb = *reinterpret_cast<const float2*>(kbar + e);
        const float y0 = r2.x * fac, y1 = r2.y * fac;
        *reinterpret_cast<float2*>(yvec + e) = make_float2(y0, y1);
        if (p16.yh) {
            uint32_t h, l;
            split_pack(y0, y1, h, l);
            p16.yh[e >> 1] = h; p16.yl[e >> 1] = l;
            split_pack(-t2.x, -t2.y, h, l);
            p16.tnh[e >> 1] = h; p16.tnl[e >> 1] = l;
        } else {
            *reinterpret_cast<float2*>(dq + e) = t2;
        }
        ky = fmaf(kb.x, y0, fmaf(kb.y, y1, ky));
        kt = fmaf(kb.x, t2.x, fmaf(kb.y, t2.y, kt));
        ty = fmaf(t2.x, y0, fmaf(t2.y, y1, ty));
        qt = fmaf(__bfloat162float(q[e]), t2.x, fmaf(__bfloat162float(q[e + 1]), t2.y, qt));
        go = fmaf(ld_any(dout, dout_dtype, e), ld_any(out, out_dtype, e), fmaf(ld_any(dout, dout_dtype, e + 1), ld_any(out, out_dtype, e + 1), go));
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        ky += __shfl_xor_sync(0xffffffffu, ky, o);
        kt += __shfl_xor_sync(0xffffffffu, kt, o);
        qt += __shfl_xor_sync(0xffffffffu, qt, o);
        go += __shfl_xor_sync(0xffffffffu, go, o);
        ty += __shfl_xor_sync(0xffffffffu, ty, o);
    }
    if (lane == 0) {
        float* rs = rowsc + row * BW_ROWSC;
        rs[0] = m;
        rs[1] = 1.f / omega;
        rs[3] = go + kt - qt;      // kappa = g.o + t.(kbar - q)
        rs[4] = ky;
        rs[5] = kt;
        if (p16.yh) {
            const float kappa = go + kt - qt;
            store_pair_record(p16, row / n, i, -(m * 1.4426950408889634f + log2f(omega)), ky, rs[2] - kt, kt - kappa);
            if (i == n - 1 && (n & 1)) store_pair_record(p16, row / n, n, -1e30f, 0.f, 0.f, 0.f);      // the record's unused half
        }
        // dL/d(lambda_i): lambda enters C as (e^{-m} / omega) lambda I and dL = t^T dC y
        if (dlambda) dlambda[row] = __expf(-m) / omega * ty;
    }
}

// fp32 upstream gradient -> bf16 pairs hi + lo (the tensor-core kernels' operand format), four elements per thread
__global__ void __launch_bounds__(256)
bwd_split_kernel(const float* __restrict__ src, uint2* __restrict__ hi, uint2* __restrict__ lo, size_t quads) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= quads) return;
    const float4 x = reinterpret_cast<const float4*>(src)[i];
    uint2 h, l;
    split_pack(x.x, x.y, h.x, l.x);
    split_pack(x.z, x.w, h.y, l.y);
    hi[i] = h;
    lo[i] = l;
}

// ------------------------------------------------------------------------------------------------
// One block per 64-key tile: dK and dV of its keys accumulate in registers over every query tile that
// sees them; each query tile's dQ contribution goes out with atomic adds.
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(BW_THREADS)
bwd_pairs_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                 const __nv_bfloat16* __restrict__ v, const void* __restrict__ dout, int dout_dtype,
                 const float* __restrict__ yvec, const float* __restrict__ tvec, const float* __restrict__ rowsc,
                 float* __restrict__ dq, float* __restrict__ dk, float* __restrict__ dv, int n, int first, float scale, int H, int kv_group) {
    using C = BwCfg<D>;
    constexpr int BI = C::BI, LD = C::LD, RI = C::RI, CU = C::CU, LDT = C::LDT, LDP = BW_LDP;
    extern __shared__ __align__(16) float bw_smem[];
    float* Ks = bw_smem;
    float* Vs = Ks + BW_BJ * LD;
    float* Qs = Vs + BW_BJ * LD;
    float* Ys = Qs + BI * LD;
    float* Ts = Ys + BI * LD;
    float* Gs = Ts + BI * LD;
    float* Am = Gs + BI * LD;             // [query][key]: a_ij
    float* DSm = Am + BI * LDP;           //               scale dL/ds_ij
    float* P1m = DSm + BI * LDP;          //               p_ij (f_ij - gamma_ij + gbar_i)
    float* DSt = P1m + BI * LDP;          // [key][query]: scale dL/ds_ij
    const int tid = threadIdx.x, ti = tid >> 4, tj = tid & 15;
    const int bh = blockIdx.x;
    const int j0 = blockIdx.y * BW_BJ;    // key tile 0 sees the most query tiles and starts first (heads fastest)
    const size_t base = (size_t)bh * n;
    const size_t kvbase = (size_t)kv_unit(bh, H, kv_group) * n;     // grouped heads: the key/value head's rows
    load_tile<D>(Ks, k, LLA_BF16, kvbase + j0, BW_BJ, min(BW_BJ, n - j0));
    load_tile<D>(Vs, v, LLA_BF16, kvbase + j0, BW_BJ, min(BW_BJ, n - j0));
    float adk[4][4 * CU] = {}, adv[4][4 * CU] = {};
    const int it0 = max(j0, first) / BI, it1 = (n + BI - 1) / BI;
    for (int it = it0; it < it1; ++it) {
        const int i0 = it * BI;
        const int nrow = min(BI, n - i0);
        __syncthreads();
        load_tile<D>(Qs, q, LLA_BF16, base + i0, BI, nrow);
        load_tile<D>(Ys, yvec, LLA_F32, base + i0, BI, nrow, first - i0);
        load_tile<D>(Ts, tvec, LLA_F32, base + i0, BI, nrow, first - i0);
        load_tile<D>(Gs, dout, dout_dtype, base + i0, BI, nrow);
        __syncthreads();
        float s[RI][4] = {}, e[RI][4] = {}, f[RI][4] = {}, gm[RI][4] = {};
#pragma unroll 1
        for (int c = 0; c < D; c += 4) {
            float4 kv[4], vv[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                kv[x] = *reinterpret_cast<const float4*>(Ks + (tj + 16 * x) * LD + c);
                vv[x] = *reinterpret_cast<const float4*>(Vs + (tj + 16 * x) * LD + c);
            }
#pragma unroll
            for (int r = 0; r < RI; ++r) {
                const float4 qv = *reinterpret_cast<const float4*>(Qs + (ti + 16 * r) * LD + c);
                const float4 yv = *reinterpret_cast<const float4*>(Ys + (ti + 16 * r) * LD + c);
                const float4 tv = *reinterpret_cast<const float4*>(Ts + (ti + 16 * r) * LD + c);
                const float4 gv = *reinterpret_cast<const float4*>(Gs + (ti + 16 * r) * LD + c);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    s[r][x] = fmaf(qv.x, kv[x].x, fmaf(qv.y, kv[x].y, fmaf(qv.z, kv[x].z, fmaf(qv.w, kv[x].w, s[r][x]))));
                    e[r][x] = fmaf(yv.x, kv[x].x, fmaf(yv.y, kv[x].y, fmaf(yv.z, kv[x].z, fmaf(yv.w, kv[x].w, e[r][x]))));
                    f[r][x] = fmaf(tv.x, kv[x].x, fmaf(tv.y, kv[x].y, fmaf(tv.z, kv[x].z, fmaf(tv.w, kv[x].w, f[r][x]))));
                    gm[r][x] = fmaf(gv.x, vv[x].x, fmaf(gv.y, vv[x].y, fmaf(gv.z, vv[x].z, fmaf(gv.w, vv[x].w, gm[r][x]))));
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RI; ++r) {
            const int il = ti + 16 * r, gi = i0 + il;
            const bool okr = gi < n && gi >= first;
            const float* rs = rowsc + (base + gi) * BW_ROWSC;
            const float m = okr ? rs[0] : 0.f, iom = okr ? rs[1] : 0.f, gbar = okr ? rs[2] : 0.f;
            const float kappa = okr ? rs[3] : 0.f, ky = okr ? rs[4] : 0.f, kt = okr ? rs[5] : 0.f;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int jl = tj + 16 * x, gj = j0 + jl;
                const float p = (okr && gj <= gi) ? __expf(fmaf(scale, s[r][x], -m)) * iom : 0.f;
                const float ev = e[r][x] - ky, fv = f[r][x] - kt, gam = gm[r][x];
                const float a = p * (1.f - ev);
                const float ds = scale * p * (gam * (1.f - ev) + (gbar + fv) * ev - fv - kappa);
                Am[il * LDP + jl] = a;
                DSm[il * LDP + jl] = ds;
                P1m[il * LDP + jl] = p * (fv - gam + gbar);
                DSt[jl * LDT + il] = ds;
            }
        }
        __syncthreads();
        // dV += A^T G;  dK += DS^T Q + P1^T Y - A^T T      (rows = this thread's four keys)
        mac_tile<4, CU>(adv, Am, LDP, 4 * ti, Gs, LD, tj, nrow);
        mac_tile<4, CU>(adk, DSm, LDP, 4 * ti, Qs, LD, tj, nrow);
        mac_tile<4, CU>(adk, P1m, LDP, 4 * ti, Ys, LD, tj, nrow);
        mac_tile<4, CU>(adk, Am, LDP, 4 * ti, Ts, LD, tj, nrow, -1.f);
        // dQ += DS K                                        (rows = RI query rows)
        float adq[RI][4 * CU] = {};
        mac_tile<RI, CU>(adq, DSt, LDT, RI * ti, Ks, LD, tj, BW_BJ);
#pragma unroll
        for (int r = 0; r < RI; ++r) {
            const int gi = i0 + RI * ti + r;
            if (gi >= n || gi < first) continue;
#pragma unroll
            for (int u = 0; u < CU; ++u)
#pragma unroll
                for (int x = 0; x < 4; ++x) atomicAdd(dq + (base + gi) * D + 4 * tj + 64 * u + x, adq[r][4 * u + x]);
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int gj = j0 + 4 * ti + r;
        if (gj >= n) continue;
#pragma unroll
        for (int u = 0; u < CU; ++u) {
            const int c = 4 * tj + 64 * u;
            // (added, not stored: the directly-solved rows add their share from another stream)
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                atomicAdd(dk + (kvbase + gj) * D + c + x, adk[r][4 * u + x]);
                atomicAdd(dv + (kvbase + gj) * D + c + x, adv[r][4 * u + x]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Rows that see fewer than head_rows keys: C is ill-conditioned (rank-deficient up to the ridge), so the
// whole row -- both solves and every pair term -- runs in fp64 with an explicit C and a direct LDL^T
// solve, the same split the forward makes.  One block per row; dK and dV go out with atomic adds.
// ------------------------------------------------------------------------------------------------

constexpr int HB_THREADS = 160;   // 136 4x4 tiles of the matrix build fit one round; four blocks per SM
// eight lanes per key: sum over the lanes of a group of eight
__device__ __forceinline__ double group8_sum(double x) {
#pragma unroll
    for (int o = 4; o >= 1; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
// D / 8 consecutive bf16 of a row -> doubles
template <int NE>
__device__ __forceinline__ void load_bf16_run(const __nv_bfloat16* p, double (&dst)[NE]) {
#pragma unroll
    for (int e = 0; e < NE; e += 8) {
        const uint4 r = *reinterpret_cast<const uint4*>(p + e);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            dst[e + 2 * x] = (double)__uint_as_float(w[x] << 16);
            dst[e + 2 * x + 1] = (double)__uint_as_float(w[x] & 0xFFFF0000u);
        }
    }
}
template <int D>
__global__ void __launch_bounds__(HB_THREADS, D == 64 ? 4 : 1)
bwd_head_rows_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const void* __restrict__ dout, int dout_dtype,
                     float* __restrict__ dq, float* __restrict__ dk, float* __restrict__ dv, int n, int lcap,
                     double scale, double lambda, int* __restrict__ status, float* __restrict__ dlambda, int H, int kv_group,
                     int nq) {
    constexpr int LDS = D + 1;
    extern __shared__ __align__(16) double hb_smem[];
    double* S = hb_smem;                  // D x (D + 1)
    double* rhs = S + D * LDS;            // [2][D]: mbar -> y, h -> t
    double* kb = rhs + 2 * D;
    double* mb = kb + D;
    double* qd = mb + D;
    double* gd = qd + D;
    double* hp = gd + D;                  // sum_j p_j gamma_j k_j
    double* pj = hp + D;                  // [lcap] each
    double* gam = pj + lcap;
    double* ee = gam + lcap;
    double* ff = ee + lcap;
    __nv_bfloat16* Kr = reinterpret_cast<__nv_bfloat16*>(ff + lcap);   // [lcap][D]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x;
    const int i = gridDim.y - 1 - blockIdx.y;       // rows with the most keys first
    const int L = (n - nq) + i + 1;                 // query row i sits at position n - nq + i
    if (!LLA_IN_BOUNDS(L, lcap + 1, status, 602)) return;      // (debug build: the keys must fit the arrays sized for lcap)
    const size_t base = (size_t)bh * nq;            // rows of q, dout, dq, dlambda
    const size_t kvbase = (size_t)kv_unit(bh, H, kv_group) * n;     // grouped heads: the key/value head's rows
    for (int c = tid; c < D; c += HB_THREADS) {
        qd[c] = (double)__bfloat162float(q[(base + i) * D + c]);
        gd[c] = (double)ld_any(dout, dout_dtype, (base + i) * D + c);
    }
    for (int idx = tid; idx < L * (D / 8); idx += HB_THREADS)
        reinterpret_cast<uint4*>(Kr)[idx] = reinterpret_cast<const uint4*>(k + kvbase * D)[idx];
    __syncthreads();
    // scores and gamma_j = g . v_j: eight lanes per key (D / 8 consecutive elements each), four keys per warp
    constexpr int NE = D / 8;
    const int l8 = lane & 7, kslot = warp * 4 + (lane >> 3);
    for (int j0 = 0; j0 < L; j0 += 4 * (HB_THREADS / 32)) {
        const int j = j0 + kslot;
        double s = 0.0, gv = 0.0;
        if (j < L) {
            double kk[NE], vv[NE];
            load_bf16_run<NE>(Kr + j * D + NE * l8, kk);
            load_bf16_run<NE>(v + (kvbase + j) * D + NE * l8, vv);
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                s += qd[NE * l8 + e] * kk[e];
                gv += gd[NE * l8 + e] * vv[e];
            }
        }
        s = group8_sum(s);
        gv = group8_sum(gv);
        if (j < L && l8 == 0) { pj[j] = scale * s; gam[j] = gv; }
    }
    __syncthreads();
    double m = -1e300;
    for (int j = 0; j < L; ++j) m = fmax(m, pj[j]);
    __syncthreads();
    for (int j = tid; j < L; j += HB_THREADS) pj[j] = exp(pj[j] - m);
    __syncthreads();
    double omega = 0.0;
    for (int j = 0; j < L; ++j) omega += pj[j];
    const double em_om = exp(-m) / omega;     // d(ridge of C) / d(lambda)
    const double eps = lambda * em_om;
    __syncthreads();
    for (int j = tid; j < L; j += HB_THREADS) pj[j] /= omega;
    __syncthreads();
    double gbar = 0.0;
    for (int j = 0; j < L; ++j) gbar += pj[j] * gam[j];
    for (int c = tid; c < 2 * D; c += HB_THREADS) {
        const int cc = c % D;
        double acc = 0.0;
        if (c < D) for (int j = 0; j < L; ++j) acc += pj[j] * (double)__bfloat162float(Kr[j * D + cc]);
        else for (int j = 0; j < L; ++j) acc += pj[j] * gam[j] * (double)__bfloat162float(Kr[j * D + cc]);
        (c < D ? kb : hp)[cc] = acc;
    }
    __syncthreads();
    for (int c = tid; c < D; c += HB_THREADS) {
        mb[c] = kb[c] - qd[c];
        rhs[c] = mb[c];
        rhs[D + c] = hp[c] - gbar * kb[c];
    }
    // C (lower triangle) in 4 x 4 blocks
    for (int blk = tid; blk < (D / 4) * (D / 4); blk += HB_THREADS) {
        const int a0 = (blk / (D / 4)) * 4, b0 = (blk % (D / 4)) * 4;
        if (b0 > a0) continue;
        double acc[4][4] = {};
        for (int j = 0; j < L; ++j) {
            // four consecutive bf16 keys per 8-byte load (a0, b0 are multiples of four)
            const uint2 ra = *reinterpret_cast<const uint2*>(Kr + j * D + a0);
            const uint2 rb = *reinterpret_cast<const uint2*>(Kr + j * D + b0);
            const double ka[4] = {(double)__uint_as_float(ra.x << 16), (double)__uint_as_float(ra.x & 0xFFFF0000u),
                                  (double)__uint_as_float(ra.y << 16), (double)__uint_as_float(ra.y & 0xFFFF0000u)};
            const double kc[4] = {(double)__uint_as_float(rb.x << 16), (double)__uint_as_float(rb.x & 0xFFFF0000u),
                                  (double)__uint_as_float(rb.y << 16), (double)__uint_as_float(rb.y & 0xFFFF0000u)};
            const double p = pj[j];
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] += p * ka[x] * kc[y];
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const int a = a0 + x, b = b0 + y;
                if (b <= a) S[a * LDS + b] = acc[x][y] - kb[a] * kb[b] + (a == b ? eps : 0.0);
            }
    }
    const bool okf = block_ldlt_solve<D>(S, LDS, rhs, D, 2, D);
    if (!okf && tid == 0 && status) atomicAdd(status + LLA_STATUS_BAD_PIVOT, 1);
    const double* y = rhs;
    const double* t = rhs + D;
    // e_j = xi_j . y, f_j = xi_j . t
    for (int j0 = 0; j0 < L; j0 += 4 * (HB_THREADS / 32)) {
        const int j = j0 + kslot;
        double e = 0.0, f = 0.0;
        if (j < L) {
            double kk[NE];
            load_bf16_run<NE>(Kr + j * D + NE * l8, kk);
#pragma unroll
            for (int x = 0; x < NE; ++x) {
                const double xi = kk[x] - kb[NE * l8 + x];
                e += xi * y[NE * l8 + x];
                f += xi * t[NE * l8 + x];
            }
        }
        e = group8_sum(e);
        f = group8_sum(f);
        if (j < L && l8 == 0) { ee[j] = e; ff[j] = f; }
    }
    __syncthreads();
    double kappa = 0.0;
    for (int j = 0; j < L; ++j) kappa += pj[j] * (1.0 - ee[j]) * gam[j];      // g . o_i
    double ty = 0.0;
    for (int c = 0; c < D; ++c) {
        kappa += t[c] * mb[c];
        ty += t[c] * y[c];
    }
    if (dlambda && tid == 0) dlambda[base + i] = (float)(em_om * ty);     // dL = t^T dC y
    __syncthreads();
    // per key: a_j -> pj, scale dL/ds_ij -> gam, p (f - gamma + gbar) -> ff, p (e - 1) -> ee
    for (int j = tid; j < L; j += HB_THREADS) {
        const double p = pj[j], e = ee[j], f = ff[j], gmj = gam[j];
        pj[j] = p * (1.0 - e);
        gam[j] = scale * p * (gmj * (1.0 - e) + (gbar + f) * e - f - kappa);
        ff[j] = p * (f - gmj + gbar);
        ee[j] = p * (e - 1.0);
    }
    __syncthreads();
    for (int c = tid; c < D; c += HB_THREADS) {
        double acc = t[c];
        for (int j = 0; j < L; ++j) acc += gam[j] * (double)__bfloat162float(Kr[j * D + c]);
        dq[(base + i) * D + c] = (float)acc;
    }
    // (one atomic per row and output: a version that wrote the per-key coefficients out and summed the rows in
    //  a second kernel was slower, the sum's serial loop costing more than the atomics it saved)
    for (int idx = tid; idx < L * D; idx += HB_THREADS) {
        const int j = idx / D, c = idx % D;
        atomicAdd(dk + (kvbase + j) * D + c, (float)(gam[j] * qd[c] + ff[j] * y[c] + ee[j] * t[c]));
        atomicAdd(dv + (kvbase + j) * D + c, (float)(pj[j] * gd[c]));
    }
}

template <int D>
size_t head_smem_bytes(int lcap) {
    return sizeof(double) * ((size_t)D * (D + 1) + 7 * D + 4 * lcap) + sizeof(__nv_bfloat16) * (size_t)lcap * D;
}

// workspace: kbar, h, t, y as [rows][D] fp32, the scalar records, then the tensor-core kernels' bf16 operand arrays
// (y and -t as hi and lo; the upstream gradient's hi and lo, used when it comes in fp32)
size_t ws_floats(long long rows, int d) { return (size_t)rows * (4 * (size_t)d + BW_ROWSC); }
size_t ws_pairsc_floats(long long heads, int n) { return (size_t)heads * ((n + 1) / 2) * 8; }      // two rows per record
size_t ws_fp32_bytes(long long rows, int d, long long heads) {
    return ((ws_floats(rows, d) + ws_pairsc_floats(heads, (int)(rows / heads))) * sizeof(float) + 255) & ~(size_t)255;
}
size_t ws_pair_bytes(long long rows, int d) { return ((size_t)rows * d * 2 + 255) & ~(size_t)255; }      // one bf16 array
size_t ws_own_bytes(long long rows, int d, long long heads) { return ws_fp32_bytes(rows, d, heads) + 6 * ws_pair_bytes(rows, d); }

template <int D>
int launch_t(const BackwardArgs& a) {
    using C = BwCfg<D>;
    const int nq = a.nq > 0 ? a.nq : a.n, off = a.n - nq;      // the queries are the positions off .. n - 1
    const long long rows = (long long)a.B * a.H * nq;          // rows of q, out, dout, rho, stats, dq
    const int BH = a.B * a.H;
    const int first = max(0, min(nq, a.head_rows - 1 - off));  // query rows [0, first) see fewer than head_rows keys: solved directly
    const int kvg = a.kv_group > 0 ? a.kv_group : 1;
    const long long kvrows = (long long)a.B * a.H * a.n / kvg; // rows of k, v, dk, dv
    if (a.workspace_bytes < ws_own_bytes(rows, D, BH) || !a.workspace) return LLA_ERR_WORKSPACE;
    if (first > 0 && off + first > 2 * D) return LLA_ERR_UNSUPPORTED;      // (head_rows beyond 2 d + 1)
    float* kbar = static_cast<float*>(a.workspace);
    float* hvec = kbar + rows * D;
    float* tvec = hvec + rows * D;
    float* yvec = tvec + rows * D;
    float* rowsc = yvec + rows * D;
    float* pairsc = rowsc + rows * BW_ROWSC;
    char* pairs = static_cast<char*>(a.workspace) + ws_fp32_bytes(rows, D, BH);
    const size_t pb = ws_pair_bytes(rows, D);
    const bool tensor = !a.cuda_core_pairs;
    const auto* q = static_cast<const __nv_bfloat16*>(a.q);
    const auto* k = static_cast<const __nv_bfloat16*>(a.k);
    const auto* v = static_cast<const __nv_bfloat16*>(a.v);
    const int lcap = first > 0 ? off + first : 0;              // most keys a directly-solved row sees
    const size_t head_smem = head_smem_bytes<D>(lcap);
    if (head_smem > 227u * 1024u) return LLA_ERR_UNSUPPORTED;
    LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_head_rows_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)head_smem));
    LLA_CUDA_TRY(cudaMemsetAsync(a.dk, 0, sizeof(float) * kvrows * D, a.stream));
    LLA_CUDA_TRY(cudaMemsetAsync(a.dv, 0, sizeof(float) * kvrows * D, a.stream));
    // the directly-solved rows depend on nothing the other kernels make: they run beside them on the side stream
    const bool forked = first > 0 && a.side_stream != nullptr;
    cudaStream_t hs = forked ? a.side_stream : a.stream;
    if (forked) {
        LLA_CUDA_TRY(cudaEventRecord(a.fork, a.stream));
        LLA_CUDA_TRY(cudaStreamWaitEvent(hs, a.fork, 0));
    }
    if (first > 0) {
        const dim3 gh(BH, first);
        bwd_head_rows_kernel<D><<<gh, HB_THREADS, head_smem, hs>>>(
            q, k, v, a.dout, a.dout_dtype, a.dq, a.dk, a.dv, a.n, lcap, (double)a.scale, (double)a.lambda, a.status, a.dlambda, a.H, kvg, nq);
        LLA_CUDA_TRY(cudaGetLastError());
        if (forked) LLA_CUDA_TRY(cudaEventRecord(a.join, hs));
    }
    if (first < nq) {
        BwdTensorArgs t = {};
        Pairs16 p16 = {};
        if (tensor) {
            t.q = a.q; t.k = a.k; t.v = a.v;
            t.yh = pairs; t.yl = pairs + pb; t.tnh = pairs + 2 * pb; t.tnl = pairs + 3 * pb;
            p16.yh = reinterpret_cast<uint32_t*>(pairs); p16.yl = reinterpret_cast<uint32_t*>(pairs + pb);
            p16.tnh = reinterpret_cast<uint32_t*>(pairs + 2 * pb); p16.tnl = reinterpret_cast<uint32_t*>(pairs + 3 * pb);
            p16.pairsc = pairsc; p16.npair = (nq + 1) / 2;
            if (a.dout_dtype == LLA_F32) {
                t.gh = pairs + 4 * pb; t.gl = pairs + 5 * pb;
                const size_t quads = (size_t)rows * D / 4;
                bwd_split_kernel<<<(unsigned)((quads + 255) / 256), 256, 0, a.stream>>>(
                    static_cast<const float*>(a.dout), reinterpret_cast<uint2*>(pairs + 4 * pb), reinterpret_cast<uint2*>(pairs + 5 * pb), quads);
                LLA_CUDA_TRY(cudaGetLastError());
            } else {
                t.gh = a.dout; t.gl = nullptr;
            }
            t.rowsc = rowsc; t.pairsc = pairsc; t.stats = a.stats; t.yvec = yvec; t.tvec = tvec;
            t.kbar = kbar; t.hvec = hvec; t.dq = a.dq; t.dk = a.dk; t.dv = a.dv;
            t.B = a.B; t.H = a.H; t.n = a.n; t.nq = nq; t.d = D; t.first = first; t.kv_group = kvg; t.window = a.window;
            t.head_rows = a.head_rows; t.block_mask = a.block_mask; t.block_mask_stride = a.block_mask_stride;
            t.wait_clocks = a.wait_clocks; t.no_loads = a.no_loads;
            t.scale = a.scale; t.status = a.status; t.stream = a.stream;
            const int rc = launch_backward_tensor(t, 0);
            if (rc != LLA_OK) return rc;
        } else {
            if (nq != a.n) return LLA_ERR_UNSUPPORTED;      // the CUDA-core kernels take whole sequences only
            const dim3 gm(BH, (a.n + C::BI - 1) / C::BI);
            LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_moments_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::MOMENTS_SMEM));
            bwd_moments_kernel<D><<<gm, BW_THREADS, C::MOMENTS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, a.stats, kbar, hvec,
                                                                              rowsc, a.n, first, a.scale, a.H, kvg);
            LLA_CUDA_TRY(cudaGetLastError());
        }
        // C_i t_i = h_i for the iterative rows: the forward's tensor-core CG with h as right-hand side
        ForwardArgs f = {};
        f.q = a.q; f.k = a.k; f.v = a.v; f.out = nullptr;
        f.B = a.B; f.H = a.H; f.n = a.n; f.d = D; f.dv = D;
        f.in_dtype = LLA_BF16; f.out_dtype = LLA_F32;
        f.scale = a.scale; f.lambda = a.lambda; f.causal = 1;
        f.max_iters = a.max_iters; f.tol = a.tol; f.head_rows = a.head_rows;
        f.status = a.status; f.iters = a.iters; f.stream = a.stream;
        f.ridge_mode = LLA_RIDGE_DEFINITION; f.nq = nq; f.kv_group = kvg; f.window = a.window;
        f.block_mask = a.block_mask; f.block_mask_stride = a.block_mask_stride;
        f.wait_clocks = a.wait_clocks; f.no_loads = a.no_loads;
        f.rhs = hvec; f.sol = tvec;
        f.kbar_in = kbar; f.stats_in = a.stats;      // kbar from the moments kernel, shift and omega as the forward saved them
        f.precondition = a.precondition;      // optional: the extra solve preconditioned (the matrices come from the pre-pass below)
        f.set_contiguous();
        // what the workspace holds beyond this pass's own arrays serves the solve (the fp16 copy of k; for
        // d = 128 the row-state slots), so that the backward pass allocates nothing
        const size_t own = ws_own_bytes(rows, D, BH);
        if (a.workspace_bytes > own) {
            f.workspace = static_cast<char*>(a.workspace) + own;
            f.workspace_bytes = a.workspace_bytes - own;
        }
        const int rc_pre = forward_tensor_prepass(f);
        if (rc_pre != LLA_OK) return rc_pre;
        const int rc = launch_forward_tensor(f);
        if (rc != LLA_OK) return rc;
        bwd_rowprep_kernel<D><<<(unsigned)((rows + 7) / 8), BW_THREADS, 0, a.stream>>>(
            q, a.out, a.out_dtype, a.dout, a.dout_dtype, a.rho, a.stats, kbar, tvec, yvec, rowsc, a.dq, nq, first, rows, a.dlambda, p16);
        LLA_CUDA_TRY(cudaGetLastError());
        if (tensor) {
            int rc2 = launch_backward_tensor(t, 1);
            if (rc2 != LLA_OK) return rc2;
            rc2 = launch_backward_tensor(t, 2);
            if (rc2 != LLA_OK) return rc2;
        } else {
            const dim3 gp(BH, (a.n + BW_BJ - 1) / BW_BJ);
            LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_pairs_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::PAIRS_SMEM));
            bwd_pairs_kernel<D><<<gp, BW_THREADS, C::PAIRS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, yvec, tvec, rowsc,
                                                                          a.dq, a.dk, a.dv, a.n, first, a.scale, a.H, kvg);
            LLA_CUDA_TRY(cudaGetLastError());
        }
    }
    if (forked) LLA_CUDA_TRY(cudaStreamWaitEvent(a.stream, a.join, 0));
    return LLA_OK;
}

}  // namespace

size_t backward_workspace_bytes(int B, int H, int n, int d) {
    return ws_own_bytes((long long)B * H * n, d, (long long)B * H) + forward_tensor_workspace_bytes(B, H, n, d);
}

int launch_backward(const BackwardArgs& a) {
    if (a.d == 64) return launch_t<64>(a);
    if (a.d == 128) return launch_t<128>(a);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
