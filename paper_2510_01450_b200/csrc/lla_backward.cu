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
// Kernels (the direct rows run on a side stream beside the other four, which run in this order):
//   bwd_moments_*         per 64-row query tile: kbar_i, gbar_i, h_i
//   forward_tc_kernel     in solve mode: C_i t_i = h_i by conjugate gradients           (tcgen05 tensor cores)
//   bwd_rowprep_kernel    y_i, the per-row scalars, dQ_i = t_i, dL/dlambda_i
//   bwd_pairs_*           per 64-key tile over all later query tiles: dK, dV (registers), dQ (atomics)
//   bwd_head_rows_kernel  rows with fewer than head_rows keys: everything in fp64 with a direct solve
// The moments and pair kernels exist twice: *_mma_kernel on the tensor cores (warp-level bf16 MMAs with hi/lo
// operand splits; the default) and the fp32 CUDA-core versions (impl = LLA_IMPL_SIMT), kept as an independent
// cross-check.  With grouped heads (kv_group > 1) k, v, dk, dv are indexed by the key/value head; dk and dv are
// zeroed first and every kernel adds into them atomically.
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
// Per iterative row: y = rho omega / delta, the scalars the pair kernel needs, and dQ_i = t_i (the pair
// kernel adds the rest with atomics).  One warp per row.
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(BW_THREADS)
bwd_rowprep_kernel(const __nv_bfloat16* __restrict__ q, const void* __restrict__ out, int out_dtype,
                   const void* __restrict__ dout, int dout_dtype, const float* __restrict__ rho,
                   const float* __restrict__ stats, const float* __restrict__ kbar, const float* __restrict__ tvec,
                   float* __restrict__ yvec, float* __restrict__ rowsc, float* __restrict__ dq, int n, int first,
                   long long rows, float* __restrict__ dlambda) {
    const long long row = (long long)blockIdx.x * (BW_THREADS / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int i = (int)(row % n);
    if (i < first) return;
    const float m = stats[row * 3 + 0], omega = stats[row * 3 + 1], delta = stats[row * 3 + 2];
    const float fac = omega / delta;
    float ky = 0.f, kt = 0.f, qt = 0.f, go = 0.f, ty = 0.f;
#pragma unroll
    for (int c = lane; c < D; c += 32) {
        const size_t e = (size_t)row * D + c;
        const float yv = rho[e] * fac, tv = tvec[e], kb = kbar[e];
        yvec[e] = yv;
        dq[e] = tv;
        ky = fmaf(kb, yv, ky);
        kt = fmaf(kb, tv, kt);
        ty = fmaf(tv, yv, ty);
        qt = fmaf(__bfloat162float(q[e]), tv, qt);
        go = fmaf(ld_any(dout, dout_dtype, e), ld_any(out, out_dtype, e), go);
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
        // dL/d(lambda_i): lambda enters C as (e^{-m} / omega) lambda I and dL = t^T dC y
        if (dlambda) dlambda[row] = __expf(-m) / omega * ty;
    }
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
// The pair kernel on the tensor cores (d = 64): the same block-per-key-tile loop with every product a
// warp-level bf16 MMA (m16n8k16, fp32 accumulate).  fp32 operands (y, t, g and the pair coefficients)
// enter as bf16 hi + lo pairs and each product keeps the three leading terms, so the result has fp32-like
// accuracy.  A warp owns 16 of the block's 64 keys and forms the pair tiles transposed ([key][query]):
// their accumulator fragments are then, after packing, the A operands of the dK / dV products with no
// trip through shared memory.  Only scale dL/ds goes to shared memory, for the dQ product.
// ------------------------------------------------------------------------------------------------
// d = 128: the 128 output columns are split over two warps per key (query) group -- a warp's registers
// hold accumulators for 64 columns only -- and both form the same pair tiles.
template <int D>
struct MmCfg {
    static constexpr int LDB = D + 8;             // bf16 row stride of the operand tiles (conflict-free ldmatrix)
    static constexpr int TILE = 64 * LDB;         // bf16 elements per 64-row tile
    static constexpr int NCG = D / 64;            // column groups
    static constexpr int THREADS = 128 * NCG;
    static constexpr int KS = D / 16;             // k-steps of a contraction over the head dimension
    static constexpr size_t PAIRS_SMEM = sizeof(__nv_bfloat16) * (size_t)11 * TILE + sizeof(float) * 6 * 64;
    static constexpr size_t MOMENTS_SMEM = sizeof(__nv_bfloat16) * (size_t)5 * TILE;
};

__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], const __nv_bfloat16* p) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm4t(uint32_t (&r)[4], const __nv_bfloat16* p) {
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (x0, x1) -> packed bf16 pairs hi and lo with x = hi + lo up to 2^-17 relative
__device__ __forceinline__ void split_pack(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
    hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
    lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}
// 64 rows x D columns -> bf16 tile(s) [64][D + 8]; fp32 sources are split into hi and lo tiles
template <int D>
__device__ __forceinline__ void mm_load_bf16(__nv_bfloat16* dst, const __nv_bfloat16* src, size_t row0, int nvalid) {
    for (int idx = threadIdx.x; idx < 64 * (D / 8); idx += MmCfg<D>::THREADS) {
        const int r = idx / (D / 8), c = (idx % (D / 8)) * 8;
        uint4 x = make_uint4(0, 0, 0, 0);
        if (r < nvalid) x = *reinterpret_cast<const uint4*>(src + (row0 + r) * D + c);
        *reinterpret_cast<uint4*>(dst + r * MmCfg<D>::LDB + c) = x;
    }
}
template <int D>
__device__ __forceinline__ void mm_load_split(__nv_bfloat16* hi, __nv_bfloat16* lo, const void* src, int dtype, size_t row0,
                                              int nvalid, int lo_row) {
    constexpr int MM_LDB = MmCfg<D>::LDB;
    for (int idx = threadIdx.x; idx < 64 * (D / 4); idx += MmCfg<D>::THREADS) {
        const int r = idx / (D / 4), c = (idx % (D / 4)) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < nvalid && r >= lo_row) {
            if (dtype == LLA_F32) x = load4(static_cast<const float*>(src) + (row0 + r) * D + c);
            else x = load4(static_cast<const __nv_bfloat16*>(src) + (row0 + r) * D + c);
        }
        uint2 h, l;
        split_pack(x.x, x.y, h.x, l.x);
        split_pack(x.z, x.w, h.y, l.y);
        *reinterpret_cast<uint2*>(hi + r * MM_LDB + c) = h;
        *reinterpret_cast<uint2*>(lo + r * MM_LDB + c) = l;
    }
}

template <int D>
__global__ void __launch_bounds__(MmCfg<D>::THREADS, D == 64 ? 2 : 1)
bwd_pairs_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const void* __restrict__ dout, int dout_dtype,
                     const float* __restrict__ yvec, const float* __restrict__ tvec, const float* __restrict__ rowsc,
                     float* __restrict__ dq, float* __restrict__ dk, float* __restrict__ dv, int n, int first, float scale, int H, int kv_group) {
    constexpr int LDB = MmCfg<D>::LDB, MM_TILE = MmCfg<D>::TILE, MM_THREADS = MmCfg<D>::THREADS, KS = MmCfg<D>::KS;
    extern __shared__ __align__(16) unsigned char mm_smem[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(mm_smem);
    __nv_bfloat16* Vs = Ks + MM_TILE;
    __nv_bfloat16* Qs = Vs + MM_TILE;
    __nv_bfloat16* Gh = Qs + MM_TILE;
    __nv_bfloat16* Gl = Gh + MM_TILE;
    __nv_bfloat16* Yh = Gl + MM_TILE;
    __nv_bfloat16* Yl = Yh + MM_TILE;
    __nv_bfloat16* Th = Yl + MM_TILE;
    __nv_bfloat16* Tl = Th + MM_TILE;
    __nv_bfloat16* DSh = Tl + MM_TILE;      // [key][query]
    __nv_bfloat16* DSl = DSh + MM_TILE;
    float* rs = reinterpret_cast<float*>(DSl + MM_TILE);   // [6][64]: m, 1/omega, gbar, kappa, kbar.y, kbar.t
    const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int warp = (tid >> 5) & 3;      // key group (16 keys); query group in the dQ product
    const int cg = tid >> 7;              // column group (64 output columns)
    const int bh = blockIdx.x;
    const int j0 = blockIdx.y * 64;
    const size_t base = (size_t)bh * n;
    const size_t kvbase = (size_t)kv_unit(bh, H, kv_group) * n;     // grouped heads: the key/value head's rows
    mm_load_bf16<D>(Ks, k, kvbase + j0, min(64, n - j0));
    mm_load_bf16<D>(Vs, v, kvbase + j0, min(64, n - j0));
    // ldmatrix lane offsets: (rows +8 by bit 3, columns +8 by bit 4) and (columns +8 by bit 3, rows +8 by bit 4)
    const int l7 = lane & 7, b3 = (lane >> 3) & 1, b4 = lane >> 4;
    const int offA = (l7 + 8 * b3) * LDB + 8 * b4;     // A operand, or B^T-stored operand read with .trans
    const int offB = (l7 + 8 * b4) * LDB + 8 * b3;     // B operand stored [n][k], or A^T-stored operand read with .trans
    const int kr0 = 16 * warp;
    float adk[8][4] = {}, adv[8][4] = {};
    const int it0 = max(j0, first) / 64, it1 = (n + 63) / 64;
    for (int it = it0; it < it1; ++it) {
        const int i0 = it * 64;
        const int nrow = min(64, n - i0);
        __syncthreads();
        mm_load_bf16<D>(Qs, q, base + i0, nrow);
        mm_load_split<D>(Gh, Gl, dout, dout_dtype, base + i0, nrow, 0);
        mm_load_split<D>(Yh, Yl, yvec, LLA_F32, base + i0, nrow, first - i0);
        mm_load_split<D>(Th, Tl, tvec, LLA_F32, base + i0, nrow, first - i0);
        for (int idx = tid; idx < 6 * 64; idx += MM_THREADS) {
            const int w = idx >> 6, r = idx & 63, gi = i0 + r;
            rs[idx] = (gi < n && gi >= first) ? rowsc[(base + gi) * BW_ROWSC + w] : 0.f;
        }
        __syncthreads();
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
            const int ih = 32 * half;
            float sT[4][4] = {}, eT[4][4] = {}, fT[4][4] = {}, gT[4][4] = {};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t ak[4], av[4];
                ldsm4(ak, Ks + kr0 * LDB + 16 * ks + offA);
                ldsm4(av, Vs + kr0 * LDB + 16 * ks + offA);
#pragma unroll
                for (int nbp = 0; nbp < 2; ++nbp) {
                    const int o = (ih + 16 * nbp) * LDB + 16 * ks + offB;
                    uint32_t b[4];
                    ldsm4(b, Qs + o);
                    mma_bf16(sT[2 * nbp], ak, b[0], b[1]);
                    mma_bf16(sT[2 * nbp + 1], ak, b[2], b[3]);
                    ldsm4(b, Yh + o);
                    mma_bf16(eT[2 * nbp], ak, b[0], b[1]);
                    mma_bf16(eT[2 * nbp + 1], ak, b[2], b[3]);
                    ldsm4(b, Yl + o);
                    mma_bf16(eT[2 * nbp], ak, b[0], b[1]);
                    mma_bf16(eT[2 * nbp + 1], ak, b[2], b[3]);
                    ldsm4(b, Th + o);
                    mma_bf16(fT[2 * nbp], ak, b[0], b[1]);
                    mma_bf16(fT[2 * nbp + 1], ak, b[2], b[3]);
                    ldsm4(b, Tl + o);
                    mma_bf16(fT[2 * nbp], ak, b[0], b[1]);
                    mma_bf16(fT[2 * nbp + 1], ak, b[2], b[3]);
                    ldsm4(b, Gh + o);
                    mma_bf16(gT[2 * nbp], av, b[0], b[1]);
                    mma_bf16(gT[2 * nbp + 1], av, b[2], b[3]);
                    ldsm4(b, Gl + o);
                    mma_bf16(gT[2 * nbp], av, b[0], b[1]);
                    mma_bf16(gT[2 * nbp + 1], av, b[2], b[3]);
                }
            }
            // pair coefficients in place: sT <- a, eT <- scale dL/ds, fT <- p (f - gamma + gbar)
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const int il = ih + 8 * nb + 2 * t4 + (x & 1), gi = i0 + il;
                    const int gj = j0 + kr0 + g + 8 * (x >> 1);
                    const float iom = rs[64 + il];
                    const float p = (iom > 0.f && gj <= gi) ? __expf(fmaf(scale, sT[nb][x], -rs[il])) * iom : 0.f;
                    const float gbar = rs[128 + il], kappa = rs[192 + il];
                    const float ev = eT[nb][x] - rs[256 + il], fv = fT[nb][x] - rs[320 + il], gam = gT[nb][x];
                    sT[nb][x] = p * (1.f - ev);
                    eT[nb][x] = scale * p * (gam * (1.f - ev) + (gbar + fv) * ev - fv - kappa);
                    fT[nb][x] = p * (fv - gam + gbar);
                }
            }
#pragma unroll
            for (int ks2 = 0; ks2 < 2; ++ks2) {
                // A fragments (rows = this warp's keys, k = 16 queries) of a, -a, ds, p1 as hi and lo
                uint32_t ah[4], al[4], nh[4], nl[4], dh[4], dl[4], ph[4], pl[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int nb = 2 * ks2 + (r >> 1), x = 2 * (r & 1);
                    split_pack(sT[nb][x], sT[nb][x + 1], ah[r], al[r]);
                    nh[r] = ah[r] ^ 0x80008000u;
                    nl[r] = al[r] ^ 0x80008000u;
                    split_pack(eT[nb][x], eT[nb][x + 1], dh[r], dl[r]);
                    split_pack(fT[nb][x], fT[nb][x + 1], ph[r], pl[r]);
                    const int row = kr0 + g + 8 * (r & 1), col = ih + 8 * nb + 2 * t4;
                    if (cg == 0) {
                        *reinterpret_cast<uint32_t*>(DSh + row * LDB + col) = dh[r];
                        *reinterpret_cast<uint32_t*>(DSl + row * LDB + col) = dl[r];
                    }
                }
#pragma unroll
                for (int ncp = 0; ncp < 4; ++ncp) {
                    const int o = (ih + 16 * ks2) * LDB + 64 * cg + 16 * ncp + offA;
                    uint32_t b[4], c[4];
                    ldsm4t(b, Gh + o);
                    ldsm4t(c, Gl + o);
                    mma_bf16(adv[2 * ncp], ah, b[0], b[1]);  mma_bf16(adv[2 * ncp + 1], ah, b[2], b[3]);
                    mma_bf16(adv[2 * ncp], al, b[0], b[1]);  mma_bf16(adv[2 * ncp + 1], al, b[2], b[3]);
                    mma_bf16(adv[2 * ncp], ah, c[0], c[1]);  mma_bf16(adv[2 * ncp + 1], ah, c[2], c[3]);
                    ldsm4t(b, Qs + o);
                    mma_bf16(adk[2 * ncp], dh, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], dh, b[2], b[3]);
                    mma_bf16(adk[2 * ncp], dl, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], dl, b[2], b[3]);
                    ldsm4t(b, Yh + o);
                    ldsm4t(c, Yl + o);
                    mma_bf16(adk[2 * ncp], ph, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], ph, b[2], b[3]);
                    mma_bf16(adk[2 * ncp], pl, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], pl, b[2], b[3]);
                    mma_bf16(adk[2 * ncp], ph, c[0], c[1]);  mma_bf16(adk[2 * ncp + 1], ph, c[2], c[3]);
                    ldsm4t(b, Th + o);
                    ldsm4t(c, Tl + o);
                    mma_bf16(adk[2 * ncp], nh, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], nh, b[2], b[3]);
                    mma_bf16(adk[2 * ncp], nl, b[0], b[1]);  mma_bf16(adk[2 * ncp + 1], nl, b[2], b[3]);
                    mma_bf16(adk[2 * ncp], nh, c[0], c[1]);  mma_bf16(adk[2 * ncp + 1], nh, c[2], c[3]);
                }
            }
        }
        __syncthreads();
        // dQ rows 16 warp .. +15 of the tile: sum over the block's 64 keys of (scale dL/ds) k_j
        float adq[8][4] = {};
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t ah[4], al[4];
            ldsm4t(ah, DSh + 16 * ks * LDB + 16 * warp + offB);
            ldsm4t(al, DSl + 16 * ks * LDB + 16 * warp + offB);
#pragma unroll
            for (int ncp = 0; ncp < 4; ++ncp) {
                uint32_t b[4];
                ldsm4t(b, Ks + 16 * ks * LDB + 64 * cg + 16 * ncp + offA);
                mma_bf16(adq[2 * ncp], ah, b[0], b[1]);  mma_bf16(adq[2 * ncp + 1], ah, b[2], b[3]);
                mma_bf16(adq[2 * ncp], al, b[0], b[1]);  mma_bf16(adq[2 * ncp + 1], al, b[2], b[3]);
            }
        }
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int gi = i0 + 16 * warp + g + 8 * (x >> 1);
                if (gi < n && gi >= first) atomicAdd(dq + (base + gi) * D + 64 * cg + 8 * nb + 2 * t4 + (x & 1), adq[nb][x]);
            }
    }
#pragma unroll
    for (int nb = 0; nb < 8; ++nb)
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const int gj = j0 + kr0 + g + 8 * (x >> 1);
            if (gj >= n) continue;
            const size_t e = (kvbase + gj) * D + 64 * cg + 8 * nb + 2 * t4 + (x & 1);
            atomicAdd(dk + e, adk[nb][x]);
            atomicAdd(dv + e, adv[nb][x]);
        }
}

// The moments kernel on the tensor cores (d = 64): a warp owns 16 of the tile's 64 query rows; S = Q K^T
// and Gamma = G V^T accumulate in registers, p and p gamma are packed straight into A fragments (hi + lo)
// and multiply the key tile again for kbar and sum_j p gamma k.
template <int D>
__global__ void __launch_bounds__(MmCfg<D>::THREADS, D == 64 ? 2 : 1)
bwd_moments_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                       const __nv_bfloat16* __restrict__ v, const void* __restrict__ dout, int dout_dtype,
                       const float* __restrict__ stats, float* __restrict__ kbar, float* __restrict__ hvec,
                       float* __restrict__ rowsc, int n, int first, float scale, int H, int kv_group) {
    constexpr int LDB = MmCfg<D>::LDB, MM_TILE = MmCfg<D>::TILE, KS = MmCfg<D>::KS;
    extern __shared__ __align__(16) unsigned char mm_smem[];
    __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(mm_smem);
    __nv_bfloat16* Gh = Qs + MM_TILE;
    __nv_bfloat16* Gl = Gh + MM_TILE;
    __nv_bfloat16* Ks = Gl + MM_TILE;
    __nv_bfloat16* Vs = Ks + MM_TILE;
    const int tid = threadIdx.x, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int warp = (tid >> 5) & 3;      // query group (16 rows)
    const int cg = tid >> 7;              // column group (64 output columns)
    const int tile = gridDim.y - 1 - blockIdx.y;
    const int bh = blockIdx.x;
    const int i0 = tile * 64;
    if (i0 + 64 <= first) return;
    const size_t base = (size_t)bh * n;
    const size_t kvbase = (size_t)kv_unit(bh, H, kv_group) * n;     // grouped heads: the key/value head's rows
    const int nrow = min(64, n - i0);
    mm_load_bf16<D>(Qs, q, base + i0, nrow);
    mm_load_split<D>(Gh, Gl, dout, dout_dtype, base + i0, nrow, 0);
    const int l7 = lane & 7, b3 = (lane >> 3) & 1, b4 = lane >> 4;
    const int offA = (l7 + 8 * b3) * LDB + 8 * b4;
    const int offB = (l7 + 8 * b4) * LDB + 8 * b3;
    const int r0 = 16 * warp;
    float mrow[2], iom[2], gb[2] = {0.f, 0.f};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int gi = i0 + r0 + g + 8 * h;
        const bool okr = gi < n && gi >= first;
        mrow[h] = okr ? stats[(base + gi) * 3 + 0] : 0.f;
        iom[h] = okr ? 1.f / stats[(base + gi) * 3 + 1] : 0.f;
    }
    float akb[8][4] = {}, ah[8][4] = {};
    const int jt_end = (min(n, i0 + 64) + 63) / 64;
    for (int jt = 0; jt < jt_end; ++jt) {
        const int j0 = jt * 64;
        __syncthreads();
        mm_load_bf16<D>(Ks, k, kvbase + j0, min(64, n - j0));
        mm_load_bf16<D>(Vs, v, kvbase + j0, min(64, n - j0));
        __syncthreads();
        float s[8][4] = {}, gm[8][4] = {};
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t aq[4], agh[4], agl[4];
            ldsm4(aq, Qs + r0 * LDB + 16 * ks + offA);
            ldsm4(agh, Gh + r0 * LDB + 16 * ks + offA);
            ldsm4(agl, Gl + r0 * LDB + 16 * ks + offA);
#pragma unroll
            for (int nbp = 0; nbp < 4; ++nbp) {
                uint32_t b[4];
                ldsm4(b, Ks + 16 * nbp * LDB + 16 * ks + offB);
                mma_bf16(s[2 * nbp], aq, b[0], b[1]);
                mma_bf16(s[2 * nbp + 1], aq, b[2], b[3]);
                ldsm4(b, Vs + 16 * nbp * LDB + 16 * ks + offB);
                mma_bf16(gm[2 * nbp], agh, b[0], b[1]);
                mma_bf16(gm[2 * nbp + 1], agh, b[2], b[3]);
                mma_bf16(gm[2 * nbp], agl, b[0], b[1]);
                mma_bf16(gm[2 * nbp + 1], agl, b[2], b[3]);
            }
        }
        // s <- p, gm <- p gamma
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int h = x >> 1, gi = i0 + r0 + g + 8 * h, gj = j0 + 8 * nb + 2 * t4 + (x & 1);
                const float p = (gj <= gi && iom[h] > 0.f) ? __expf(fmaf(scale, s[nb][x], -mrow[h])) * iom[h] : 0.f;
                s[nb][x] = p;
                gm[nb][x] *= p;
                gb[h] += gm[nb][x];
            }
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t ph[4], pl[4], gh[4], gl[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int nb = 2 * ks + (r >> 1), x = 2 * (r & 1);
                split_pack(s[nb][x], s[nb][x + 1], ph[r], pl[r]);
                split_pack(gm[nb][x], gm[nb][x + 1], gh[r], gl[r]);
            }
#pragma unroll
            for (int ncp = 0; ncp < 4; ++ncp) {
                uint32_t b[4];
                ldsm4t(b, Ks + 16 * ks * LDB + 64 * cg + 16 * ncp + offA);
                mma_bf16(akb[2 * ncp], ph, b[0], b[1]);  mma_bf16(akb[2 * ncp + 1], ph, b[2], b[3]);
                mma_bf16(akb[2 * ncp], pl, b[0], b[1]);  mma_bf16(akb[2 * ncp + 1], pl, b[2], b[3]);
                mma_bf16(ah[2 * ncp], gh, b[0], b[1]);   mma_bf16(ah[2 * ncp + 1], gh, b[2], b[3]);
                mma_bf16(ah[2 * ncp], gl, b[0], b[1]);   mma_bf16(ah[2 * ncp + 1], gl, b[2], b[3]);
            }
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        gb[h] += __shfl_xor_sync(0xffffffffu, gb[h], 1);
        gb[h] += __shfl_xor_sync(0xffffffffu, gb[h], 2);
        const int gi = i0 + r0 + g + 8 * h;
        if (gi >= n || gi < first) continue;
        if (t4 == 0 && cg == 0) rowsc[(base + gi) * BW_ROWSC + 2] = gb[h];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            const float kb0 = akb[nb][2 * h], kb1 = akb[nb][2 * h + 1];
            const size_t e = (base + gi) * D + 64 * cg + 8 * nb + 2 * t4;
            *reinterpret_cast<float2*>(kbar + e) = make_float2(kb0, kb1);
            *reinterpret_cast<float2*>(hvec + e) = make_float2(ah[nb][2 * h] - gb[h] * kb0, ah[nb][2 * h + 1] - gb[h] * kb1);
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
                     double scale, double lambda, int* __restrict__ status, float* __restrict__ dlambda, int H, int kv_group) {
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
    const int L = i + 1;
    const size_t base = (size_t)bh * n;
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

// workspace: kbar, h, t, y as [rows][D] fp32, then the scalar records
size_t ws_floats(long long rows, int d, long long heads) {
    (void)heads;
    return (size_t)rows * (4 * (size_t)d + BW_ROWSC);
}

template <int D>
int launch_t(const BackwardArgs& a) {
    using C = BwCfg<D>;
    const long long rows = (long long)a.B * a.H * a.n;
    const int BH = a.B * a.H;
    const int first = max(0, min(a.n, a.head_rows - 1));      // rows [0, first) are solved directly
    const int kvg = a.kv_group > 0 ? a.kv_group : 1;
    const long long kvrows = rows / kvg;                       // rows of k, v, dk, dv
    if (a.workspace_bytes < ws_floats(rows, D, BH) * sizeof(float) || !a.workspace) return LLA_ERR_WORKSPACE;
    if (first > 2 * D) return LLA_ERR_UNSUPPORTED;
    float* kbar = static_cast<float*>(a.workspace);
    float* hvec = kbar + rows * D;
    float* tvec = hvec + rows * D;
    float* yvec = tvec + rows * D;
    float* rowsc = yvec + rows * D;
    const auto* q = static_cast<const __nv_bfloat16*>(a.q);
    const auto* k = static_cast<const __nv_bfloat16*>(a.k);
    const auto* v = static_cast<const __nv_bfloat16*>(a.v);
    const size_t head_smem = head_smem_bytes<D>(first);
    if (head_smem > 227u * 1024u) return LLA_ERR_UNSUPPORTED;
    LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_moments_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::MOMENTS_SMEM));
    LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_pairs_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::PAIRS_SMEM));
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
            q, k, v, a.dout, a.dout_dtype, a.dq, a.dk, a.dv, a.n, first, (double)a.scale, (double)a.lambda, a.status, a.dlambda, a.H, kvg);
        LLA_CUDA_TRY(cudaGetLastError());
        if (forked) LLA_CUDA_TRY(cudaEventRecord(a.join, hs));
    }
    if (first < a.n) {
        const dim3 gm(BH, (a.n + C::BI - 1) / C::BI);
        if (!a.cuda_core_pairs) {
            using M = MmCfg<D>;
            const dim3 gm(BH, (a.n + 63) / 64);
            LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_moments_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)M::MOMENTS_SMEM));
            bwd_moments_mma_kernel<D><<<gm, M::THREADS, M::MOMENTS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, a.stats, kbar, hvec,
                                                                               rowsc, a.n, first, a.scale, a.H, kvg);
        } else {
            bwd_moments_kernel<D><<<gm, BW_THREADS, C::MOMENTS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, a.stats, kbar, hvec,
                                                                              rowsc, a.n, first, a.scale, a.H, kvg);
        }
        LLA_CUDA_TRY(cudaGetLastError());
        // C_i t_i = h_i for the iterative rows: the forward's tensor-core CG with h as right-hand side
        ForwardArgs f = {};
        f.q = a.q; f.k = a.k; f.v = a.v; f.out = nullptr;
        f.B = a.B; f.H = a.H; f.n = a.n; f.d = D; f.dv = D;
        f.in_dtype = LLA_BF16; f.out_dtype = LLA_F32;
        f.scale = a.scale; f.lambda = a.lambda; f.causal = 1;
        f.max_iters = a.max_iters; f.tol = a.tol; f.head_rows = a.head_rows;
        f.status = a.status; f.iters = a.iters; f.stream = a.stream;
        f.ridge_mode = LLA_RIDGE_DEFINITION; f.nq = a.n; f.kv_group = kvg;
        f.rhs = hvec; f.sol = tvec;
        f.set_contiguous();
        // what the workspace holds beyond this pass's own vectors serves the solve (the fp16 copy of k; for
        // d = 128 the row-state slots), so that the backward pass allocates nothing
        const size_t own = (ws_floats(rows, D, BH) * sizeof(float) + 255) & ~(size_t)255;
        if (a.workspace_bytes > own) {
            f.workspace = static_cast<char*>(a.workspace) + own;
            f.workspace_bytes = a.workspace_bytes - own;
        }
        const int rc_pre = forward_tensor_prepass(f);
        if (rc_pre != LLA_OK) return rc_pre;
        const int rc = launch_forward_tensor(f);
        if (rc != LLA_OK) return rc;
        bwd_rowprep_kernel<D><<<(unsigned)((rows + 7) / 8), BW_THREADS, 0, a.stream>>>(
            q, a.out, a.out_dtype, a.dout, a.dout_dtype, a.rho, a.stats, kbar, tvec, yvec, rowsc, a.dq, a.n, first, rows, a.dlambda);
        LLA_CUDA_TRY(cudaGetLastError());
    }
    {
        const dim3 gp(BH, (a.n + BW_BJ - 1) / BW_BJ);
        if (!a.cuda_core_pairs) {
            using M = MmCfg<D>;
            LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_pairs_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)M::PAIRS_SMEM));
            bwd_pairs_mma_kernel<D><<<gp, M::THREADS, M::PAIRS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, yvec, tvec, rowsc, a.dq,
                                                                     a.dk, a.dv, a.n, first, a.scale, a.H, kvg);
        } else {
            bwd_pairs_kernel<D><<<gp, BW_THREADS, C::PAIRS_SMEM, a.stream>>>(q, k, v, a.dout, a.dout_dtype, yvec, tvec, rowsc,
                                                                          a.dq, a.dk, a.dv, a.n, first, a.scale, a.H, kvg);
        }
        LLA_CUDA_TRY(cudaGetLastError());
    }
    if (forked) LLA_CUDA_TRY(cudaStreamWaitEvent(a.stream, a.join, 0));
    return LLA_OK;
}

}  // namespace

size_t backward_workspace_bytes(int B, int H, int n, int d) {
    const size_t own = (ws_floats((long long)B * H * n, d, (long long)B * H) * sizeof(float) + 255) & ~(size_t)255;
    return own + forward_tensor_workspace_bytes(B, H, n, d);
}

int launch_backward(const BackwardArgs& a) {
    if (a.d == 64) return launch_t<64>(a);
    if (a.d == 128) return launch_t<128>(a);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
