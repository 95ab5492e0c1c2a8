// Backward pass of causal local linear attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 inputs,
// d = dv in {64, 128}: the pair sums of the paper's backward appendix in the centred form that lla_backward.cu
// derives (same symbols).  Three kernels share one skeleton -- TMA brings 128B-swizzled bf16 tiles, one warp issues
// the MMAs, eight warps (two threads per TMEM lane) turn score tiles into coefficient tiles:
//
//   bwd_qtile_tc_kernel<D, 0>   per 128-row query tile, over its key blocks of 64:
//                                 S = Q K^T, Gamma = G V^T  ->  p, p gamma  ->  kbar += P K, sum_j p gamma k += (P Gamma) K
//   bwd_qtile_tc_kernel<D, 1>   the same loop with S, E = Y K^T, F = T K^T, Gamma  ->  scale dL/ds  ->  dQ += DS K
//                                 (a query tile owns its rows of dQ: plain stores, the same bits on every run)
//   bwd_ktile_tc_kernel<D>      per 128-key tile, over the later query rows in steps of 64, everything transposed
//                               (keys on the TMEM lanes):  S^T = K Q^T, E^T = K Y^T, F^T = K T^T, Gamma^T = V G^T  ->
//                               a^T, (scale dL/ds)^T, (p (f - gamma + gbar))^T  ->  dV += A^T G,  dK += DS^T Q + P1^T Y - A^T T
//
// Every product of a score tile is an SS MMA of the forward kernel's shape (128 x 64 x d, both operands K-major);
// every product of a coefficient tile takes the coefficients from TMEM, where the compute threads leave them in
// the columns the scores came from, and the other operand MN-major from the tile TMA delivered.  The fp32
// operands (y, t, g and the coefficient tiles) enter as bf16 pairs hi + lo and a product keeps the three leading
// terms, which gives fp32-like accuracy; q, k, v are exact.  y, -t and g come as bf16 arrays written by the row
// preparation kernel (-t, so that "- A^T T" is an accumulation like the others).  In the dQ kernel y sits in TMEM
// (the tile's five other stationary operands fill the shared memory at d = 128).
//
// Score tiles are single-buffered (4 x 64 columns plus the accumulators take all 512 TMEM columns at d = 128), so
// a step is pipelined inside itself: the MMA warp commits the score products in two groups and the compute threads
// hand the coefficient tiles back in two groups, so that each side works on one group while the other side is busy
// with the other.
// All waits are bounded; a wait that expires sets LLA_STATUS_TIMEOUT and the block leaves through the common exit.
#include "lla_sm100.cuh"

namespace lla {
namespace {

using namespace sm100;

constexpr int BT_COMPUTE = 256;       // compute threads (warps 0..7)
constexpr int BT_THREADS = 320;       // + TMA warp (8) + MMA warp (9)
constexpr int BT_TMEM_COLS = 512;
constexpr float BT_LOG2E = 1.4426950408889634f;

constexpr uint32_t BT_IDESC_SS = make_idesc(128, 64, 0, 0);       // score tiles: [128 x 64], both operands K-major

struct BtParams {
    int n, first, H, kv_group;      // n keys; first: the query rows [0, first) are not handled here
    int nq;               // query rows: the positions n - nq .. n - 1 (a chunk of queries; nq = n: the whole sequence)
    int window;           // causal sliding window (0: none): a row sees its last `window` positions
    int head_rows;        // block sparsity: the key blocks that start below this position are always attended
    const unsigned char* block_mask;   // optional [query tiles of 128][key blocks of 64] (+ unit * block_mask_stride), as in the forward
    long long block_mask_stride;
    int has_glo;          // the upstream gradient has a lo half (fp32 dout)
    float scale;
    const float* stats;   // [rows][3] saved by the forward
    const float* pairsc;  // [heads][npair][8] per-row scalars, two rows per record (see bwd_rowprep_kernel)
    int npair;            // records per head: ceil(n / 2)
    const float* yvec;    // [rows][D] fp32
    const float* tvec;    // [rows][D] fp32
    float* rowsc_w;       // moments kernel: gbar goes to slot 2
    float* kbar;
    float* hvec;
    float* dq;
    float* dk;
    float* dv;
    int* status;
    long long wait_clocks;    // cap of every bounded wait, in SM clocks
    int no_loads;             // test aid: the TMA warp issues no copy at all, so that every wait expires with nothing in flight
};

// ------------------------------------------------------------------------------------------------
// dK, dV: one block per (head, 128-key tile)
// ------------------------------------------------------------------------------------------------
template <int D>
struct KtCfg {
    static constexpr int KSUB = D / 64;
    static constexpr int T128 = KSUB * 16384;      // a 128-row operand tile
    static constexpr int T64 = KSUB * 8192;        // a 64-row operand tile
    static constexpr int NST = D == 64 ? 2 : 1;    // stages of the query-side ring
    static constexpr int SM_K = 0, SM_V = T128, SM_ST = 2 * T128;
    static constexpr int ST_Q = 0, ST_YH = T64, ST_YL = 2 * T64, ST_TH = 3 * T64, ST_TL = 4 * T64, ST_GH = 5 * T64, ST_GL = 6 * T64;
    static constexpr int ST_RS = 7 * T64;          // 32 records of 8 floats: the scalars of the step's 64 rows, two rows each
    static constexpr int STAGE = 7 * T64 + 1024;
    static constexpr int SM_BAR = SM_ST + NST * STAGE;
    static constexpr int SM_MISC = SM_BAR + 128;
    static constexpr int SM_ALLOC = SM_MISC + 64 + 1024;
    static constexpr uint32_t IDESC_TS = make_idesc(128, D, 0, 1);      // accumulators: A from TMEM, B MN-major, N = D
    // TMEM columns
    static constexpr int C_S = 0, C_E = 64, C_F = 128, C_G = 192, C_DK = 256, C_DV = 256 + D;
};
static_assert(KtCfg<64>::SM_ALLOC <= 227 * 1024 && KtCfg<128>::SM_ALLOC <= 227 * 1024, "shared memory budget");
// A stage of the query-side ring is loaded and released in two halves: A = the T and G tiles (read last by the
// products of a^T), B = the Q and Y tiles and the row records (read last by the products of ds^T and p1^T).
enum { KB_KV = 0, KB_FULL_A = 1, KB_FULL_B = 3, KB_EMPTY_A = 5, KB_EMPTY_B = 7, KB_SF_SE = 9, KB_SF_FG = 10, KB_PRA = 11, KB_PRB = 12,
       KB_ACCFULL = 13, KB_EXIT = 14, KB_COUNT = 15 };
static_assert(KB_COUNT * 8 <= 128, "barrier area too small");

// one MMA with the A operand in TMEM, predicated on the elected lane
__device__ __forceinline__ void mma_ts1(uint32_t el, uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], [%2], %3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
// bf16 pair of two packed fp32 values: returns the hi word, writes the lo word
__device__ __forceinline__ uint32_t split2(uint64_t v, uint32_t& lo) {
    float a, b;
    upk2(v, a, b);
    return split_bf16x2(a, b, lo);
}
__device__ __forceinline__ uint64_t pku(uint32_t a, uint32_t b) { return pk2(__uint_as_float(a), __uint_as_float(b)); }
__device__ __forceinline__ uint64_t ex2_2(uint64_t t) {
    float a, b;
    upk2(t, a, b);
    return pk2(ex2f(a), ex2f(b));
}

template <int D>
__global__ void __launch_bounds__(BT_THREADS, 1)
bwd_ktile_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmYh,
                    const __grid_constant__ CUtensorMap tmYl, const __grid_constant__ CUtensorMap tmTh,
                    const __grid_constant__ CUtensorMap tmTl, const __grid_constant__ CUtensorMap tmGh,
                    const __grid_constant__ CUtensorMap tmGl, const __grid_constant__ CUtensorMap tmRS, const BtParams prm) {
    using Cfg = KtCfg<D>;
    constexpr int KSUB = Cfg::KSUB, NST = Cfg::NST, STAGE = Cfg::STAGE, T64 = Cfg::T64;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + Cfg::SM_BAR;
    auto bar = [&](int i) { return bars + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + Cfg::SM_MISC);     // [0] tmem base, [2] abort
    volatile int* abort_flag = misc + 2;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x;
    const int kvu = kv_unit(bh, prm.H, prm.kv_group);
    const int n = prm.n, nq = prm.nq, off = n - nq;      // query row i sits at position off + i
    const int j0 = blockIdx.y * 128;          // key tile 0 sees the most query rows and starts first (heads fastest)
    // query steps of 64 rows: from the first row that sees the tile's first key (or the first row these kernels
    // handle) to the last row that still sees a key of the tile
    const int W = prm.window;
    const int last_row = W > 0 ? min(nq - 1, j0 + 127 + W - 1 - off) : nq - 1;
    const int it0 = max(max(j0 - off, 0), prm.first) / 64, it1 = last_row < 0 ? 0 : last_row / 64 + 1;
    const int nstep = it1 - it0;
    const long long wcap = prm.wait_clocks;
    if (nstep <= 0) return;
    // Block sparsity (the forward's rule): query tile t = rows 128 t .. 128 t + 127 attends to key block c = keys
    // 64 c .. 64 c + 63 if the mask says so, if the block starts below head_rows or if it is a diagonal block of the
    // tile.  This tile's keys are the blocks 2 J and 2 J + 1 (TMEM lanes 0..63 and 64..127): bit 0 and bit 1 of the
    // result.  A step (64 query rows) with neither is skipped by every role; g counts the steps taken.
    const unsigned char* bmask = prm.block_mask ? prm.block_mask + (size_t)bh * prm.block_mask_stride : nullptr;
    const int nblk_all = (n + 63) / 64;
    auto blocks_on = [&](int i0) -> int {
        if (!bmask) return 3;
        const int t = i0 >> 7, c0 = (int)(2 * blockIdx.y);
        int r = 0;
        for (int x = 0; x < 2; ++x) {
            const int c = c0 + x;
            if (c < nblk_all && (bmask[(size_t)t * nblk_all + c] != 0 || c * 64 < prm.head_rows || c * 64 + 63 >= off + 128 * t)) r |= 1 << x;
        }
        return r;
    };

    if (tid == 0) {
        mbar_init(bar(KB_KV), 1);
        for (int s = 0; s < NST; ++s) {
            mbar_init(bar(KB_FULL_A + s), 1);
            mbar_init(bar(KB_FULL_B + s), 1);
            mbar_init(bar(KB_EMPTY_A + s), 1);
            mbar_init(bar(KB_EMPTY_B + s), 1);
        }
        mbar_init(bar(KB_SF_SE), 1);
        mbar_init(bar(KB_SF_FG), 1);
        mbar_init(bar(KB_PRA), BT_COMPUTE / 32);
        mbar_init(bar(KB_PRB), BT_COMPUTE / 32);
        mbar_init(bar(KB_ACCFULL), 1);
        mbar_init(bar(KB_EXIT), 1);
        misc[2] = 0;
        fence_barrier_init();
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(sbase + Cfg::SM_MISC), "r"(BT_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[0];

    if (warp == 8) {
        // ================================ TMA producer ================================
        if (lane == 0 && !prm.no_loads) {
            mbar_expect_tx(bar(KB_KV), 2 * Cfg::T128);
            for (int sub = 0; sub < KSUB; ++sub) {
                tma_load_3d(sbase + Cfg::SM_K + sub * 16384, &tmK, bar(KB_KV), 64 * sub, j0, kvu);
                tma_load_3d(sbase + Cfg::SM_V + sub * 16384, &tmV, bar(KB_KV), 64 * sub, j0, kvu);
            }
            int issued_a = 0, issued_b = 0;
            for (int it = it0, g = 0; it < it1; ++it) {
                const int i0 = 64 * it;
                if (!blocks_on(i0)) continue;
                const int s = g % NST;
                const uint32_t st = sbase + Cfg::SM_ST + s * STAGE;
                if (!mbar_wait(bar(KB_EMPTY_A + s), ((g / NST) & 1) ^ 1, abort_flag, wcap)) break;
                const uint32_t fa = bar(KB_FULL_A + s);
                mbar_expect_tx(fa, (3 + (prm.has_glo ? 1 : 0)) * T64);
                for (int sub = 0; sub < KSUB; ++sub) {
                    tma_load_3d(st + Cfg::ST_TH + sub * 8192, &tmTh, fa, 64 * sub, i0, bh);
                    tma_load_3d(st + Cfg::ST_TL + sub * 8192, &tmTl, fa, 64 * sub, i0, bh);
                    tma_load_3d(st + Cfg::ST_GH + sub * 8192, &tmGh, fa, 64 * sub, i0, bh);
                    if (prm.has_glo) tma_load_3d(st + Cfg::ST_GL + sub * 8192, &tmGl, fa, 64 * sub, i0, bh);
                }
                issued_a = g + 1;
                if (!mbar_wait(bar(KB_EMPTY_B + s), ((g / NST) & 1) ^ 1, abort_flag, wcap)) break;
                const uint32_t fb = bar(KB_FULL_B + s);
                mbar_expect_tx(fb, 3 * T64 + 1024);
                for (int sub = 0; sub < KSUB; ++sub) {
                    tma_load_3d(st + Cfg::ST_Q + sub * 8192, &tmQ, fb, 64 * sub, i0, bh);
                    tma_load_3d(st + Cfg::ST_YH + sub * 8192, &tmYh, fb, 64 * sub, i0, bh);
                    tma_load_3d(st + Cfg::ST_YL + sub * 8192, &tmYl, fb, 64 * sub, i0, bh);
                }
                tma_load_3d(st + Cfg::ST_RS, &tmRS, fb, 0, i0 / 2, bh);
                issued_b = ++g;
            }
            if (*abort_flag) {      // an aborted block: what was issued must have landed before the block exits
                (void)mbar_wait_landed(bar(KB_KV), 0, wcap);
                for (int g = max(0, issued_a - NST); g < issued_a; ++g) (void)mbar_wait_landed(bar(KB_FULL_A + g % NST), (g / NST) & 1, wcap);
                for (int g = max(0, issued_b - NST); g < issued_b; ++g) (void)mbar_wait_landed(bar(KB_FULL_B + g % NST), (g / NST) & 1, wcap);
            }
        }
    } else if (warp == 9) {
        // ================================ MMA issuer ================================
        const uint32_t el = elect_one();
        const uint32_t sb_u = __shfl_sync(0xffffffffu, sbase, 0);
        const uint32_t tm_u = __shfl_sync(0xffffffffu, tmem, 0);
        bool ok = mbar_wait(bar(KB_KV), 0, abort_flag, wcap);
        const uint64_t kdesc = make_desc(sb_u + Cfg::SM_K), vdesc = make_desc(sb_u + Cfg::SM_V);
        for (int it = it0, g = 0; it < it1 && ok; ++it) {
            if (!blocks_on(64 * it)) continue;
            const int s = g % NST;
            const uint32_t st = sb_u + Cfg::SM_ST + s * STAGE;
            auto score = [&](uint32_t col, uint64_t adesc, int off, uint32_t acc) {
                const uint64_t bdesc = make_desc(st + off);
#pragma unroll
                for (int sub = 0; sub < KSUB; ++sub)
                    mma_ss_k64(el, tm_u + col, adesc + sub * (16384 >> 4), bdesc + sub * (8192 >> 4), BT_IDESC_SS, acc | (sub > 0));
            };
            // Two groups of score products: (S, E), which a^T needs, and (F, Gamma).  With two stages (S, E) go
            // first, so that a^T is formed while (F, Gamma) run.  With one stage (d = 128) the order is reversed: half A
            // of the stage was released first by the previous step and lands first, and the wait for half B hides
            // behind the products of half A.
            auto group_se = [&]() -> bool {
                if (!mbar_wait(bar(KB_FULL_B + s), (g / NST) & 1, abort_flag, wcap)) return false;
                tc_fence_after();
                score(Cfg::C_S, kdesc, Cfg::ST_Q, 0);
                score(Cfg::C_E, kdesc, Cfg::ST_YH, 0);
                score(Cfg::C_E, kdesc, Cfg::ST_YL, 1);
                tc_commit_el(el, bar(KB_SF_SE));
                return true;
            };
            auto group_fg = [&]() -> bool {
                if (!mbar_wait(bar(KB_FULL_A + s), (g / NST) & 1, abort_flag, wcap)) return false;
                tc_fence_after();
                score(Cfg::C_F, kdesc, Cfg::ST_TH, 0);
                score(Cfg::C_F, kdesc, Cfg::ST_TL, 1);
                score(Cfg::C_G, vdesc, Cfg::ST_GH, 0);
                if (prm.has_glo) score(Cfg::C_G, vdesc, Cfg::ST_GL, 1);
                tc_commit_el(el, bar(KB_SF_FG));
                return true;
            };
            if (NST > 1) {
                if (!group_se() || !group_fg()) break;
            } else {
                if (!group_fg() || !group_se()) break;
            }
            // coefficient tiles (hi + lo pairs) sit where the scores were: a^T in S, then ds^T in E and p1^T in F
            auto bd = [&](int off) { return make_desc(st + off, 8192); };
            const uint32_t acc = g > 0;
            if (!mbar_wait(bar(KB_PRA), g & 1, abort_flag, wcap)) break;
            tc_fence_after();
            mma_ts_hilo_k64(el, tm_u + Cfg::C_DV, tm_u + Cfg::C_S, bd(Cfg::ST_GH), Cfg::IDESC_TS, acc);
            if (prm.has_glo) mma_ts_hi_k64(el, tm_u + Cfg::C_DV, tm_u + Cfg::C_S, bd(Cfg::ST_GL), Cfg::IDESC_TS, 1);
            mma_ts_hilo_k64(el, tm_u + Cfg::C_DK, tm_u + Cfg::C_S, bd(Cfg::ST_TH), Cfg::IDESC_TS, acc);
            mma_ts_hi_k64(el, tm_u + Cfg::C_DK, tm_u + Cfg::C_S, bd(Cfg::ST_TL), Cfg::IDESC_TS, 1);
            tc_commit_el(el, bar(KB_EMPTY_A + s));
            if (!mbar_wait(bar(KB_PRB), g & 1, abort_flag, wcap)) break;
            tc_fence_after();
            mma_ts_hilo_k64(el, tm_u + Cfg::C_DK, tm_u + Cfg::C_E, bd(Cfg::ST_Q), Cfg::IDESC_TS, 1);
            mma_ts_hilo_k64(el, tm_u + Cfg::C_DK, tm_u + Cfg::C_F, bd(Cfg::ST_YH), Cfg::IDESC_TS, 1);
            mma_ts_hi_k64(el, tm_u + Cfg::C_DK, tm_u + Cfg::C_F, bd(Cfg::ST_YL), Cfg::IDESC_TS, 1);
            tc_commit_el(el, bar(KB_EMPTY_B + s));
            ++g;
        }
        tc_commit_el(el, bar(KB_ACCFULL));      // the last step's products (the diagonal steps are always taken)
        if (*abort_flag) {      // an aborted block: the MMAs issued above must be done before TMEM and shared memory go
            tc_commit_el(el, bar(KB_EXIT));
            (void)mbar_wait_landed(bar(KB_EXIT), 0, wcap);
        }
    } else {
        // ================================ compute warps ================================
        const int quad = warp & 3, half = warp >> 2;
        const int lrow = quad * 32 + lane;            // key inside the tile == TMEM lane
        const int gj = j0 + lrow;
        const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
        const float c1 = prm.scale * BT_LOG2E;
        const uint64_t c1c1 = pk2(c1, c1), one2 = pk2(1.f, 1.f), sc2 = pk2(prm.scale, prm.scale);
        bool ok = true;
        for (int it = it0, g = 0; it < it1; ++it) {
            const int i0 = 64 * it;
            const int on = blocks_on(i0);
            if (!on) continue;
            const bool lane_on = (on >> (lrow >> 6)) & 1;      // this lane's key block is attended by the step's query tile
            const int s = g % NST;
            if (!mbar_wait(bar(KB_FULL_B + s), (g / NST) & 1, abort_flag, wcap)) { ok = false; break; }      // the row records
            if (!mbar_wait(bar(KB_SF_SE), g & 1, abort_flag, wcap)) { ok = false; break; }
            tc_fence_after();
            // records of this thread's 32 query rows (16 pairs): (nm2, nm2, kbar.y, kbar.y), (gk, gk, kk, kk)
            const float4* rsp = reinterpret_cast<const float4*>(smem + Cfg::SM_ST + s * STAGE + Cfg::ST_RS) + 32 * half;
            const uint32_t col0 = 32 * half;
            uint64_t p2[16], e2v[16];
            {
                // a = p (1 - e) from S and E: p = 2^(c1 s + nm2) carries 1 / omega; rows switched off have nm2 = -1e30
                uint32_t sv[32], ev[32], pa[32];
                tmem_ld32(tm_lane + Cfg::C_S + col0, sv);
                tmem_ld32(tm_lane + Cfg::C_E + col0, ev);
                tc_wait_ld();
                if (off + i0 < j0 + 128 || i0 + 64 > nq || (W > 0 && off + i0 + 63 - j0 >= W) || on != 3) {
                    // a diagonal or last step, one that reaches past the window or one with a key block left out: hide
                    // the pairs with j > position, row >= nq or position - j >= window, and the lanes of the block that
                    // is not attended
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int gi = i0 + (int)col0 + e, pos = off + gi;
                        if (gj > pos || gi >= nq || (W > 0 && pos - gj >= W) || !lane_on) sv[e] = __float_as_uint(-1e30f);
                    }
                }
#pragma unroll
                for (int e2 = 0; e2 < 16; ++e2) {
                    const float4 ra = rsp[2 * e2];
                    const uint64_t p = ex2_2(fma2(pku(sv[2 * e2], sv[2 * e2 + 1]), c1c1, pk2(ra.x, ra.y)));
                    const uint64_t evv = sub2(pku(ev[2 * e2], ev[2 * e2 + 1]), pk2(ra.z, ra.w));
                    const int ks = e2 >> 3, e = e2 & 7;
                    pa[ks * 16 + e] = split2(mul2(p, sub2(one2, evv)), pa[ks * 16 + 8 + e]);
                    p2[e2] = p;
                    e2v[e2] = evv;
                }
                tmem_st32(tm_lane + Cfg::C_S + col0, pa);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(KB_PRA));
            }
            if (!mbar_wait(bar(KB_SF_FG), g & 1, abort_flag, wcap)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int chunk = 0; chunk < 2; ++chunk) {
                // with u = gbar - f (the F tile holds (-t) . k, so u = gk - F with gk = gbar - kbar.t):
                //   p1 = p (u - gamma),  ds = scale p (gamma (1 - e) + u e + F + kk),  kk = kbar.t - kappa
                uint32_t fv[16], gv[16], pd[16], pp[16];
                tmem_ld16(tm_lane + Cfg::C_F + col0 + 16 * chunk, fv);
                tmem_ld16(tm_lane + Cfg::C_G + col0 + 16 * chunk, gv);
                tc_wait_ld();
#pragma unroll
                for (int e2 = 0; e2 < 8; ++e2) {
                    const int idx = 8 * chunk + e2;
                    const float4 rb = rsp[2 * idx + 1];
                    const uint64_t f2 = pku(fv[2 * e2], fv[2 * e2 + 1]), g2 = pku(gv[2 * e2], gv[2 * e2 + 1]);
                    const uint64_t u = sub2(pk2(rb.x, rb.y), f2);
                    const uint64_t inner = fma2(g2, sub2(one2, e2v[idx]), fma2(u, e2v[idx], add2(f2, pk2(rb.z, rb.w))));
                    pd[e2] = split2(mul2(mul2(p2[idx], sc2), inner), pd[8 + e2]);
                    pp[e2] = split2(mul2(p2[idx], sub2(u, g2)), pp[8 + e2]);
                }
                tmem_st16(tm_lane + Cfg::C_E + col0 + 16 * chunk, pd);
                tmem_st16(tm_lane + Cfg::C_F + col0 + 16 * chunk, pp);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(KB_PRB));
            ++g;
        }
        if (ok && mbar_wait(bar(KB_ACCFULL), 0, abort_flag, wcap)) {
            tc_fence_after();
            // Key rows below `first` also get the directly-solved rows' shares (from another stream), and with grouped
            // heads every query head of the group adds into the same rows: those are added atomically.  Any other
            // row is this block's alone and is stored.
            const bool plain = prm.kv_group == 1 && (prm.first == 0 || j0 >= off + prm.first);
            const size_t rowoff = ((size_t)kvu * n + gj) * D + half * (D / 2);
            const bool inb = gj < n && LLA_IN_BOUNDS((size_t)kvu * n + gj, (size_t)(gridDim.x / prm.kv_group) * n, prm.status, 702);
#pragma unroll 1
            for (int part = 0; part < 2; ++part) {
                float* dst = (part == 0 ? prm.dk : prm.dv) + rowoff;
#pragma unroll 1
                for (int cb = 0; cb < D / 2; cb += 32) {
                    uint32_t v[32];
                    tmem_ld32(tm_lane + (part == 0 ? Cfg::C_DK : Cfg::C_DV) + half * (D / 2) + cb, v);
                    tc_wait_ld();
                    if (!inb) continue;
                    if (plain) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            *reinterpret_cast<float4*>(dst + cb + e) = make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]),
                                                                                   __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) atomicAdd(dst + cb + e, __uint_as_float(v[e]));
                    }
                }
            }
        }
    }
    // ================================ common exit ================================
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(BT_TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag && prm.status) atomicAdd(prm.status + LLA_STATUS_TIMEOUT, 1);
}

// ------------------------------------------------------------------------------------------------
// Query-tile kernels: MODE 0 = moments (kbar, gbar, h), MODE 1 = dQ
// ------------------------------------------------------------------------------------------------
template <int D>
struct QtCfg {
    static constexpr int KSUB = D / 64;
    static constexpr int T128 = KSUB * 16384, T64 = KSUB * 8192;
    static constexpr int SM_Q = 0, SM_GH = T128, SM_GL = 2 * T128, SM_TH = 3 * T128, SM_TL = 4 * T128;
    static constexpr int SM_KV = 5 * T128;         // stage 0: K block, V block.  A second stage: see stage_base()
    static constexpr int STAGE = 2 * T64;
    static constexpr int NST_FIXED = D == 64 ? 3 : 2;      // stages at SM_KV
    static constexpr int SM_RED = SM_KV + NST_FIXED * STAGE;        // 2 x 128 floats
    static constexpr int SM_BAR = SM_RED + 1024;
    static constexpr int SM_MISC = SM_BAR + 128;
    static constexpr int SM_BITS = SM_MISC + 64;      // block sparsity: one bit per key block of the tile (n <= 65536)
    static constexpr int SM_ALLOC = SM_BITS + 128 + 1024;
    static constexpr uint32_t IDESC_TS = make_idesc(128, D, 0, 1);
    // TMEM columns.  MODE 1: S, E, F, Gamma, dQ, then y as bf16 pairs (hi D / 2 columns, lo D / 2 columns)
    static constexpr int C_S = 0, C_E = 64, C_F = 128, C_G1 = 192, C_DQ = 256, C_Y = 384;
    // MODE 0: S, Gamma, kbar, sum p gamma k
    static constexpr int C_G0 = 64, C_KB = 128, C_H = 128 + D;
};
static_assert(QtCfg<64>::SM_ALLOC <= 227 * 1024 && QtCfg<128>::SM_ALLOC <= 227 * 1024, "shared memory budget");
enum { QB_QFULL = 0, QB_YREADY = 1, QB_FULL = 2, QB_EMPTY = 5, QB_SF1 = 8, QB_SF2 = 9, QB_PRA = 10, QB_PRB = 11, QB_ACCFULL = 12,
       QB_EXIT = 13, QB_COUNT = 14 };

template <int D, int MODE>
__global__ void __launch_bounds__(BT_THREADS, 1)
bwd_qtile_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmGh,
                    const __grid_constant__ CUtensorMap tmGl, const __grid_constant__ CUtensorMap tmTh,
                    const __grid_constant__ CUtensorMap tmTl, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const BtParams prm) {
    using Cfg = QtCfg<D>;
    constexpr int KSUB = Cfg::KSUB, STAGE = Cfg::STAGE, T64 = Cfg::T64, T128 = Cfg::T128;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + Cfg::SM_BAR;
    auto bar = [&](int i) { return bars + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + Cfg::SM_MISC);
    volatile int* abort_flag = misc + 2;
    float* red = reinterpret_cast<float*>(smem + Cfg::SM_RED);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x;
    const int kvu = kv_unit(bh, prm.H, prm.kv_group);
    const int n = prm.n, nq = prm.nq, off = n - nq;      // query row i sits at position off + i
    const int tile = gridDim.y - 1 - blockIdx.y;      // longest tiles first, heads fastest
    const int i0 = tile * 128;
    if (i0 + 128 <= prm.first) return;                // every row of the tile is solved directly
    // key blocks [cbeg, cend): with a sliding window the loop starts at the block of the first row's first visible key
    const int W = prm.window;
    const int cend = (off + min(nq, i0 + 128) + 63) / 64;
    const int cbeg = W > 0 ? max(0, off + i0 + 1 - W) / 64 : 0;
    const long long wcap = prm.wait_clocks;
    // Block sparsity: the loops visit only the key blocks that the mask lists for this query tile, plus the ones that
    // are always attended (the forward's rule): the blocks of the first head_rows keys and the tile's diagonal blocks.
    // Every role walks the blocks in order and skips the same ones; c counts the blocks visited.
    const bool sparse = prm.block_mask != nullptr;
    uint32_t* bits = reinterpret_cast<uint32_t*>(smem + Cfg::SM_BITS);
    if (sparse && tid < 32) {
        const unsigned char* mrow = prm.block_mask + (size_t)bh * prm.block_mask_stride + (size_t)tile * ((n + 63) / 64);
        uint32_t word = 0;
        for (int b = 0; b < 32; ++b) {
            const int cb = 32 * tid + b;
            if (cb < cend && (mrow[cb] != 0 || cb * 64 < prm.head_rows || cb * 64 + 63 >= off + i0)) word |= 1u << b;
        }
        bits[tid] = word;
    }
    auto block_on = [&](int cb) { return !sparse || ((bits[cb >> 5] >> (cb & 31)) & 1u) != 0; };
    // Stages of the K/V ring.  d = 128: the tiles that stay for the whole block leave room for two stages; a third one
    // takes the place of a tile that is not loaded (the upstream gradient's lo half when it comes in bf16; the T tiles
    // in the moments kernel).
    const int nst = D == 64 ? 3 : (MODE == 0 ? 3 : (prm.has_glo ? 2 : 3));
    auto stage_base = [&](int s) -> uint32_t {
        if (D == 64 || s < 2) return Cfg::SM_KV + s * STAGE;
        return MODE == 0 ? Cfg::SM_TH : Cfg::SM_GL;
    };
    static_assert(D == 64 || QtCfg<D>::STAGE == QtCfg<D>::T128, "a d = 128 stage takes the place of one stationary tile");

    if (tid == 0) {
        mbar_init(bar(QB_QFULL), 1);
        mbar_init(bar(QB_YREADY), BT_COMPUTE / 32);
        for (int s = 0; s < 3; ++s) {
            mbar_init(bar(QB_FULL + s), 1);
            mbar_init(bar(QB_EMPTY + s), 1);
        }
        mbar_init(bar(QB_SF1), 1);
        mbar_init(bar(QB_SF2), 1);
        mbar_init(bar(QB_PRA), BT_COMPUTE / 32);
        mbar_init(bar(QB_PRB), BT_COMPUTE / 32);
        mbar_init(bar(QB_ACCFULL), 1);
        mbar_init(bar(QB_EXIT), 1);
        misc[2] = 0;
        fence_barrier_init();
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(sbase + Cfg::SM_MISC), "r"(BT_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[0];

    if (warp == 8) {
        // ================================ TMA producer ================================
        if (lane == 0 && !prm.no_loads) {
            const int ntile = (MODE == 1 ? 4 : 2) + (prm.has_glo ? 1 : 0);
            mbar_expect_tx(bar(QB_QFULL), ntile * T128);
            for (int sub = 0; sub < KSUB; ++sub) {
                tma_load_3d(sbase + Cfg::SM_Q + sub * 16384, &tmQ, bar(QB_QFULL), 64 * sub, i0, bh);
                tma_load_3d(sbase + Cfg::SM_GH + sub * 16384, &tmGh, bar(QB_QFULL), 64 * sub, i0, bh);
                if (prm.has_glo) tma_load_3d(sbase + Cfg::SM_GL + sub * 16384, &tmGl, bar(QB_QFULL), 64 * sub, i0, bh);
                if (MODE == 1) {
                    tma_load_3d(sbase + Cfg::SM_TH + sub * 16384, &tmTh, bar(QB_QFULL), 64 * sub, i0, bh);
                    tma_load_3d(sbase + Cfg::SM_TL + sub * 16384, &tmTl, bar(QB_QFULL), 64 * sub, i0, bh);
                }
            }
            int issued = 0;
            for (int cb = cbeg, c = 0; cb < cend; ++cb) {
                if (!block_on(cb)) continue;
                const int s = c % nst;
                if (!mbar_wait(bar(QB_EMPTY + s), ((c / nst) & 1) ^ 1, abort_flag, wcap)) break;
                const uint32_t st = sbase + stage_base(s), fb = bar(QB_FULL + s);
                mbar_expect_tx(fb, STAGE);
                for (int sub = 0; sub < KSUB; ++sub) {
                    tma_load_3d(st + sub * 8192, &tmK, fb, 64 * sub, 64 * cb, kvu);
                    tma_load_3d(st + T64 + sub * 8192, &tmV, fb, 64 * sub, 64 * cb, kvu);
                }
                issued = ++c;
            }
            if (*abort_flag) {
                (void)mbar_wait_landed(bar(QB_QFULL), 0, wcap);
                for (int c = max(0, issued - nst); c < issued; ++c) (void)mbar_wait_landed(bar(QB_FULL + c % nst), (c / nst) & 1, wcap);
            }
        }
    } else if (warp == 9) {
        // ================================ MMA issuer ================================
        const uint32_t el = elect_one();
        const uint32_t sb_u = __shfl_sync(0xffffffffu, sbase, 0);
        const uint32_t tm_u = __shfl_sync(0xffffffffu, tmem, 0);
        bool ok = mbar_wait(bar(QB_QFULL), 0, abort_flag, wcap);
        if (MODE == 1) ok = ok && mbar_wait(bar(QB_YREADY), 0, abort_flag, wcap);
        tc_fence_after();
        auto next_block = [&](int cb) { while (cb < cend && !block_on(cb)) ++cb; return cb; };
        auto score = [&](uint32_t st, uint32_t col, int aoff, bool v_tile, uint32_t acc) {
            const uint64_t adesc = make_desc(sb_u + aoff), bdesc = make_desc(st + (v_tile ? T64 : 0));
#pragma unroll
            for (int sub = 0; sub < KSUB; ++sub)
                mma_ss_k64(el, tm_u + col, adesc + sub * (16384 >> 4), bdesc + sub * (8192 >> 4), BT_IDESC_SS, acc | (sub > 0));
        };
        // S = Q K^T of visited block number c (waits for its stage); the weights can be formed as soon as it is done
        auto issue_s = [&](int c) -> bool {
            const int s = c % nst;
            if (!mbar_wait(bar(QB_FULL + s), (c / nst) & 1, abort_flag, wcap)) return false;
            tc_fence_after();
            score(sb_u + stage_base(s), Cfg::C_S, Cfg::SM_Q, false, 0);
            tc_commit_el(el, bar(QB_SF1));
            return true;
        };
        auto issue_g = [&](int c) {
            const uint32_t st = sb_u + stage_base(c % nst), cg = MODE == 1 ? Cfg::C_G1 : Cfg::C_G0;
            score(st, cg, Cfg::SM_GH, true, 0);
            if (prm.has_glo) score(st, cg, Cfg::SM_GL, true, 1);
        };
        // The score products of the next block are issued as early as the columns they overwrite allow: S as soon as
        // the compute warps have read the current S (they signal it on PRA: with the weights stored in the moments
        // kernel, after the read in the dQ kernel, whose coefficient tile goes to the E columns), Gamma in the moments
        // kernel right after the product that read the current one.  The tensor pipe runs its instructions in order,
        // so a product issued after the one that reads a tile may overwrite that tile.
        int cb = next_block(cbeg);
        ok = ok && cb < cend && issue_s(0);
        if (ok && MODE == 0) {
            issue_g(0);
            tc_commit_el(el, bar(QB_SF2));
        }
        for (int c = 0; ok && cb < cend; ++c) {
            const int s = c % nst;
            const uint32_t st = sb_u + stage_base(s);
            const uint64_t kdesc = make_desc(st);
            const uint64_t kmn = make_desc(st, 8192);       // the K block read MN-major, N = D
            const int nb = next_block(cb + 1);
            if (MODE == 1) {
                // E = Y K^T with y (hi, then lo) from TMEM: D / 16 steps of 8 columns each
#pragma unroll
                for (int part = 0; part < 2; ++part)
#pragma unroll
                    for (int sub = 0; sub < KSUB; ++sub)
                        mma_ts_kmajor_k64(el, tm_u + Cfg::C_E, tm_u + Cfg::C_Y + part * (D / 2) + 32 * sub, kdesc + sub * (8192 >> 4),
                                          BT_IDESC_SS, (part | sub) > 0);
                score(st, Cfg::C_F, Cfg::SM_TH, false, 0);
                score(st, Cfg::C_F, Cfg::SM_TL, false, 1);
                issue_g(c);
                tc_commit_el(el, bar(QB_SF2));
                if (nb < cend) {
                    if (!mbar_wait(bar(QB_PRA), c & 1, abort_flag, wcap)) break;      // S of this block has been read
                    if (!issue_s(c + 1)) break;
                }
                if (!mbar_wait(bar(QB_PRB), c & 1, abort_flag, wcap)) break;
                tc_fence_after();
                mma_ts_hilo_k64(el, tm_u + Cfg::C_DQ, tm_u + Cfg::C_E, kmn, Cfg::IDESC_TS, c > 0);
                tc_commit_el(el, bar(QB_EMPTY + s));
            } else {
                if (!mbar_wait(bar(QB_PRA), c & 1, abort_flag, wcap)) break;
                tc_fence_after();
                mma_ts_hilo_k64(el, tm_u + Cfg::C_KB, tm_u + Cfg::C_S, kmn, Cfg::IDESC_TS, c > 0);
                if (nb < cend && !issue_s(c + 1)) break;
                if (!mbar_wait(bar(QB_PRB), c & 1, abort_flag, wcap)) break;
                tc_fence_after();
                mma_ts_hilo_k64(el, tm_u + Cfg::C_H, tm_u + Cfg::C_G0, kmn, Cfg::IDESC_TS, c > 0);
                tc_commit_el(el, bar(QB_EMPTY + s));
                if (nb < cend) {
                    issue_g(c + 1);
                    tc_commit_el(el, bar(QB_SF2));
                }
            }
            cb = nb;
        }
        tc_commit_el(el, bar(QB_ACCFULL));      // the last block's products (at least the diagonal blocks were visited)
        if (*abort_flag) {
            tc_commit_el(el, bar(QB_EXIT));
            (void)mbar_wait_landed(bar(QB_EXIT), 0, wcap);
        }
    } else {
        // ================================ compute warps ================================
        const int quad = warp & 3, half = warp >> 2;
        const int lrow = quad * 32 + lane;            // query row inside the tile == TMEM lane
        const int gi = i0 + lrow;
        const size_t row = (size_t)bh * nq + gi;
        const bool okr = gi < nq && gi >= prm.first && LLA_IN_BOUNDS(row, (size_t)gridDim.x * nq, prm.status, 701);
        const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
        const float c1 = prm.scale * BT_LOG2E;
        // per-row scalars (see bwd_rowprep_kernel): p = 2^(c1 s + nm2) carries 1 / omega; a row that is switched off
        // has nm2 = -1e30 and no weight
        float nm2 = -1e30f, ky = 0.f, gk = 0.f, kk = 0.f;
        if (okr) {
            if (MODE == 1) {
                const float* rp = prm.pairsc + ((size_t)bh * prm.npair + (gi >> 1)) * 8 + (gi & 1);
                nm2 = rp[0]; ky = rp[2]; gk = rp[4]; kk = rp[6];
            } else {
                nm2 = -(prm.stats[row * 3 + 0] * BT_LOG2E + log2f(prm.stats[row * 3 + 1]));
            }
        }
        const uint64_t c1c1 = pk2(c1, c1), nm22 = pk2(nm2, nm2), one2 = pk2(1.f, 1.f), sc2 = pk2(prm.scale, prm.scale);
        const uint64_t ky2 = pk2(ky, ky), gk2 = pk2(gk, gk), kk2 = pk2(kk, kk);
        if (MODE == 1) {
            // this thread's half of y_i -> bf16 pairs in TMEM: 16-element steps of 8 columns, hi block then lo block
            constexpr int NW = D / 4;      // packed words per half row and part
            uint32_t yh[NW], yl[NW];
#pragma unroll
            for (int e = 0; e < NW; e += 2) {
                float4 y4 = make_float4(0.f, 0.f, 0.f, 0.f);
                if (okr) y4 = *reinterpret_cast<const float4*>(prm.yvec + row * D + half * (D / 2) + 2 * e);
                yh[e] = split_bf16x2(y4.x, y4.y, yl[e]);
                yh[e + 1] = split_bf16x2(y4.z, y4.w, yl[e + 1]);
            }
            if constexpr (NW == 16) {
                tmem_st16(tm_lane + Cfg::C_Y + half * NW, yh);
                tmem_st16(tm_lane + Cfg::C_Y + D / 2 + half * NW, yl);
            } else {
                tmem_st32(tm_lane + Cfg::C_Y + half * NW, yh);
                tmem_st32(tm_lane + Cfg::C_Y + D / 2 + half * NW, yl);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(QB_YREADY));
        }
        uint64_t gb2 = pk2(0.f, 0.f);
        bool ok = true;
        for (int cb = cbeg, c = 0; cb < cend; ++cb) {
            if (!block_on(cb)) continue;
            if (!mbar_wait(bar(QB_SF1), c & 1, abort_flag, wcap)) { ok = false; break; }
            tc_fence_after();
            const uint32_t col0 = 32 * half;      // this thread's 32 keys of the block
            uint64_t p2[16];
            {
                uint32_t sv[32];
                tmem_ld32(tm_lane + Cfg::C_S + col0, sv);
                tc_wait_ld();
                const int key0 = 64 * cb + (int)col0;
                const int jlim = off + gi + 1 - key0;                     // keys jfirst <= e < jlim are visible
                const int jfirst = W > 0 ? off + gi + 1 - W - key0 : 0;
                if (jlim < 32 || jfirst > 0) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (e >= jlim || e < jfirst) sv[e] = __float_as_uint(-1e30f);
                }
#pragma unroll
                for (int e2 = 0; e2 < 16; ++e2) p2[e2] = ex2_2(fma2(pku(sv[2 * e2], sv[2 * e2 + 1]), c1c1, nm22));
                if (MODE == 1) {      // S has been read: the next block's S may take its place
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(QB_PRA));
                }
                if (MODE == 0) {      // P over S, ready for kbar += P K while Gamma is still being formed
                    uint32_t pp[32];
#pragma unroll
                    for (int e2 = 0; e2 < 16; ++e2) {
                        const int ks = e2 >> 3, e = e2 & 7;
                        pp[ks * 16 + e] = split2(p2[e2], pp[ks * 16 + 8 + e]);
                    }
                    tmem_st32(tm_lane + Cfg::C_S + col0, pp);
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(QB_PRA));
                }
            }
            if (!mbar_wait(bar(QB_SF2), c & 1, abort_flag, wcap)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int chunk = 0; chunk < 2; ++chunk) {
                const uint32_t colbase = col0 + 16 * chunk;      // 16 keys = one 16-element step of the products
                if (MODE == 1) {
                    // with u = gbar - f (the F tile holds (-t) . k, so u = gk - F with gk = gbar - kbar.t):
                    //   ds = scale p (gamma (1 - e) + u e + F + kk),  kk = kbar.t - kappa
                    uint32_t ev[16], fv[16], gv[16], pd[16];
                    tmem_ld16(tm_lane + Cfg::C_E + colbase, ev);
                    tmem_ld16(tm_lane + Cfg::C_F + colbase, fv);
                    tmem_ld16(tm_lane + Cfg::C_G1 + colbase, gv);
                    tc_wait_ld();
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) {
                        const uint64_t f2 = pku(fv[2 * e2], fv[2 * e2 + 1]), g2 = pku(gv[2 * e2], gv[2 * e2 + 1]);
                        const uint64_t evv = sub2(pku(ev[2 * e2], ev[2 * e2 + 1]), ky2);
                        const uint64_t u = sub2(gk2, f2);
                        const uint64_t inner = fma2(g2, sub2(one2, evv), fma2(u, evv, add2(f2, kk2)));
                        pd[e2] = split2(mul2(mul2(p2[8 * chunk + e2], sc2), inner), pd[8 + e2]);
                    }
                    tmem_st16(tm_lane + Cfg::C_E + colbase, pd);      // over the E columns this thread has just read
                } else {
                    uint32_t gv[16], pg[16];
                    tmem_ld16(tm_lane + Cfg::C_G0 + colbase, gv);
                    tc_wait_ld();
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) {
                        const uint64_t q2 = mul2(p2[8 * chunk + e2], pku(gv[2 * e2], gv[2 * e2 + 1]));
                        gb2 = add2(gb2, q2);
                        pg[e2] = split2(q2, pg[8 + e2]);
                    }
                    tmem_st16(tm_lane + Cfg::C_G0 + colbase, pg);
                }
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(QB_PRB));
            ++c;
        }
        float gb;
        {
            float g0, g1;
            upk2(gb2, g0, g1);
            gb = g0 + g1;
        }
        if (MODE == 0) {      // gbar: the two halves of a row meet (all compute threads take part, aborted or not)
            red[half * 128 + lrow] = gb;
            named_sync_compute();
            gb = red[lrow] + red[128 + lrow];
        }
        if (ok && mbar_wait(bar(QB_ACCFULL), 0, abort_flag, wcap)) {
            tc_fence_after();
            const size_t e0 = row * D + half * (D / 2);
            if (MODE == 0 && okr && half == 0) prm.rowsc_w[row * 8 + 2] = gb;
#pragma unroll 1
            for (int cb = 0; cb < D / 2; cb += 32) {
                uint32_t v[32];
                if (MODE == 1) {
                    tmem_ld32(tm_lane + Cfg::C_DQ + half * (D / 2) + cb, v);
                    tc_wait_ld();
                    if (okr)
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            const float4 t4 = *reinterpret_cast<const float4*>(prm.tvec + e0 + cb + e);
                            *reinterpret_cast<float4*>(prm.dq + e0 + cb + e) =
                                make_float4(__uint_as_float(v[e]) + t4.x, __uint_as_float(v[e + 1]) + t4.y,
                                            __uint_as_float(v[e + 2]) + t4.z, __uint_as_float(v[e + 3]) + t4.w);
                        }
                } else {
                    uint32_t h[32];
                    tmem_ld32(tm_lane + Cfg::C_KB + half * (D / 2) + cb, v);
                    tmem_ld32(tm_lane + Cfg::C_H + half * (D / 2) + cb, h);
                    tc_wait_ld();
                    if (okr)
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            const float k0 = __uint_as_float(v[e]), k1 = __uint_as_float(v[e + 1]), k2 = __uint_as_float(v[e + 2]),
                                        k3 = __uint_as_float(v[e + 3]);
                            *reinterpret_cast<float4*>(prm.kbar + e0 + cb + e) = make_float4(k0, k1, k2, k3);
                            *reinterpret_cast<float4*>(prm.hvec + e0 + cb + e) =
                                make_float4(__uint_as_float(h[e]) - gb * k0, __uint_as_float(h[e + 1]) - gb * k1,
                                            __uint_as_float(h[e + 2]) - gb * k2, __uint_as_float(h[e + 3]) - gb * k3);
                        }
                }
            }
        }
    }
    // ================================ common exit ================================
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(BT_TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag && prm.status) atomicAdd(prm.status + LLA_STATUS_TIMEOUT, 1);
}

template <int D>
int launch_t(const BwdTensorArgs& a, int which) {
    const int BH = a.B * a.H, kvg = a.kv_group > 0 ? a.kv_group : 1, KVU = BH / kvg;
    BtParams p = {};
    p.n = a.n; p.nq = a.nq; p.first = a.first; p.H = a.H; p.kv_group = kvg; p.window = a.window;
    p.head_rows = a.head_rows; p.block_mask = a.block_mask; p.block_mask_stride = a.block_mask_stride; p.has_glo = a.gl != nullptr; p.scale = a.scale;
    p.stats = a.stats; p.pairsc = a.pairsc; p.npair = (a.nq + 1) / 2; p.yvec = a.yvec; p.tvec = a.tvec; p.rowsc_w = a.rowsc;
    p.kbar = a.kbar; p.hvec = a.hvec; p.dq = a.dq; p.dk = a.dk; p.dv = a.dv; p.status = a.status;
    p.wait_clocks = a.wait_clocks > 0 ? a.wait_clocks : kWaitClocks;
    p.no_loads = a.no_loads;
    const void* gl = a.gl ? a.gl : a.gh;        // a valid map either way; never loaded without a lo half
    if (which == 2) {
        using Cfg = KtCfg<D>;
        CUtensorMap mK, mV, mQ, mYh, mYl, mTh, mTl, mGh, mGl, mRS;
        bool ok = make_map_bf16(&mK, a.k, KVU, a.n, D, 128) && make_map_bf16(&mV, a.v, KVU, a.n, D, 128) &&
                  make_map_bf16(&mQ, a.q, BH, a.nq, D, 64) && make_map_bf16(&mYh, a.yh, BH, a.nq, D, 64) &&
                  make_map_bf16(&mYl, a.yl, BH, a.nq, D, 64) && make_map_bf16(&mTh, a.tnh, BH, a.nq, D, 64) &&
                  make_map_bf16(&mTl, a.tnl, BH, a.nq, D, 64) && make_map_bf16(&mGh, a.gh, BH, a.nq, D, 64) &&
                  make_map_bf16(&mGl, gl, BH, a.nq, D, 64) && make_map_f32_rows(&mRS, a.pairsc, BH, (a.nq + 1) / 2, 8, 32);
        if (!ok) return LLA_ERR_CUDA;
        LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_ktile_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SM_ALLOC));
        const dim3 grid(BH, (a.n + 127) / 128);
        bwd_ktile_tc_kernel<D><<<grid, BT_THREADS, Cfg::SM_ALLOC, a.stream>>>(mK, mV, mQ, mYh, mYl, mTh, mTl, mGh, mGl, mRS, p);
        LLA_CUDA_TRY(cudaGetLastError());
        return LLA_OK;
    }
    using Cfg = QtCfg<D>;
    CUtensorMap mQ, mGh, mGl, mTh, mTl, mK, mV;
    const void* th = which == 1 ? a.tnh : a.q;      // the moments kernel loads no T tiles
    const void* tl = which == 1 ? a.tnl : a.q;
    bool ok = make_map_bf16(&mQ, a.q, BH, a.nq, D, 128) && make_map_bf16(&mGh, a.gh, BH, a.nq, D, 128) &&
              make_map_bf16(&mGl, gl, BH, a.nq, D, 128) && make_map_bf16(&mTh, th, BH, a.nq, D, 128) &&
              make_map_bf16(&mTl, tl, BH, a.nq, D, 128) && make_map_bf16(&mK, a.k, KVU, a.n, D, 64) &&
              make_map_bf16(&mV, a.v, KVU, a.n, D, 64);
    if (!ok) return LLA_ERR_CUDA;
    const dim3 grid(BH, (a.nq + 127) / 128);
    if (which == 0) {
        LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_qtile_tc_kernel<D, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SM_ALLOC));
        bwd_qtile_tc_kernel<D, 0><<<grid, BT_THREADS, Cfg::SM_ALLOC, a.stream>>>(mQ, mGh, mGl, mTh, mTl, mK, mV, p);
    } else {
        LLA_CUDA_TRY(cudaFuncSetAttribute(bwd_qtile_tc_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SM_ALLOC));
        bwd_qtile_tc_kernel<D, 1><<<grid, BT_THREADS, Cfg::SM_ALLOC, a.stream>>>(mQ, mGh, mGl, mTh, mTl, mK, mV, p);
    }
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

}  // namespace

int launch_backward_tensor(const BwdTensorArgs& a, int which) {
    if (a.d == 64) return launch_t<64>(a, which);
    if (a.d == 128) return launch_t<128>(a, which);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
