// LLA forward on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 inputs, d = dv = 64 or 128.
//
// One thread block per (batch*head, 128-row query tile).  The three loops of Algorithm 1 and the
// per-iteration loop of Algorithm 2 are all "sweeps" over 64-key blocks with the same skeleton:
//
//   TMA            K block (and V block in the last sweep) -> 128B-swizzled shared memory
//   MMA 1 (SS)     S = Q K^T                     [128 x 64] fp32 in TMEM
//                  A = P_hi K^T + P_lo K^T       [128 x 64] fp32 in TMEM   (CG and output sweeps)
//   CUDA cores     one thread pair per query row reads S, A from TMEM, forms
//                      max sweep     running row maximum m_i
//                      stats sweep   w = exp(s - m),                 omega += w
//                      CG sweep      u = w (a - kbar.p)              (Algorithm 2's W .* (P K^T))
//                      output sweep  c = w (1 - (a - kbar.y)),       den += c
//                  splits the result into bf16 hi + lo and stores both back into the TMEM columns S
//                  came from (two 16-bit values per column)
//   MMA 2 (TS)     ACC += U_hi B + U_lo B, A operand straight from TMEM, B = the same K block read
//                  MN-major (or the V block in the output sweep)
//
// S/A/U cycle through three TMEM buffers (3 x 128 columns) and ACC takes D more (all 512 columns for
// D = 128); K/V blocks go through a 4-stage ring (3 stages for D = 128).  Operands wider than 64 columns
// are held as 64-column sub-tiles so every tile keeps the 128-byte swizzled row.  For D = 128 the fp32
// row vectors x, kbar and r do not fit in shared memory or registers next to the operand tiles; each
// thread keeps its own entries in a global scratch slot owned by the SM (L2-resident, thread-private).  Roles: warps 0-7 compute (warp w owns TMEM lanes 32*(w%4).. and key half w/4 of each
// block; two threads share a row and exchange partial sums through shared memory), warp 8 issues TMA,
// warps 9 and 10 issue the two MMA streams.  Every on-the-fly MMA operand (P, y, U) is carried as a bf16 pair hi + lo so
// the products keep ~16 mantissa bits: a single bf16 rounding of those operands would leave a
// 2e-3..5e-3 error in the output, above the 2e-3 gate.  Q, K, V are exact bf16 inputs.
//
// The mathematics is the centred form described in lla_forward_simt.cu (same CG, same freeze rule).
// All waits on mbarriers are bounded; a wait that expires sets LLA_STATUS_TIMEOUT and the block
// leaves through the common exit (TMEM is released there).
#include <cuda_fp16.h>

#include <algorithm>
#include <type_traits>
#include <mutex>

#include "lla_sm100.cuh"

namespace lla {
namespace {

using namespace sm100;

constexpr int TC_BR = 128;           // query rows per block (TMEM lanes)
constexpr int TC_BC = 64;            // keys per block
constexpr int TC_COMPUTE = 256;      // compute threads (warps 0..7)
constexpr int TC_THREADS = 352;      // + TMA warp + two MMA warps (d = 128: 384, with an idle warp that completes the third warpgroup)
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_NBUF = 3;           // S/A/U buffers in TMEM (128 columns each)
constexpr int TC_ACC_COL = TC_NBUF * 128;   // ACC columns [384, 384 + D)
constexpr int TC_R_COL = 0;                 // preconditioner product, between sweeps: R (fp16) in buffer 0's columns,
constexpr int TC_Z_COL = 128;               // Z = R M (fp32, D columns) from buffer 1's columns on
constexpr int TC_NST_MAX = 4;
constexpr int TC_ORDER_MAX = 256;    // launch-order table size (query tiles)
constexpr int TC_BLIST_MAX = 1024;   // key blocks a block-sparse tile can list (n <= 65536)
constexpr int TC_SPLIT_MAX = 4;      // sweeps of at most this many key blocks run in split mode (see the compute role)

// SW_CG16: a CG sweep whose on-the-fly operands (P, U) are single fp16 values instead of bf16 hi + lo pairs
enum SweepKind : int { SW_STATS = 1, SW_CG = 2, SW_OUT = 3, SW_DONE = 4, SW_CG16 = 5 };

// Shared-memory carve-up (bytes, from a 1024-byte aligned base), per head size D (64 or 128).
// Operand tiles are stored as D/64 sub-tiles of 64 columns (128-byte rows, 128B swizzle) one after
// the other.  For D = 64 the row vectors x and kbar live in shared memory as fp32 [D][128]; for
// D = 128 there is no room for them, so x, kbar and r live in an L2-resident global scratch slot
// owned by the SM (one block per SM at a time) and the ring has three stages.
template <int D>
struct TcCfg {
    static constexpr int KSUB = D / 64;                         // 64-column sub-tiles per operand row
    static constexpr int NCOL = D / 2;                          // row-vector columns per thread
    static constexpr int NST = D == 64 ? 4 : 3;                 // K/V ring stages
    static constexpr int QSUB_BYTES = TC_BR * 128;              // one sub-tile of a 128-row operand
    static constexpr int KSUB_BYTES = TC_BC * 128;              // one sub-tile of a 64-key block
    static constexpr int OPER_BYTES = KSUB * QSUB_BYTES;        // Q, P_hi, P_lo
    static constexpr int KBLK_BYTES = KSUB * KSUB_BYTES;        // K block (V block follows it)
    static constexpr int STAGE_BYTES = 2 * KBLK_BYTES;
    static constexpr bool STATE_IN_SMEM = D == 64;
    static constexpr int SM_Q = 0;
    static constexpr int SM_PHI = SM_Q + OPER_BYTES;
    static constexpr int SM_PLO = SM_PHI + OPER_BYTES;
    static constexpr int SM_KV = SM_PLO + OPER_BYTES;
    static constexpr int SM_X = SM_KV + NST * STAGE_BYTES;                        // fp32 [D][128] (D = 64 only)
    static constexpr int SM_KBAR = SM_X + (STATE_IN_SMEM ? D * TC_BR * 4 : 0);
    static constexpr int SM_RED = SM_KBAR + (STATE_IN_SMEM ? D * TC_BR * 4 : 0);  // pair reductions: 2 buffers x 4 values x 2 x 128 floats
    static constexpr int SM_FLAGS = SM_RED + 8192;                                // 2 x 8 ints
    static constexpr int SM_BAR = SM_FLAGS + 64;                                  // mbarriers
    static constexpr int SM_MISC = SM_BAR + 256;                                  // tmem base, ctl kind, abort
    static constexpr int SM_BLIST = SM_MISC + 64;                                 // block-sparse: the tile's key blocks (uint16)
    static constexpr int SM_TOTAL = SM_BLIST + 2 * TC_BLIST_MAX;
    static constexpr int SM_ALLOC = SM_TOTAL + 1024;                              // slack for 1024-byte alignment
    static constexpr uint32_t IDESC_TS = sm100::make_idesc(TC_BR, D, 0, 1);   // ACC: A from TMEM, B MN-major, N = D
    static constexpr uint32_t IDESC_TS16 = sm100::make_idesc(TC_BR, D, 0, 1, /*f16=*/1);   // same, both operands fp16
    static constexpr size_t SCRATCH_FLOATS_PER_SM = STATE_IN_SMEM ? 0 : 3 * (size_t)D * TC_BR;   // x, kbar, r
};
static_assert(TcCfg<64>::SM_ALLOC <= 227 * 1024 && TcCfg<128>::SM_ALLOC <= 227 * 1024, "shared memory budget");

// mbarrier indices
enum { B_QFULL = 0, B_KVFULL = 1, B_KVEMPTY = B_KVFULL + TC_NST_MAX, B_VFULL = B_KVEMPTY + TC_NST_MAX,
       B_SAFULL = B_VFULL + TC_NST_MAX,
       B_UFULL = B_SAFULL + TC_NBUF, B_BUFFREE = B_UFULL + TC_NBUF, B_ACCFULL = B_BUFFREE + TC_NBUF, B_CTL = B_ACCFULL + 1,
       B_EXIT = B_CTL + 1,   // two: the MMA warps' last commits on an aborted run
       B_MFULL = B_EXIT + 2, // the preconditioner matrix has landed
       B_COUNT = B_MFULL + 1 };
static_assert(B_COUNT * 8 <= 256, "barrier area too small");

constexpr uint32_t IDESC_SS = make_idesc(TC_BR, TC_BC, 0, 0);   // S/A: A, B K-major; ACC uses make_idesc(128, D, 0, 1)
constexpr uint32_t IDESC_SS16 = make_idesc(TC_BR, TC_BC, 0, 0, /*f16=*/1);   // the same products with both operands fp16

struct TcParams {
    int n, nq, causal, head_rows, max_iters, first_tile;   // n keys; nq query rows at positions n - nq .. n - 1
    int precise_iters;   // CG iterations whose operands are bf16 hi + lo pairs; later ones use single fp16 operands
    int precise_iters_early;   // the same for the row tiles that end within the first 8 D positions
    long long wait_clocks;   // cap of every bounded wait, in SM clocks
    int no_loads;        // test aid: the TMA warp issues no copy at all, so that every wait expires with nothing in flight
    const int* f16_ok;   // device word written by the conversion pre-pass: nonzero = q and k fit the fp16 range and
                         // the fp16 copy of k (tmK16) is valid; NULL or zero = every sweep in bf16
    float scale, lambda, tol;
    float* rho;
    float* stats;
    int H, kv_group;     // query heads per (batch), query heads per key/value head
    Strides so;          // layout of out [B, H, nq, D]
    int window;          // causal sliding window (0: none): a row sees its last `window` positions
    const float* rhs;    // solve mode: right-hand sides h_i [B, H, nq, D]; the CG then solves C_i x = h_i ...
    float* sol;          // ... and x_i is written here instead of running the output sweep
    const float* kbar_in;    // solve mode, optional: kbar_i [B, H, nq, D] and the forward's saved stats [B, H, nq, 3] (the
    const float* stats_in;   // shift and omega): given both, the statistics sweep that would recompute them is skipped
    int* iters;
    int* status;
    float* scratch;      // D = 128: per-SM slots for x, kbar, r (TcCfg::SCRATCH_FLOATS_PER_SM each)
    int scratch_slots;
    const float* lambda_rows;   // optional per-row ridge [B, H, n]
    const unsigned char* block_mask;   // optional [query tiles][key blocks] (+ bh * block_mask_stride): nonzero = attended
    long long block_mask_stride;
    int ridge_mode;
    int use_order;       // 1: blockIdx.y -> tile through order[]; 0: last tile first
    unsigned short order[TC_ORDER_MAX];
};

// PC: preconditioned CG compiled in (an instance of its own, so that the plain path carries none of its code).
// GIVEN: solve mode with kbar and the saved row statistics supplied (fp32 output type only), likewise an instance
// of its own: the statistics sweep is compiled out.
template <int D, typename TOut, bool PC, bool GIVEN = false>
__global__ void __launch_bounds__(D == 128 ? 384 : TC_THREADS, 1)
forward_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmK16,
                  const __grid_constant__ CUtensorMap tmM, TOut* __restrict__ out, const TcParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    using Cfg = TcCfg<D>;
    constexpr int TC_NST = Cfg::NST, NCOL = Cfg::NCOL, KSUB = Cfg::KSUB;
    constexpr int SM_Q = Cfg::SM_Q, SM_PHI = Cfg::SM_PHI, SM_PLO = Cfg::SM_PLO, SM_KV = Cfg::SM_KV;
    constexpr int SM_RED = Cfg::SM_RED, SM_FLAGS = Cfg::SM_FLAGS, SM_BAR = Cfg::SM_BAR, SM_MISC = Cfg::SM_MISC;
    constexpr int STAGE = Cfg::STAGE_BYTES, KBLK = Cfg::KBLK_BYTES;
    constexpr uint32_t IDESC_TS = Cfg::IDESC_TS, IDESC_TS16 = Cfg::IDESC_TS16;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + SM_BAR;
    auto bar = [&](int i) { return bars + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + SM_MISC);   // [0] tmem base, [2] abort, [3] kv unit, [4..5] kind
    volatile int* abort_flag = misc + 2;
    // row-vector state: shared memory (D = 64) or this SM's slot of the global scratch (D = 128)
    float* xs;
    float* kbs;
    float* rs = nullptr;
    if constexpr (Cfg::STATE_IN_SMEM) {
        xs = reinterpret_cast<float*>(smem + Cfg::SM_X);
        kbs = reinterpret_cast<float*>(smem + Cfg::SM_KBAR);
    } else {
        uint32_t smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        if (smid >= (uint32_t)prm.scratch_slots) {     // never expected: SM ids are dense on this part
            if (threadIdx.x == 0 && prm.status) atomicAdd(prm.status + LLA_STATUS_TIMEOUT, 1);
            return;
        }
        xs = prm.scratch + (size_t)smid * Cfg::SCRATCH_FLOATS_PER_SM;
        kbs = xs + (size_t)D * TC_BR;
        rs = kbs + (size_t)D * TC_BR;
    }
    float* red = reinterpret_cast<float*>(smem + SM_RED);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // blockIdx.x runs fastest in launch order: all heads of one query tile start together, the tiles
    // in order of decreasing estimated cost (see tile_order on the host side)
    const int bh = blockIdx.x;
    const int tile = prm.first_tile + (prm.use_order ? (int)prm.order[blockIdx.y] : (int)(gridDim.y - 1 - blockIdx.y));
    const int r0 = tile * TC_BR;
    const int n = prm.n, nq = prm.nq, off = n - nq;     // query row r sits at position off + r
    const int nblk_all = (n + TC_BC - 1) / TC_BC;
    const int cend = prm.causal ? min(nblk_all, (off + r0 + TC_BR + TC_BC - 1) / TC_BC) : nblk_all;
    // sliding window: the tile's sweeps start at the block that holds its first row's first visible key
    const int cbeg = (prm.causal && prm.window > 0) ? max(0, off + r0 + 1 - prm.window) / TC_BC : 0;
    // Block sparsity: the sweeps visit only the key blocks that the caller's mask lists for this query tile, plus
    // the ones that are always attended -- the blocks of the first head_rows keys (so that every row keeps enough
    // keys for its system to be well posed and the directly-solved rows are untouched) and the tile's diagonal blocks.
    unsigned short* blist = reinterpret_cast<unsigned short*>(smem + Cfg::SM_BLIST);
    if (prm.block_mask) {
        if (warp == 0) {
            const unsigned char* mrow = prm.block_mask + (size_t)bh * prm.block_mask_stride + (size_t)tile * nblk_all;
            int cnt = 0;
            for (int c0 = cbeg; c0 < cend; c0 += 32) {
                const int c = c0 + lane;
                const bool on = c < cend && (mrow[c] != 0 || c * TC_BC < prm.head_rows || c * TC_BC + TC_BC - 1 >= off + r0);
                const unsigned m = __ballot_sync(0xffffffffu, on);
                if (on) blist[cnt + __popc(m & ((1u << lane) - 1))] = (unsigned short)c;
                cnt += __popc(m);
            }
            if (lane == 0) misc[6] = cnt;
        }
        __syncthreads();
    }
    const int nblk = prm.block_mask ? misc[6] : cend - cbeg;      // key blocks per sweep
    auto kblock = [&](int c) { return prm.block_mask ? (int)blist[c] : cbeg + c; };     // c-th key block of a sweep
    const bool split = nblk <= TC_SPLIT_MAX;
    // Operand format of a sweep over the keys.  The statistics sweep(s) and the first `precise` CG sweeps run on
    // the bf16 inputs; every later sweep (the remaining CG sweeps and, if CG got that far, the output sweep) runs
    // its Q K^T and P K^T products on fp16 copies of Q and K (one kind::f16 MMA takes both operands in the same
    // 16-bit format).  The values of the copies equal the bf16 inputs (the pre-pass checks the range).  Every role
    // counts the CG sweeps it has seen, so all of them know a sweep's format, and the next one's, without being
    // told.  (Tiles whose rows see fewer than 8 D keys converge more slowly and keep the pairs for longer.)
    const int precise = off + r0 + TC_BR <= 8 * D ? prm.precise_iters_early : prm.precise_iters;
    const bool f16_on = prm.f16_ok && *prm.f16_ok && precise < (1 << 29);
    const long long wcap = prm.wait_clocks;

    if (tid == 0) {
        mbar_init(bar(B_QFULL), 1);
        for (int s = 0; s < TC_NST; ++s) {
            mbar_init(bar(B_KVFULL + s), 1);
            mbar_init(bar(B_KVEMPTY + s), 1);
            mbar_init(bar(B_VFULL + s), 1);
        }
        for (int b = 0; b < TC_NBUF; ++b) {
            mbar_init(bar(B_SAFULL + b), 1);
            mbar_init(bar(B_UFULL + b), (split ? TC_COMPUTE : TC_COMPUTE / 2) / 32);   // one arrival per warp
            mbar_init(bar(B_BUFFREE + b), 1);
        }
        mbar_init(bar(B_ACCFULL), 1);
        mbar_init(bar(B_CTL), TC_COMPUTE / 32);
        mbar_init(bar(B_EXIT), 1);
        mbar_init(bar(B_EXIT + 1), 1);
        mbar_init(bar(B_MFULL), 1);
        misc[4] = SW_STATS;
        misc[5] = SW_STATS;
        misc[2] = 0;
        fence_barrier_init();
    }
    if (warp == 8) {   // TMEM allocation by one full warp; the base address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(sbase + SM_MISC), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[0];

    // Register hand-over between the warpgroups: the copy- and MMA-issuing warps need few registers and give theirs
    // up, the compute warps take them (168 a thread at launch, the most that twelve warps can have).
    auto regs_give = [&]() { if constexpr (D == 128) asm volatile("setmaxnreg.dec.sync.aligned.u32 64;" ::: "memory"); };
    auto regs_take = [&]() { if constexpr (D == 128) asm volatile("setmaxnreg.inc.sync.aligned.u32 216;" ::: "memory"); };

    if (warp == 8) {
        regs_give();
        // ================================ TMA producer ================================
        // K blocks stream through the ring continuously: once a sweep's blocks are issued the first
        // blocks of the next sweep are prefetched without waiting to learn what kind of sweep it is
        // (every kind needs K).  V blocks are added, on their own barriers, once the output sweep
        // is announced.
        if (lane == 0 && !prm.no_loads) {
            mbar_expect_tx(bar(B_QFULL), Cfg::OPER_BYTES);
            // tensor-map coordinates: (column, row, head, batch); keys and values by their own head
            const int bb = bh / prm.H, hq = bh % prm.H, hk = hq / prm.kv_group;
            for (int sub = 0; sub < KSUB; ++sub)
                tma_load_4d(sbase + SM_Q + sub * Cfg::QSUB_BYTES, &tmQ, bar(B_QFULL), 64 * sub, r0, hq, bb);
            if (PC) {
                // the preconditioner of this tile's key range: D x D fp16, laid out like D / 64 key blocks, into the
                // V halves of the first ring stages (idle until the output sweep, when it is no longer needed)
                const int gm = precond_block_used((prm.causal ? min(n - 1, off + r0 + TC_BR - 1) : n - 1) / 128);
                mbar_expect_tx(bar(B_MFULL), D * D * 2);
                for (int rb = 0; rb < D / 64; ++rb)
                    for (int sub = 0; sub < KSUB; ++sub)
                        tma_load_4d(sbase + SM_KV + rb * STAGE + KBLK + sub * Cfg::KSUB_BYTES, &tmM, bar(B_MFULL), 64 * sub,
                                    gm * D + 64 * rb, hk, bb);
            }
            uint32_t kit = 0;      // K blocks issued so far
            int pre = 0;           // blocks of the coming sweep already issued
            bool ok = true;
            auto issue_k = [&](int c, bool f16) {
                const uint32_t s = kit % TC_NST;
                if (!mbar_wait(bar(B_KVEMPTY + s), ((kit / TC_NST) & 1) ^ 1, abort_flag, wcap)) { ok = false; return; }
                mbar_expect_tx(bar(B_KVFULL + s), KBLK);
                for (int sub = 0; sub < KSUB; ++sub)
                    tma_load_4d(sbase + SM_KV + s * STAGE + sub * Cfg::KSUB_BYTES, f16 ? &tmK16 : &tmK, bar(B_KVFULL + s), 64 * sub,
                                kblock(c) * TC_BC, hk, bb);
                ++kit;
            };
            uint32_t v_g0 = 0;
            int v_issued = 0;      // V blocks issued (output sweep only), the first at ring position v_g0
            auto issue_v = [&](int c, uint32_t g) {
                if (v_issued == 0) v_g0 = g - c;
                v_issued = c + 1;
                const uint32_t s = g % TC_NST;
                mbar_expect_tx(bar(B_VFULL + s), KBLK);
                for (int sub = 0; sub < KSUB; ++sub)
                    tma_load_4d(sbase + SM_KV + s * STAGE + KBLK + sub * Cfg::KSUB_BYTES, &tmV, bar(B_VFULL + s), 64 * sub, kblock(c) * TC_BC, hk, bb);
            };
            int cg_seen = 0;       // CG sweeps issued so far
            for (uint32_t ctl = 0; ok; ++ctl) {
                if (!mbar_wait(bar(B_CTL), ctl & 1, abort_flag, wcap)) break;
                const int kind = misc[4 + (ctl & 1)];
                if (kind == SW_DONE) {
                    // prefetched blocks nobody will consume: wait until they have landed
                    for (int i = 0; i < pre; ++i) {
                        const uint32_t g = kit - pre + i;
                        if (!mbar_wait(bar(B_KVFULL + g % TC_NST), (g / TC_NST) & 1, abort_flag, wcap)) break;
                    }
                    break;
                }
                const uint32_t g0 = kit - pre;
                if (kind == SW_OUT)
                    for (int c = 0; c < pre; ++c) issue_v(c, g0 + c);
                const bool f16_cur = kind == SW_CG16 || (kind == SW_OUT && f16_on && cg_seen >= precise);
                for (int c = pre; c < nblk && ok; ++c) {
                    issue_k(c, f16_cur);
                    if (ok && kind == SW_OUT) issue_v(c, g0 + c);
                }
                pre = 0;
                if (kind == SW_CG || kind == SW_CG16) ++cg_seen;
                // first blocks of the next sweep, in the format it will have.  After a statistics sweep the next one
                // is another statistics sweep, the first CG sweep or the output sweep: all on the bf16 inputs unless
                // precise == 0, where nothing is fetched ahead
                const bool f16_next = f16_on && cg_seen >= precise;
                if (kind != SW_OUT && !(kind == SW_STATS && f16_next))
                    for (int c = 0; c < min(TC_NST, nblk) && ok; ++c) { issue_k(c, f16_next); ++pre; }
            }
            if (*abort_flag) {
                if (PC) (void)mbar_wait_landed(bar(B_MFULL), 0, wcap);
                // an aborted block: the copies issued above write into this block's shared memory, so they must
                // have landed before the block exits (on a completed run their consumers have waited for them)
                (void)mbar_wait_landed(bar(B_QFULL), 0, wcap);
                for (uint32_t g = kit > (uint32_t)TC_NST ? kit - TC_NST : 0; g < kit; ++g)
                    (void)mbar_wait_landed(bar(B_KVFULL + g % TC_NST), (g / TC_NST) & 1, wcap);
                for (int c = max(0, v_issued - TC_NST); c < v_issued; ++c)
                    (void)mbar_wait_landed(bar(B_VFULL + (v_g0 + c) % TC_NST), (c / TC_NST) & 1, wcap);
            }
        }
    } else if (warp == 9) {
        regs_give();
        // ================================ MMA issuer 1: S = Q K^T, A = P K^T ================================
        // All 32 lanes run the loop convergently; the MMAs and commits are predicated on one lane.
        // tcgen05.mma issue is throttled to the execution rate, so the time an issuing warp spends
        // in barrier waits is tensor-pipe idle time: two warps (this one and warp 10) feed the pipe
        // and each one's waits hide behind the other's instructions.
        const uint32_t el = elect_one();
        // broadcast through a shuffle so the compiler treats these as warp-uniform values and keeps
        // the MMA operands in uniform registers (otherwise every operand is moved there one by one)
        const uint32_t sb_u = __shfl_sync(0xffffffffu, sbase, 0);
        const uint32_t tm_u = __shfl_sync(0xffffffffu, tmem, 0);
        bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, wcap);
        const uint64_t qdesc = make_desc(sb_u + SM_Q);
        const uint64_t phdesc = make_desc(sb_u + SM_PHI);
        const uint64_t pldesc = make_desc(sb_u + SM_PLO);
        uint32_t it = 0;   // global block counter (stage = it % NST, buffer = it % NBUF)
        int cg_seen = 0;   // CG sweeps issued so far
        for (uint32_t ctl = 0; ok; ++ctl) {
            if (!mbar_wait(bar(B_CTL), ctl & 1, abort_flag, wcap)) break;
            const int kind = misc[4 + (ctl & 1)];
            if (kind == SW_DONE) break;
            tc_fence_after();
            const uint32_t idesc = (kind == SW_CG16 || (kind == SW_OUT && f16_on && cg_seen >= precise)) ? IDESC_SS16 : IDESC_SS;
            if (kind == SW_CG || kind == SW_CG16) ++cg_seen;
            for (int c = 0; c < nblk && ok; ++c, ++it) {
                const uint32_t s = it % TC_NST, b = it % TC_NBUF, bu = it / TC_NBUF;
                if (!mbar_wait(bar(B_KVFULL + s), (it / TC_NST) & 1, abort_flag, wcap)) { ok = false; break; }
                if (!mbar_wait(bar(B_BUFFREE + b), (bu & 1) ^ 1, abort_flag, wcap)) { ok = false; break; }
                tc_fence_after();
                const uint64_t kdesc = make_desc(sb_u + SM_KV + s * STAGE);
                const uint32_t s_tm = tm_u + b * 128, a_tm = s_tm + 64;
                // contraction over D: one group of four 16-wide steps per 64-column sub-tile
                // (sub-tiles are QSUB_BYTES / KSUB_BYTES apart: 1024 / 512 descriptor units)
#pragma unroll
                for (int sub = 0; sub < KSUB; ++sub)
                    mma_ss_k64(el, s_tm, qdesc + sub * (Cfg::QSUB_BYTES >> 4), kdesc + sub * (Cfg::KSUB_BYTES >> 4), idesc, sub > 0);
                if (kind == SW_CG || kind == SW_OUT || kind == SW_CG16) {
#pragma unroll
                    for (int sub = 0; sub < KSUB; ++sub)
                        mma_ss_k64(el, a_tm, phdesc + sub * (Cfg::QSUB_BYTES >> 4), kdesc + sub * (Cfg::KSUB_BYTES >> 4), idesc, sub > 0);
                    if (kind != SW_CG16) {     // second half of the operand pair
#pragma unroll
                        for (int sub = 0; sub < KSUB; ++sub)
                            mma_ss_k64(el, a_tm, pldesc + sub * (Cfg::QSUB_BYTES >> 4), kdesc + sub * (Cfg::KSUB_BYTES >> 4), idesc, 1);
                    }
                }
                tc_commit_el(el, bar(B_SAFULL + b));
            }
        }
        if (*abort_flag) {      // an aborted block: the MMAs this warp issued must be done before TMEM and shared memory go
            tc_commit_el(el, bar(B_EXIT + 0));
            (void)mbar_wait_landed(bar(B_EXIT + 0), 0, wcap);
        }
    } else if (warp == 10) {
        regs_give();
        // ================================ MMA issuer 2: ACC += U B ================================
        const uint32_t el = elect_one();
        const uint32_t sb_u = __shfl_sync(0xffffffffu, sbase, 0);
        const uint32_t tm_u = __shfl_sync(0xffffffffu, tmem, 0);
        bool ok = true;
        uint32_t it = 0;
        for (uint32_t ctl = 0; ok; ++ctl) {
            if (!mbar_wait(bar(B_CTL), ctl & 1, abort_flag, wcap)) break;
            const int kind = misc[4 + (ctl & 1)];
            if (kind == SW_DONE) break;
            for (int c = 0; c < nblk && ok; ++c, ++it) {
                const uint32_t s = it % TC_NST, b = it % TC_NBUF, bu = it / TC_NBUF;
                if (!mbar_wait(bar(B_UFULL + b), bu & 1, abort_flag, wcap)) { ok = false; break; }
                if (kind == SW_OUT && !mbar_wait(bar(B_VFULL + s), (c / TC_NST) & 1, abort_flag, wcap)) { ok = false; break; }
                tc_fence_after();
                const uint32_t bsm = sb_u + SM_KV + s * STAGE + (kind == SW_OUT ? KBLK : 0);
                // B = the K (or V) block read MN-major, N = D: 64-wide column groups are one sub-tile apart
                if (kind == SW_CG16) mma_ts_k64(el, tm_u + TC_ACC_COL, tm_u + b * 128, make_desc(bsm, Cfg::KSUB_BYTES), IDESC_TS16, c > 0);
                else mma_ts_hilo_k64(el, tm_u + TC_ACC_COL, tm_u + b * 128, make_desc(bsm, Cfg::KSUB_BYTES), IDESC_TS, c > 0);
                tc_commit_el(el, bar(B_KVEMPTY + s));
                tc_commit_el(el, bar(B_BUFFREE + b));
                if (c == nblk - 1) tc_commit_el(el, bar(B_ACCFULL));
            }
        }
        if (*abort_flag) {      // an aborted block: the MMAs this warp issued must be done before TMEM and shared memory go
            tc_commit_el(el, bar(B_EXIT + 1));
            (void)mbar_wait_landed(bar(B_EXIT + 1), 0, wcap);
        }
    } else if (warp == 11) {
        regs_give();
    } else {
        regs_take();
        // ================================ compute warps ================================
        const int quad = warp & 3, half = warp >> 2;
        const int lrow = quad * 32 + lane;                 // row inside the tile == TMEM lane
        const int row = r0 + lrow;
        const int L = prm.causal ? off + row + 1 : n;
        const int jlo = (prm.causal && prm.window > 0) ? max(0, L - prm.window) : 0;     // first visible key
        const bool row_ok = row < nq && L >= prm.head_rows;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const int c0 = half * NCOL;                        // first row-vector column owned by this thread
        // byte offset of this thread's chunk ch (8 columns) of row lrow inside a swizzled operand
        auto oper_off = [&](int ch) {
            const int col8 = half * (NCOL / 8) + ch;      // 8-column chunk index within the row
            return (uint32_t)((col8 >> 3) * Cfg::QSUB_BYTES) + swz(lrow, col8 & 7);
        };
        // The two threads of a row sit in warps w and w+4; only those two warps need to meet, so
        // each lane quadrant has its own 64-thread named barrier (ids 2..5).
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(2 + quad) : "memory"); };
        int red_sel = 0;
        auto pair_sum = [&](float v) {
            float* buf = red + red_sel * 1024;
            red_sel ^= 1;
            buf[half * 128 + lrow] = v;
            pair_sync();
            return buf[lrow] + buf[128 + lrow];
        };
        // two sums for one barrier
        auto pair_sum2 = [&](float& a, float& b) {
            float* buf = red + red_sel * 1024;
            red_sel ^= 1;
            buf[half * 128 + lrow] = a;
            buf[256 + half * 128 + lrow] = b;
            pair_sync();
            a = buf[lrow] + buf[128 + lrow];
            b = buf[256 + lrow] + buf[384 + lrow];
        };
        // four sums for one barrier
        auto pair_sum4 = [&](float& a, float& b, float& c, float& d4) {
            float* buf = red + red_sel * 1024;
            red_sel ^= 1;
            buf[half * 128 + lrow] = a;
            buf[256 + half * 128 + lrow] = b;
            buf[512 + half * 128 + lrow] = c;
            buf[768 + half * 128 + lrow] = d4;
            pair_sync();
            a = buf[lrow] + buf[128 + lrow];
            b = buf[256 + lrow] + buf[384 + lrow];
            c = buf[512 + lrow] + buf[640 + lrow];
            d4 = buf[768 + lrow] + buf[896 + lrow];
        };
        auto pair_max = [&](float v) {
            float* buf = red + red_sel * 1024;
            red_sel ^= 1;
            buf[half * 128 + lrow] = v;
            pair_sync();
            return fmaxf(buf[lrow], buf[128 + lrow]);
        };
        // OR over the 256 compute threads
        auto group_any = [&](bool v) { return bar_or(1, TC_COMPUTE, v); };
        // After the waits of a sweep every compute thread learns whether any of them gave up, so that all of them
        // take the same path from there on: a thread whose waits all succeeded must not go on to a pair
        // exchange with a partner that has left.
        auto all_ok = [&](bool mine) { return !bar_or(1, TC_COMPUTE, !mine); };
        // store this thread's NCOL fp32 values of the row as bf16 hi/lo into the swizzled operand tiles
        auto write_operand = [&](const float* vec) {
#pragma unroll
            for (int ch = 0; ch < NCOL / 8; ++ch) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    hi[e] = split_bf16x2(vec[ch * 8 + 2 * e], vec[ch * 8 + 2 * e + 1], lo[e]);
                }
                const uint32_t off = oper_off(ch);
                *reinterpret_cast<uint4*>(smem + SM_PHI + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(smem + SM_PLO + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        };

        // the same vector as an fp16 hi + lo pair (the output sweep's y once the sweeps run on fp16 operands)
        auto write_operand16_pair = [&](const float* vec) {
#pragma unroll
            for (int ch = 0; ch < NCOL / 8; ++ch) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float a = vec[ch * 8 + 2 * e], b = vec[ch * 8 + 2 * e + 1];
                    const __half2 h2 = __floats2half2_rn(a, b);
                    const float2 f = __half22float2(h2);
                    const __half2 l2 = __floats2half2_rn(a - f.x, b - f.y);
                    hi[e] = *reinterpret_cast<const uint32_t*>(&h2);
                    lo[e] = *reinterpret_cast<const uint32_t*>(&l2);
                }
                const uint32_t off = oper_off(ch);
                *reinterpret_cast<uint4*>(smem + SM_PHI + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(smem + SM_PLO + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
        };
        // Q tile: bf16 as loaded, or fp16 once the sweeps have switched format (converted in place by
        // convert_q, each thread its own chunks, between two sweeps when no MMA reads the tile)
        bool q_is_f16 = false;
        auto q_elem = [&](const uint32_t* qw, int e) -> float {
            if (q_is_f16) {
                const __half2 h2 = *reinterpret_cast<const __half2*>(&qw[e >> 1]);
                return (e & 1) ? __high2float(h2) : __low2float(h2);
            }
            return (e & 1) ? __uint_as_float(qw[e >> 1] & 0xFFFF0000u) : __uint_as_float(qw[e >> 1] << 16);
        };
        auto convert_q = [&]() {
#pragma unroll
            for (int ch = 0; ch < NCOL / 8; ++ch) {
                uint4* qp = reinterpret_cast<uint4*>(smem + SM_Q + oper_off(ch));
                const uint4 qraw = *qp;
                const uint32_t qw[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
                uint32_t h[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    h[e] = pack_f16(__uint_as_float(qw[e] << 16), __uint_as_float(qw[e] & 0xFFFF0000u));
                *qp = make_uint4(h[0], h[1], h[2], h[3]);
            }
            q_is_f16 = true;
        };
        // the same vector as one fp16 value per entry, scaled by the power of two sc (see write_p)
        auto write_operand16 = [&](const float* vec, float sc) {
#pragma unroll
            for (int ch = 0; ch < NCOL / 8; ++ch) {
                uint32_t h[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) h[e] = pack_f16(vec[ch * 8 + 2 * e] * sc, vec[ch * 8 + 2 * e + 1] * sc);
                *reinterpret_cast<uint4*>(smem + SM_PHI + oper_off(ch)) = make_uint4(h[0], h[1], h[2], h[3]);
            }
        };

        const float c1 = prm.scale * 1.4426950408889634f;    // scores in log2 units
        float mx2 = -INFINITY, omega = 0.f, inv_omega = 0.f, ridge = 0.f, den = 0.f;
        float abar = 0.f;                                     // kbar.p (CG) or kbar.y (output)
        // fp16 sweeps: the search direction is stored as p * psc with psc a power of two that brings |p| to
        // [1, 2.83), so that its entries and u = w (a - abar) sit in the middle of the fp16 range whatever the
        // scale of the right-hand side; pn2 tracks |p|^2 through the recurrence |p'|^2 = |r'|^2 + beta^2 |p|^2
        float pn2 = 0.f, psc = 1.f, ipsc = 1.f;
        float smax = -INFINITY;                               // statistics sweep: largest score of the row, relative to the shift
        uint32_t blk = 0;                                     // global block counter (buffer = blk & 1)
        bool ok = true;

        // One sweep over the key blocks.  kind is uniform over the block.
        // Long sweeps: warps 0-3 (group 0) take the even blocks, warps 4-7 (group 1) the odd ones,
        // each thread all 64 keys of its row in two passes of 32: the two warps that share a
        // scheduler are then in different phases of the load -> math -> store chain and hide each
        // other's latency.  Short sweeps (split mode, the first query tiles) are latency-bound
        // instead: there both groups work on every block, each thread on its half of the keys, which
        // halves the time from a block's scores to its contribution.
        auto sweep = [&](int kind) {
            float part = 0.f;                                 // omega / den partial
            const uint64_t c1c1 = pk2(c1, c1), nmx = pk2(-mx2, -mx2);
            const float ab_s = kind == SW_CG16 ? abar * psc : abar;
            const uint64_t nab = pk2(-ab_s, -ab_s), oab = pk2(1.f + abar, 1.f + abar), neg1 = pk2(-1.f, -1.f);
            uint64_t part2 = pk2(0.f, 0.f);
            for (int c = 0; c < nblk; ++c, ++blk) {
                if (!split && (int)(blk & 1) != half) continue;
                const uint32_t b = blk % TC_NBUF;
                if (!mbar_wait(bar(B_SAFULL + b), (blk / TC_NBUF) & 1, abort_flag, wcap)) { ok = false; return part; }
                tc_fence_after();
#pragma unroll 1
                for (int h = split ? half : 0; h < (split ? half + 1 : 2); ++h) {
                    const uint32_t s_addr = tmem + lane_addr + b * 128 + 32 * h;
                    uint32_t sv[32], av[32];
                    tmem_ld32(s_addr, sv);
                    if (kind == SW_CG || kind == SW_OUT || kind == SW_CG16) tmem_ld32(s_addr + 64, av);
                    tc_wait_ld();
                    // keys jfirst <= e < jlim of this half block are visible.  Only the diagonal blocks and a
                    // window's first blocks hide any: there the hidden scores are overwritten with a large negative
                    // number, whose weight is exactly zero, so the loops below carry no mask
                    const int jlim = min(L, n) - (kblock(c) * TC_BC + 32 * h);
                    const int jfirst = jlo - (kblock(c) * TC_BC + 32 * h);
                    if (jlim < 32 || jfirst > 0) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (e >= jlim || e < jfirst) sv[e] = __float_as_uint(-1e30f);
                    }
                    if (kind == SW_CG16) {
                        // u = w (a - abar) as one fp16 value per key: 16 keys per k-step in 8 columns
                        uint32_t pk[16];
#pragma unroll
                        for (int e2 = 0; e2 < 16; ++e2) {
                            const uint64_t t2 = fma2(pk2(__uint_as_float(sv[2 * e2]), __uint_as_float(sv[2 * e2 + 1])), c1c1, nmx);
                            float t0, t1;
                            upk2(t2, t0, t1);
                            const uint64_t u2 = mul2(pk2(ex2f(t0), ex2f(t1)),
                                                     add2(pk2(__uint_as_float(av[2 * e2]), __uint_as_float(av[2 * e2 + 1])), nab));
                            float u0, u1;
                            upk2(u2, u0, u1);
                            pk[e2] = pack_f16(u0, u1);
                        }
                        tmem_st16(s_addr, pk);
                    } else {
                        uint32_t pk[32];
#pragma unroll
                        for (int e2 = 0; e2 < 16; ++e2) {
                            const uint64_t t2 = fma2(pk2(__uint_as_float(sv[2 * e2]), __uint_as_float(sv[2 * e2 + 1])), c1c1, nmx);
                            float t0, t1;
                            upk2(t2, t0, t1);
                            if (kind == SW_STATS) smax = fmaxf(smax, fmaxf(t0, t1));     // largest score, relative to the shift
                            uint64_t u2 = pk2(ex2f(t0), ex2f(t1));
                            if (kind == SW_CG)
                                u2 = mul2(u2, add2(pk2(__uint_as_float(av[2 * e2]), __uint_as_float(av[2 * e2 + 1])), nab));
                            if (kind == SW_OUT)
                                u2 = mul2(u2, fma2(pk2(__uint_as_float(av[2 * e2]), __uint_as_float(av[2 * e2 + 1])), neg1, oab));
                            float u0, u1;
                            upk2(u2, u0, u1);
                            if (kind != SW_CG) part2 = add2(part2, u2);
                            // 16 keys per k-step: 8 columns of hi, then 8 columns of lo
                            const int ks = e2 >> 3, e = e2 & 7;
                            pk[ks * 16 + e] = split_bf16x2(u0, u1, pk[ks * 16 + 8 + e]);
                        }
                        tmem_st32(s_addr, pk);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                // one arrival per warp: 32 lanes arriving on one mbarrier are 32 serialised atomics
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_UFULL + b));
            }
            float p0, p1;
            upk2(part2, p0, p1);
            part = p0 + p1;
            return part;
        };
        // read this thread's NCOL ACC columns after the sweep's last MMA
        uint32_t acc_uses = 0;
        // (in two steps, so that the threads can agree on success between the wait and the loads: no array of
        //  accumulator values is live across that barrier)
        auto acc_wait = [&]() {
            if (!mbar_wait(bar(B_ACCFULL), acc_uses & 1, abort_flag, wcap)) { ok = false; return; }
            ++acc_uses;
            tc_fence_after();
        };
        auto acc_load = [&](float* dst) {
#pragma unroll
            for (int cb = 0; cb < NCOL; cb += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + TC_ACC_COL + c0 + cb, v);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) dst[cb + e] = __uint_as_float(v[e]);
            }
            tc_fence_before();
        };
        uint32_t ctl_phase = 0;
        auto start_sweep = [&](int kind, bool f16 = false) {
            if (f16 && !q_is_f16) convert_q();
            if (tid == 0) misc[4 + (ctl_phase & 1)] = kind;
            ++ctl_phase;
            fence_proxy_async();       // operand tiles written with ordinary stores -> visible to the MMA
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_CTL));
        };

        // residual r: registers for D = 64, the scratch slot for D = 128 (no registers to spare)
        float r[Cfg::STATE_IN_SMEM ? NCOL : 1] = {}, p[NCOL];
        auto r_get = [&](int e) -> float {
            if constexpr (Cfg::STATE_IN_SMEM) return r[e];
            else return rs[(c0 + e) * TC_BR + lrow];
        };
        auto r_set = [&](int e, float v) {
            if constexpr (Cfg::STATE_IN_SMEM) r[e] = v;
            else rs[(c0 + e) * TC_BR + lrow] = v;
        };
        float rr = 0.f, stop = 0.f;
        int its = 0;
        bool active = false;
        // P operand for CG iteration t_next: bf16 hi + lo for the first precise_iters iterations, one fp16 after
        // (the products of an iteration enter x and r scaled by |p|, which has fallen by then: the coarser
        // operands of the later iterations cost no accuracy that the early ones have not already spent)
        auto write_p = [&](int t_next) {
            if (f16_on && t_next >= precise) {
                const int e2 = (int)((__float_as_uint(pn2) >> 23) & 0xffu) - 127;      // floor(log2 |p|^2)
                const int k = max(-100, min(100, -(e2 >> 1)));
                psc = __uint_as_float((uint32_t)(127 + k) << 23);
                ipsc = __uint_as_float((uint32_t)(127 - k) << 23);
                write_operand16(p, psc);
            } else {
                write_operand(p);
            }
        };

        // z = M r with the tile's preconditioner: vec holds this thread's NCOL entries of r on entry (|r|^2 is about
        // nrm2 over the whole row) and of z on return.  r goes to TMEM as fp16, scaled by a power of two into the
        // middle of the fp16 range (M is stored with a largest entry of one); once every compute thread has stored
        // its part, warp 0 issues the product Z = R M itself (no hand-over to the MMA warps, which are idle between
        // sweeps, as are the TMEM columns of the S/A/U buffers that R and Z use).
        const uint32_t el0 = PC ? elect_one() : 0u;
        const uint32_t sb_c = PC ? __shfl_sync(0xffffffffu, sbase, 0) : 0u, tm_c = PC ? __shfl_sync(0xffffffffu, tmem, 0) : 0u;
        bool m_ready = false;
        auto precondition = [&](float* vec, float nrm2) {
            const int e2 = (int)((__float_as_uint(nrm2) >> 23) & 0xffu) - 127;
            const int k = max(-100, min(100, -(e2 >> 1)));
            const float sc = __uint_as_float((uint32_t)(127 + k) << 23), isc = __uint_as_float((uint32_t)(127 - k) << 23);
            uint32_t pk[NCOL / 2];
#pragma unroll
            for (int e = 0; e < NCOL / 2; ++e) pk[e] = pack_f16(vec[2 * e] * sc, vec[2 * e + 1] * sc);
            const uint32_t r_addr = tmem + lane_addr + TC_R_COL + half * (NCOL / 2);
            if constexpr (NCOL == 32) tmem_st16(r_addr, pk);
            else tmem_st32(r_addr, pk);
            tc_wait_st();
            tc_fence_before();
            named_sync_compute();
            if (warp == 0) {
                if (!m_ready) m_ready = mbar_wait(bar(B_MFULL), 0, abort_flag, wcap);     // the matrix has landed (first use)
                tc_fence_after();
                if (m_ready) {
#pragma unroll
                    for (int rb = 0; rb < D / 64; ++rb)
                        mma_ts_k64c(el0, tm_c + TC_Z_COL, tm_c + TC_R_COL + 32 * rb,
                                    make_desc(sb_c + SM_KV + rb * STAGE + KBLK, Cfg::KSUB_BYTES), IDESC_TS16, rb > 0);
                    tc_commit_el(el0, bar(B_ACCFULL));
                }
            }
            if (!mbar_wait(bar(B_ACCFULL), acc_uses & 1, abort_flag, wcap)) { ok = false; return; }
            ++acc_uses;
            tc_fence_after();
#pragma unroll
            for (int cb = 0; cb < NCOL; cb += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_addr + TC_Z_COL + c0 + cb, v);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) vec[cb + e] = __uint_as_float(v[e]) * isc;
            }
            tc_fence_before();
        };
        float rz = 0.f;      // r . z of the preconditioned recurrence
        bool prec_row = true;   // false once the preconditioner has failed this row (z = r from then on)

        // ---- statistics sweep: omega and kbar ----
        // No sweep of its own finds the row maxima: Eq. "lla" is unchanged under a joint scaling of the weights and
        // the ridge, so any shift of the scores serves as long as the weights stay in range.  The sweep runs with
        // shift zero and notes the largest score on the way; only if some row's maximum lies outside 2^+-8 (the
        // fp16 operands of the later sweeps want the leading weights near one) is it run again with every row's
        // own maximum as shift, which is then known.
        float tmax = 0.f;          // the row's largest scaled score (log2 units)
        {
            float part = 0.f;
            mx2 = 0.f;
            // (solve mode with the row statistics given: nothing to sweep for)
            constexpr bool given = GIVEN;
            if (given && row_ok) {
                mx2 = prm.stats_in[((size_t)bh * nq + row) * 3 + 0] * 1.4426950408889634f;
                tmax = mx2;
            }
            for (int attempt = 0; attempt < 2 && ok && !given; ++attempt) {
                smax = -INFINITY;
                start_sweep(SW_STATS);
                part = sweep(SW_STATS);
                if (ok) acc_wait();
                ok = all_ok(ok);
                if (!ok) break;
                tmax = pair_max(smax) + mx2;
                if (attempt == 1 || !group_any(row_ok && !(fabsf(tmax) <= 8.f))) break;
                mx2 = fabsf(tmax) < 1e30f ? tmax : 0.f;     // (a row without a finite score keeps shift zero)
            }
            if (ok) {
                float acc[NCOL];
                if (given) {
                    omega = row_ok ? prm.stats_in[((size_t)bh * nq + row) * 3 + 1] : 1.f;
#pragma unroll
                    for (int col = 0; col < NCOL; col += 4) {
                        float4 kb4 = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (row_ok) kb4 = *reinterpret_cast<const float4*>(prm.kbar_in + ((size_t)bh * nq + row) * D + c0 + col);
                        acc[col] = kb4.x * omega; acc[col + 1] = kb4.y * omega; acc[col + 2] = kb4.z * omega; acc[col + 3] = kb4.w * omega;
                    }
                } else {
                    acc_load(acc);
                    omega = pair_sum(part);
                }
                inv_omega = 1.f / omega;
                const float lam_i = (prm.lambda_rows && row < nq) ? prm.lambda_rows[(size_t)bh * nq + row] : prm.lambda;
                // ridge in the frame of the shift: lambda e^{-shift} by the definition; the printed algorithm adds
                // lambda in the frame of the row maximum, i.e. lambda e^{max - shift} here
                ridge = lam_i * ex2f((prm.ridge_mode == LLA_RIDGE_PRINTED ? tmax : 0.f) - mx2) * inv_omega;
                float rr_p = 0.f, ab_p = 0.f;
#pragma unroll
                for (int ch = 0; ch < NCOL / 8; ++ch) {
                    const uint4 qraw = *reinterpret_cast<const uint4*>(smem + SM_Q + oper_off(ch));
                    const uint32_t qw[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float qv = q_elem(qw, e);
                        const int col = ch * 8 + e;
                        const float kb = acc[col] * inv_omega;
                        kbs[(c0 + col) * TC_BR + lrow] = kb;
                        xs[(c0 + col) * TC_BR + lrow] = 0.f;
                        const float bv = !row_ok ? 0.f : prm.rhs ? prm.rhs[((size_t)bh * nq + row) * D + c0 + col] : kb - qv;
                        r_set(col, bv);
                        p[col] = bv;
                        rr_p += bv * bv;
                        ab_p += kb * bv;
                    }
                }
                rr = pair_sum(rr_p);
                abar = pair_sum(ab_p);
                stop = prm.tol * prm.tol * rr;
                active = row_ok && rr > 0.f;
                pn2 = rr;
                rz = rr;
            }
        }
        if (ok && PC) {
            // preconditioned start: p = z = M r, with r . z, kbar . z and |z|^2 for the recurrences
            precondition(p, rr);
            ok = all_ok(ok);
            if (ok) {
                float rz_p = 0.f, kz_p = 0.f, zz_p = 0.f, unused = 0.f;
#pragma unroll
                for (int e = 0; e < NCOL; ++e) {
                    rz_p = fmaf(r_get(e), p[e], rz_p);
                    kz_p = fmaf(kbs[(c0 + e) * TC_BR + lrow], p[e], kz_p);
                    zz_p = fmaf(p[e], p[e], zz_p);
                }
                pair_sum4(rz_p, kz_p, zz_p, unused);
                if (rz_p > 0.f) {
                    rz = rz_p; abar = kz_p; pn2 = zz_p;
                } else {
                    // the rounded matrix is not positive on this residual: the row runs unpreconditioned
                    // (abar, pn2 and rz already hold the values for p = r)
                    prec_row = false;
#pragma unroll
                    for (int e = 0; e < NCOL; ++e) p[e] = r_get(e);
                }
            }
        }
        if (ok) write_p(0);
        // ---- conjugate gradients (Algorithm 2) ----
        int t = 0;      // CG sweeps run
        for (; ok && t < prm.max_iters; ++t) {
            active = active && rr > stop;
            if (!group_any(active)) break;
            const bool cheap = f16_on && t >= precise;
            start_sweep(cheap ? SW_CG16 : SW_CG, cheap);
            sweep(cheap ? SW_CG16 : SW_CG);
            if (ok) acc_wait();
            ok = all_ok(ok);
            if (!ok) break;
            float ap[NCOL];
            acc_load(ap);
            // (the loops below keep four independent partial sums and move the row-vector state in
            //  batches of eight so that the loads overlap: two warps per scheduler hide no latency)
            float pp[4] = {0.f, 0.f, 0.f, 0.f};
            const float acc_scale = cheap ? inv_omega * ipsc : inv_omega;
#pragma unroll
            for (int e = 0; e < NCOL; ++e) {
                ap[e] = fmaf(ap[e], acc_scale, ridge * p[e]);
                pp[e & 3] = fmaf(p[e], ap[e], pp[e & 3]);
            }
            const float pap = pair_sum((pp[0] + pp[1]) + (pp[2] + pp[3]));
            if (active && !(pap > 0.f)) active = false;
            const float alpha = active ? rz / pap : 0.f;       // rz = |r|^2 without a preconditioner
            float r2[4] = {0.f, 0.f, 0.f, 0.f}, kr[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int e0 = 0; e0 < NCOL; e0 += 8) {
                float xv[8], kv[8], rv[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    xv[i] = xs[(c0 + e0 + i) * TC_BR + lrow];
                    kv[i] = kbs[(c0 + e0 + i) * TC_BR + lrow];
                    rv[i] = r_get(e0 + i);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    xv[i] = fmaf(alpha, p[e0 + i], xv[i]);
                    rv[i] = fmaf(-alpha, ap[e0 + i], rv[i]);
                    ap[e0 + i] = rv[i];                       // ap now holds the new residual
                    r2[i & 3] = fmaf(rv[i], rv[i], r2[i & 3]);
                    kr[i & 3] = fmaf(kv[i], rv[i], kr[i & 3]);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    xs[(c0 + e0 + i) * TC_BR + lrow] = xv[i];
                    r_set(e0 + i, rv[i]);
                }
            }
            float rr2 = (r2[0] + r2[1]) + (r2[2] + r2[3]), kbr = (kr[0] + kr[1]) + (kr[2] + kr[3]);
            if constexpr (!PC) {
                // ||r_new||^2 and kbar . r_new in one exchange; kbar . p_new follows from the recurrence
                pair_sum2(rr2, kbr);
                if (active) {
                    const float beta = rr2 / rr;
#pragma unroll
                    for (int e = 0; e < NCOL; ++e) p[e] = fmaf(beta, p[e], ap[e]);
                    abar = fmaf(beta, abar, kbr);
                    pn2 = fmaf(beta * beta, pn2, rr2);
                    rr = rr2;
                    rz = rr2;
                    ++its;
                }
            } else {
                // preconditioned: z = M r_new (ap <- z), then beta = (r_new . z_new) / (r . z), p = z + beta p;
                // kbar . p and a bound on |p| follow from kbar . z and |z|
                rr2 = pair_sum(rr2);
                precondition(ap, rr2);
                ok = all_ok(ok);
                if (!ok) break;
                float rz_p = 0.f, kz_p = 0.f, zz_p = 0.f;
#pragma unroll
                for (int e0 = 0; e0 < NCOL; e0 += 8) {
                    float kv[8], rv[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        kv[i] = kbs[(c0 + e0 + i) * TC_BR + lrow];
                        rv[i] = r_get(e0 + i);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (!prec_row) ap[e0 + i] = rv[i];           // a row whose preconditioner failed: z = r
                        rz_p = fmaf(rv[i], ap[e0 + i], rz_p);
                        kz_p = fmaf(kv[i], ap[e0 + i], kz_p);
                        zz_p = fmaf(ap[e0 + i], ap[e0 + i], zz_p);
                    }
                }
                pair_sum4(rz_p, kz_p, zz_p, kbr);
                if (active) {
                    float beta = rz_p / rz;
                    if (!(rz_p > 0.f)) {
                        // r . M r is not positive (the rounded matrix is not definite on this residual): restart the
                        // row from its current x as plain CG, p = r
                        prec_row = false;
                        beta = 0.f;
                        rz_p = rr2; kz_p = kbr; zz_p = rr2;
#pragma unroll
                        for (int e = 0; e < NCOL; ++e) ap[e] = r_get(e);
                    }
#pragma unroll
                    for (int e = 0; e < NCOL; ++e) p[e] = fmaf(beta, p[e], ap[e]);
                    abar = fmaf(beta, abar, kz_p);
                    const float pn = sqrtf(zz_p) + fabsf(beta) * sqrtf(pn2);      // |p_new| <= |z| + |beta| |p|
                    pn2 = pn * pn;
                    rr = rr2;
                    rz = rz_p;
                    ++its;
                }
            }
            write_p(t + 1);
        }
        const bool at_cap = active && rr > stop;
        // ---- output sweep ----
        float gfac = 1.f;
        if (ok && prm.sol) {
            if (row_ok && LLA_IN_BOUNDS((size_t)bh * nq + row, (size_t)gridDim.x * nq, prm.status, 101)) {
                const size_t rowi = (size_t)bh * nq + row;
#pragma unroll
                for (int e = 0; e < NCOL; ++e) prm.sol[rowi * D + c0 + e] = xs[(c0 + e) * TC_BR + lrow];
                if (half == 0 && prm.iters) prm.iters[rowi] = its;
                if (half == 0 && prm.status) {
                    if (at_cap) atomicAdd(prm.status + LLA_STATUS_ROWS_AT_CAP, 1);
                    atomicAdd(prm.status + LLA_STATUS_ITER_SUM, its);
                }
            }
        } else if (ok) {
            float y[NCOL];
            float yb_p = 0.f, g_p = 0.f;
#pragma unroll
            for (int ch = 0; ch < NCOL / 8; ++ch) {
                const uint4 qraw = *reinterpret_cast<const uint4*>(smem + SM_Q + oper_off(ch));
                const uint32_t qw[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float qv = q_elem(qw, e);
                    const int col = ch * 8 + e;
                    const float kb = kbs[(c0 + col) * TC_BR + lrow];
                    y[col] = xs[(c0 + col) * TC_BR + lrow];
                    yb_p += kb * y[col];
                    g_p += (kb - qv) * y[col];
                }
            }
            abar = pair_sum(yb_p);
            gfac = 1.f + pair_sum(g_p);
            const bool out16 = f16_on && t >= precise;      // the format every role derives from the CG sweeps it has seen
            if (out16) write_operand16_pair(y);
            else write_operand(y);
            start_sweep(SW_OUT, out16);
            const float part = sweep(SW_OUT);
            if (ok) acc_wait();
            ok = all_ok(ok);
            if (ok) {
                float o[NCOL];
                acc_load(o);
                den = pair_sum(part);
                if (row_ok && LLA_IN_BOUNDS((size_t)bh * nq + row, (size_t)gridDim.x * nq, prm.status, 102)) {
                    const float inv_den = 1.f / den;
                    const size_t rowi = (size_t)bh * nq + row;
                    TOut* orow = out + prm.so.at(bh / prm.H, bh % prm.H, row) + c0;
#pragma unroll
                    for (int e = 0; e < NCOL; ++e) store_out(orow + e, o[e] * inv_den);
                    if (prm.rho) {
                        const float ig = 1.f / gfac;
#pragma unroll
                        for (int e = 0; e < NCOL; ++e) prm.rho[rowi * D + c0 + e] = y[e] * ig;
                    }
                    if (half == 0) {
                        if (prm.stats) {
                            prm.stats[rowi * 3 + 0] = mx2 * 0.6931471805599453f;      // the shift the weights were formed with
                            prm.stats[rowi * 3 + 1] = omega;
                            prm.stats[rowi * 3 + 2] = omega / gfac;
                        }
                        if (prm.iters) prm.iters[rowi] = its;
                        if (prm.status) {
                            if (at_cap) atomicAdd(prm.status + LLA_STATUS_ROWS_AT_CAP, 1);
                            atomicAdd(prm.status + LLA_STATUS_ITER_SUM, its);
                        }
                    }
                }
            }
        }
        if (ok) start_sweep(SW_DONE);
    }

    // ================================ common exit ================================
    // (on an aborted run the TMA warp and the MMA warps have waited above for what they had issued)
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag && prm.status) atomicAdd(prm.status + LLA_STATUS_TIMEOUT, 1);
}

// Pre-pass of the fp16 sweeps: writes an fp16 copy of k and clears *ok if an entry of k or q lies outside
// the range in which that copy is faithful (magnitude above 60000; bf16 values below the fp16 subnormal
// spacing simply round, an absolute change under 3e-8).  Eight elements per thread and step.
__global__ void __launch_bounds__(256)
f16_copy_kernel(const __nv_bfloat16* __restrict__ k, uint4* __restrict__ k16, int Hk, int n, int d, Strides sk,
                const __nv_bfloat16* __restrict__ q, int H, int nq, Strides sq, int B, int* __restrict__ ok) {
    bool bad = false;
    const size_t stride = (size_t)gridDim.x * blockDim.x, t0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int vpr = d / 8;                                   // 16-byte groups per row
    const size_t k_vec = (size_t)B * Hk * n * vpr, q_vec = (size_t)B * H * nq * vpr;
    for (size_t i = t0; i < k_vec; i += stride) {
        const int c = (int)(i % vpr);
        const size_t rowi = i / vpr;
        const int row = (int)(rowi % n), unit = (int)(rowi / n);
        const uint4 raw = *reinterpret_cast<const uint4*>(k + sk.at(unit / Hk, unit % Hk, row) + 8 * c);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        uint32_t h[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float a = __uint_as_float(w[e] << 16), b = __uint_as_float(w[e] & 0xFFFF0000u);
            bad |= !(fabsf(a) <= 60000.f) || !(fabsf(b) <= 60000.f);
            h[e] = pack_f16(a, b);
        }
        k16[i] = make_uint4(h[0], h[1], h[2], h[3]);         // the copy is contiguous [B][Hk][n][d]
    }
    for (size_t i = t0; i < q_vec; i += stride) {
        const int c = (int)(i % vpr);
        const size_t rowi = i / vpr;
        const int row = (int)(rowi % nq), unit = (int)(rowi / nq);
        const uint4 raw = *reinterpret_cast<const uint4*>(q + sq.at(unit / H, unit % H, row) + 8 * c);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
            bad |= !(fabsf(__uint_as_float(w[e] << 16)) <= 60000.f) || !(fabsf(__uint_as_float(w[e] & 0xFFFF0000u)) <= 60000.f);
    }
    if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) *ok = 0;
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }
// bytes of the fp16 copy of k plus its status word
size_t f16_copy_bytes(size_t k_elems) { return round256(k_elems * 2) + 256; }
// Per-device scratch for the D = 128 kernel: one slot per SM id, shared by every launch on the device.
// A block of this kernel fills an SM (shared memory), so two blocks never use one slot at a time,
// whichever launches or streams they come from.
float* scratch_for_device(size_t bytes) {
    static std::mutex mu;
    static float* ptr[64] = {};
    static size_t have[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (have[dev] < bytes) {
        if (ptr[dev]) cudaFree(ptr[dev]);
        ptr[dev] = nullptr;
        have[dev] = 0;
        void* p = nullptr;
        if (cudaMalloc(&p, bytes) != cudaSuccess) return nullptr;
        ptr[dev] = static_cast<float*>(p);
        have[dev] = bytes;
    }
    return ptr[dev];
}

// Launch order of the query tiles: longest first, so that the blocks left for the end are short.
// A tile's cost is (sweeps) x (per-sweep overhead + key blocks).  Sweeps = 3 + CG iterations, and the
// iteration count falls with the number of visible keys per dimension (the first tiles need several
// times more than the rest), so at short sequence lengths the first tiles are the longest blocks
// even though their sweeps are the shortest.  The numbers are a fit to measured runs; they only
// steer the order, never the result.
void tile_order(TcParams& prm, int tiles, int first_tile, int n, int off, int d, int causal, int window, bool precond) {
    prm.use_order = 0;
    if (!causal || tiles > TC_ORDER_MAX) return;
    float cost[TC_ORDER_MAX];
    for (int t = 0; t < tiles; ++t) {
        const int r_end = std::min(n, off + (first_tile + t + 1) * TC_BR);      // keys the tile's last row sees
        const int seen = window > 0 ? std::min(r_end, window) : r_end;
        const float x = (float)d / (float)seen;
        const float its = precond ? std::min(16.f, 4.f + 190.f * x * x) : 6.f + 50.f * x;
        const int c_first = window > 0 ? std::max(0, off + (first_tile + t) * TC_BR + 1 - window) / TC_BC : 0;
        const float nblk = (float)((r_end + TC_BC - 1) / TC_BC - c_first);
        cost[t] = (its + 2.f) * (6.f + nblk) + (precond ? 3.f * its : 0.f);
        prm.order[t] = (unsigned short)t;
    }
    std::stable_sort(prm.order, prm.order + tiles, [&](unsigned short x, unsigned short y) { return cost[x] > cost[y]; });
    prm.use_order = 1;
}

template <int D, typename TOut>
int launch_t(const ForwardArgs& a) {
    using Cfg = TcCfg<D>;
    const int hr = head_rows_count(a);
    if (!a.causal && hr >= a.nq) return LLA_OK;
    const int first_tile = a.causal ? hr / TC_BR : 0;
    const int tiles = (a.nq + TC_BR - 1) / TC_BR - first_tile;
    if (tiles <= 0) return LLA_OK;
    CUtensorMap mq, mk, mv, mk16, mm;
    const int BH = a.B * a.H;
    const int Hk = a.H / a.kv_group;
    const auto BF = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, F16 = CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    if (!make_map_16bit_4d(&mq, a.q, a.B, a.H, a.nq, D, a.sq.b, a.sq.h, a.sq.r, TC_BR, BF) ||
        !make_map_16bit_4d(&mk, a.k, a.B, Hk, a.n, D, a.sk.b, a.sk.h, a.sk.r, TC_BC, BF) ||
        !make_map_16bit_4d(&mv, a.v, a.B, Hk, a.n, D, a.sv.b, a.sv.h, a.sv.r, TC_BC, BF))
        return LLA_ERR_CUDA;
    mk16 = mk;
    mm = mk;
    TcParams prm;
    prm.n = a.n; prm.nq = a.nq; prm.causal = a.causal; prm.head_rows = a.head_rows > 0 ? a.head_rows : 0;
    prm.max_iters = a.max_iters; prm.first_tile = first_tile;
    prm.precise_iters = a.precise_iters;
    prm.precise_iters_early = a.precise_iters_early;
    prm.wait_clocks = a.wait_clocks > 0 ? a.wait_clocks : kWaitClocks;
    prm.no_loads = a.no_loads;
    prm.scale = a.scale; prm.lambda = a.lambda; prm.tol = a.tol;
    prm.lambda_rows = a.lambda_rows; prm.ridge_mode = a.ridge_mode;
    prm.block_mask = a.block_mask; prm.block_mask_stride = a.block_mask_stride;
    prm.rhs = a.rhs; prm.sol = a.sol; prm.kbar_in = a.kbar_in; prm.stats_in = a.stats_in;
    prm.H = a.H; prm.kv_group = a.kv_group > 0 ? a.kv_group : 1;
    prm.so = a.so;
    prm.rho = a.rho; prm.stats = a.stats; prm.iters = a.iters; prm.status = a.status;
    prm.scratch = nullptr;
    prm.scratch_slots = 0;
    prm.f16_ok = nullptr;
    // the caller's workspace is cut into the D = 128 row-state slots (if it holds them) and the fp16 copy of k
    char* ws = static_cast<char*>(a.workspace);
    size_t ws_left = a.workspace ? a.workspace_bytes : 0;
    prm.window = a.causal ? a.window : 0;
    tile_order(prm, tiles, first_tile, a.n, a.n - a.nq, D, a.causal, prm.window, a.minv != nullptr);
    if constexpr (!Cfg::STATE_IN_SMEM) {
        int dev = 0, sms = 0;
        LLA_CUDA_TRY(cudaGetDevice(&dev));
        LLA_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        prm.scratch_slots = 2 * sms;     // SM ids are dense in practice; the margin is checked in the kernel
        const size_t need = (size_t)prm.scratch_slots * Cfg::SCRATCH_FLOATS_PER_SM * sizeof(float);
        // the caller's workspace if it is large enough (then nothing is allocated, but two calls that may
        // run at the same time must not share it), else the library's own per-device buffer
        if (ws && ws_left >= need) {
            prm.scratch = reinterpret_cast<float*>(ws);
            ws += round256(need);
            ws_left -= std::min(ws_left, round256(need));
        } else {
            prm.scratch = scratch_for_device(need);
        }
        if (!prm.scratch) return LLA_ERR_CUDA;
    }
    // fp16 sweeps: only with the copy of k that forward_tensor_prepass made; without it every sweep runs on
    // the bf16 inputs
    if (a.k16 && a.f16_ok) {
        const Strides c16 = contiguous_strides(Hk, a.n, D);
        if (!make_map_16bit_4d(&mk16, a.k16, a.B, Hk, a.n, D, c16.b, c16.h, c16.r, TC_BC, F16)) return LLA_ERR_CUDA;
        prm.f16_ok = a.f16_ok;
    }
    bool precond = false;
    // preconditioned CG: only with the matrices that forward_tensor_prepass made ([units][blocks][D][D] fp16)
    if (a.minv) {
        const Strides cm = contiguous_strides(Hk, (long long)precond_blocks(a.n) * D, D);
        if (!make_map_16bit_4d(&mm, a.minv, a.B, Hk, (long long)precond_blocks(a.n) * D, D, cm.b, cm.h, cm.r, 64, F16)) return LLA_ERR_CUDA;
        precond = true;
    }
    auto kern = precond ? forward_tc_kernel<D, TOut, true> : forward_tc_kernel<D, TOut, false>;
    if constexpr (std::is_same<TOut, float>::value) {
        if (a.sol && a.kbar_in && a.stats_in) kern = precond ? forward_tc_kernel<D, TOut, true, true> : forward_tc_kernel<D, TOut, false, true>;
    }
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SM_ALLOC));
    dim3 grid(BH, tiles);
    kern<<<grid, D == 128 ? 384 : TC_THREADS, Cfg::SM_ALLOC, a.stream>>>(mq, mk, mv, mk16, mm, (TOut*)a.out, prm);
    LLA_CUDA_TRY(cudaGetLastError());
    return LLA_OK;
}

}  // namespace

size_t forward_tensor_scratch_bytes() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return round256((size_t)2 * sms * TcCfg<128>::SCRATCH_FLOATS_PER_SM * sizeof(float));
}

size_t forward_tensor_workspace_bytes(int B, int H, int n, int d) {
    return (d == 128 ? forward_tensor_scratch_bytes() : 0) + f16_copy_bytes((size_t)B * H * n * d) +
           precond_gram_bytes(B * H, n, d) + precond_minv_bytes(B * H, n, d);
}

// Enqueues the fp16 copy of k (and the range check of q and k) when the tail of the caller's workspace has
// room for it, and records where it is in `a`; the head of the workspace is left to the D = 128 row state.
int forward_tensor_prepass(ForwardArgs& a) {
    a.k16 = nullptr;
    a.f16_ok = nullptr;
    a.minv = nullptr;
    if (!forward_tensor_supported(a) || !a.workspace) return LLA_OK;
    if (std::min(a.precise_iters, a.precise_iters_early) >= (1 << 29)) return LLA_OK;
    const size_t head = a.d == 128 ? forward_tensor_scratch_bytes() : 0;
    const size_t k_elems = (size_t)(a.B * a.H / a.kv_group) * a.n * a.d;
    if (a.workspace_bytes < head + f16_copy_bytes(k_elems)) return LLA_OK;
    char* ws = static_cast<char*>(a.workspace) + head;
    uint4* k16 = reinterpret_cast<uint4*>(ws);
    int* okw = reinterpret_cast<int*>(ws + round256(k_elems * 2));
    LLA_CUDA_TRY(cudaMemsetAsync(okw, 1, sizeof(int), a.stream));
    const size_t k_vec = k_elems / 8;
    const unsigned blocks = (unsigned)std::min<size_t>((k_vec + 255) / 256, 148 * 8);
    f16_copy_kernel<<<blocks, 256, 0, a.stream>>>(static_cast<const __nv_bfloat16*>(a.k), k16, a.H / a.kv_group, a.n, a.d, a.sk,
                                                   static_cast<const __nv_bfloat16*>(a.q), a.H, a.nq, a.sq, a.B, okw);
    LLA_CUDA_TRY(cudaGetLastError());
    a.k16 = k16;
    a.f16_ok = okw;
    // the preconditioner behind it, if enabled and there is room (Gram scratch, then the matrices)
    const int units = a.B * a.H / a.kv_group;
    const size_t used = head + f16_copy_bytes(k_elems);
    const size_t gram_b = precond_gram_bytes(units, a.n, a.d), minv_b = precond_minv_bytes(units, a.n, a.d);
    if (a.precondition && a.workspace_bytes >= used + gram_b + minv_b) {
        char* gram = static_cast<char*>(a.workspace) + used;
        char* minv = gram + gram_b;
        const int rc = launch_precond(a.k, a.B, a.H / a.kv_group, a.sk, a.n, a.d, a.lambda, a.causal ? a.window : 0, gram, minv, a.stream);
        if (rc != LLA_OK) return rc;
        a.minv = minv;
    }
    return LLA_OK;
}

bool forward_tensor_supported(const ForwardArgs& a) {
    return a.in_dtype == LLA_BF16 && (a.d == 64 || a.d == 128) && a.dv == a.d && get_encode() != nullptr;
}

int launch_forward_tensor(const ForwardArgs& a) {
    if (!forward_tensor_supported(a)) return LLA_ERR_UNSUPPORTED;
    if (a.d == 64) {
        if (a.out_dtype == LLA_BF16) return launch_t<64, __nv_bfloat16>(a);
        if (a.out_dtype == LLA_F32) return launch_t<64, float>(a);
    } else {
        if (a.out_dtype == LLA_BF16) return launch_t<128, __nv_bfloat16>(a);
        if (a.out_dtype == LLA_F32) return launch_t<128, float>(a);
    }
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
