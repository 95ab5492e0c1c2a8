// LLA decode on tensor cores (bf16 caches, d = dv = 64): one pass over the KV cache at HBM speed.
//
// Decode is bound by reading K and V once, so the cache is streamed a single time and folded into
// the weighted moments about the origin that the centred form of Eq. "lla_decomp" needs:
//     D = [K^T ; V^T] diag(w) [K | 1]      (128 x 80, fp32 in TMEM)
//       rows 0..63   : M = sum_j w_j k_j k_j^T   and, in column 64, a = sum_j w_j k_j
//       rows 64..127 : N = sum_j w_j v_j k_j^T   and, in column 64, c = sum_j w_j v_j
// Per 64-key tile:
//   TMA         K and V tiles -> 128B-swizzled shared memory (4-stage ring).  The two tiles sit back
//               to back and together form the MN-major A operand [K^T ; V^T] of one M = 128 MMA.
//   CUDA cores  two lanes per key (16 lanes apart): score s_j = scale q.k_j, weight w_j = exp(s_j - m_ref), then the
//               row w_j [k_j | 1] split into bf16 hi + lo is written to the B operand tiles
//               (canonical MN-major layout without swizzle, 80 columns); omega += w_j.
//   MMA (SS)    [D_hi | D_lo] += A [B_hi | B_lo]: the two B tiles lie back to back and are read as one
//               N = 160 operand, so A is fetched once per 16-key step; D = D_hi + D_lo is formed
//               when the accumulator is read out.
// m_ref is the maximum of the first tile.  The threads only note whether a later score exceeds it by more
// than 2^90 (no barrier per tile); if one did, the whole pass is repeated with the true maximum, which is
// known by then (never triggered by bounded scores, covered by a test).  After
// the last tile the moments are copied to shared memory and either solved on the spot (d x d LDL^T
// in double precision, as in lla_decode.cu) or written as a partial record for the split-key merge.
#include "lla_sm100.cuh"

namespace lla {
namespace {

using namespace sm100;

constexpr int DT_CG_CAP = 192;   // iteration cap of the d x d solve (the factorisation takes over beyond it)
constexpr int DT_D = 64;
constexpr int DT_BK = 64;             // keys per tile
constexpr int DT_NST = 4;             // K/V ring stages
constexpr int DT_COMPUTE = 128;       // warps 0..3
constexpr int DT_THREADS = 192;       // + TMA warp (4) + MMA warp (5)
constexpr int DT_TMEM_COLS = 256;     // 160 accumulator columns (hi | lo), power-of-two allocation
constexpr int DT_N = 80;              // MMA N: 64 key features + the ones column (padded to 16)
constexpr int DT_MAX_RANKED = 1024;   // batches up to this size are processed longest-first
constexpr int DT_BTILE = 10240;       // one B tile: 10 column blocks x 8 key blocks x 128 bytes

constexpr int SMD_KV = 0;                                   // DT_NST x (K 8192 + V 8192)
constexpr int SMD_B = SMD_KV + DT_NST * 16384;              // 2 buffers x (hi, lo) x DT_BTILE
constexpr int SMD_BAR = SMD_B + 4 * DT_BTILE;               // mbarriers
constexpr int SMD_MISC = SMD_BAR + 128;                     // tmem base, abort, tile maxima
constexpr int SMD_TOTAL = SMD_MISC + 128;
// the epilogue reuses everything from offset 0: M (64 x 65 doubles), a, c, rhs (3 x 64 doubles), N (64 x 64 floats)
constexpr int SMD_FIN = 8 * (64 * 65 + 3 * 64) + 4 * 64 * 65 + 8 * (128 + 24);
constexpr int SMD_ALLOC = (SMD_TOTAL > SMD_FIN ? SMD_TOTAL : SMD_FIN) + 1024;

enum { DB_KVFULL = 0, DB_KVEMPTY = DB_KVFULL + DT_NST, DB_BFULL = DB_KVEMPTY + DT_NST, DB_BFREE = DB_BFULL + 2,
       DB_DFULL = DB_BFREE + 2, DB_PASS = DB_DFULL + 1, DB_EXIT = DB_PASS + 1, DB_COUNT = DB_EXIT + 1 };
static_assert(DB_COUNT * 8 <= 128, "barrier area too small");

// A = [K^T ; V^T]: MN-major, 128B swizzle; the V tile (second group of 64 rows of M) lies 8192 bytes
// after the K tile (leading byte offset), 8-key groups are 1024 bytes apart (stride byte offset).
__device__ __forceinline__ uint64_t make_desc_a(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(8192 >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;      // SWIZZLE_128B
    return d;
}
// B: MN-major without swizzle: 8 x 8 core matrices of 128 bytes; key groups are 128 bytes apart
// (leading byte offset), column groups 1024 bytes apart (stride byte offset).
__device__ __forceinline__ uint64_t make_desc_b(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(128 >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    return d;                    // layout type 0: no swizzle
}
constexpr uint32_t IDESC_DEC = make_idesc(128, 2 * DT_N, 1, 1);

// [D_hi | D_lo] += A [B_hi | B_lo] over 64 keys.  A steps 2048 bytes (128 units) per 16 keys, B 256 bytes (16 units).
__device__ __forceinline__ void mma_tile(uint32_t el, uint32_t d, uint64_t a, uint64_t b, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 a1, a2, a3, h1, h2, h3;\n\t"
        "setp.ne.b32 q, %0, 0;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "add.u64 a1, %2, 128; add.u64 a2, %2, 256; add.u64 a3, %2, 384;\n\t"
        "add.u64 h1, %3, 16; add.u64 h2, %3, 32; add.u64 h3, %3, 48;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], %2, %3, %4, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a1, h1, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a2, h2, %4, p;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%1], a3, h3, %4, p;\n\t}"
        ::"r"(el), "r"(d), "l"(a), "l"(b), "r"(IDESC_DEC), "r"(acc0) : "memory");
}

// Solve C x = b for an explicit symmetric positive-definite 64 x 64 matrix with conjugate gradients in
// double precision, run by the 128 threads of warps 0..3: thread 2r + hh holds columns 32hh..32hh+31
// of row r in cr[] and passes b[r].  A dense factorisation is a chain of 64 dependent column steps;
// here an iteration is one short matrix-vector product and the decode systems (>= 2d keys) need one
// or two dozen of them.  The matrix stays in registers for the whole solve (re-reading it from shared
// memory every iteration costs several times more than the arithmetic).  The recurrences are the
// Chronopoulos-Gear form: both inner products of an iteration, (r, r) and (C r, r), are taken after the
// matrix-vector product, so an iteration has one reduction and two 128-thread barriers.
// x lands in xs[]; returns false if the residual did not reach 1e-9 |b| within the iteration cap or the
// recurrence broke down (the caller then falls back to the factorisation).
// Thread layout of the 64 x 64 solve over 128 threads: a thread keeps a 4 x 8 block of the matrix --
// rows cg_row0(tid) .. +3, columns cg_col0(tid) .. +7, as cr[8 i + j] -- so that a matrix-vector product
// reads eight entries of the vector per thread (the shared-memory-to-register path bounds this kernel;
// half rows of 32 entries read four times as much).  The eight lanes that share four rows then reduce
// their partial sums by recursive halving (four 64-bit shuffles), after which lane pairs hold the
// product's entry for row cg_row(tid).
__device__ __forceinline__ int cg_row0(int tid) { return 16 * (tid >> 5) + 4 * ((tid & 31) >> 3); }
__device__ __forceinline__ int cg_col0(int tid) { return 8 * (tid & 7); }
__device__ __forceinline__ int cg_row(int tid) { return cg_row0(tid) + 2 * ((tid >> 2) & 1) + ((tid >> 1) & 1); }
__device__ __forceinline__ bool cg_solve_64(const double (&cr)[32], const double b_r, double* xs, double* pbuf, double* redbuf, int& iters) {
    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
    const int r = cg_row(tid);
    const bool owner = (tid & 1) == 0, b4 = (tid & 4) != 0, b2 = (tid & 2) != 0;
    auto sync128 = [&]() { asm volatile("bar.sync 2, 128;" ::: "memory"); };
    double x = 0.0, rv = b_r, pv = 0.0, sv = 0.0, alpha = 0.0, gamma_old = 0.0, stop = 0.0;
    bool done = false;
    iters = 0;
    for (int it = 0; it <= DT_CG_CAP; ++it) {
        if (owner) pbuf[r] = rv;
        sync128();
        const double2* pp = reinterpret_cast<const double2*>(pbuf + cg_col0(tid));
        const double2 p01 = pp[0], p23 = pp[1], p45 = pp[2], p67 = pp[3];
        double a[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const double e0 = fma(cr[8 * i + 1], p01.y, cr[8 * i] * p01.x);
            const double e1 = fma(cr[8 * i + 3], p23.y, cr[8 * i + 2] * p23.x);
            const double e2 = fma(cr[8 * i + 5], p45.y, cr[8 * i + 4] * p45.x);
            const double e3 = fma(cr[8 * i + 7], p67.y, cr[8 * i + 6] * p67.x);
            a[i] = (e0 + e1) + (e2 + e3);
        }
        // recursive halving over the eight lanes of a row group: 4 -> 2 -> 1 partial sums, then the pair
        const double k0 = (b4 ? a[2] : a[0]) + __shfl_xor_sync(0xffffffffu, b4 ? a[0] : a[2], 4);
        const double k1 = (b4 ? a[3] : a[1]) + __shfl_xor_sync(0xffffffffu, b4 ? a[1] : a[3], 4);
        double wv = (b2 ? k1 : k0) + __shfl_xor_sync(0xffffffffu, b2 ? k0 : k1, 2);
        wv += __shfl_xor_sync(0xffffffffu, wv, 1);           // both lanes of a pair now hold (C r)_row
        // (r, r) and (C r, r): each parity class of lanes sums the warp's 16 rows once
        double g = rv * rv, dl = wv * rv;
#pragma unroll
        for (int off = 2; off <= 16; off <<= 1) {
            g += __shfl_xor_sync(0xffffffffu, g, off);
            dl += __shfl_xor_sync(0xffffffffu, dl, off);
        }
        double* rb = redbuf + (it & 1) * 8;
        if (lane == 0) { rb[wp] = g; rb[4 + wp] = dl; }
        sync128();
        const double gamma = (rb[0] + rb[1]) + (rb[2] + rb[3]);
        const double delta = (rb[4] + rb[5]) + (rb[6] + rb[7]);
        // |r| <= 1e-4 |b|, the forward's own CG tolerance for bf16 inputs: the output error is then 1.1e-4
        // row-wise, as for a prefill row (1e-5 |b| gives 1.6e-5, 1e-9 |b| 0.8e-5 -- from there on the fp32 moments
        // set it -- for two and five more iterations)
        if (it == 0) stop = gamma * 1e-8;
        if (!(gamma > stop)) { done = true; break; }
        double beta = 0.0, denom = delta;
        if (it > 0) {
            beta = gamma * fast_rcp(gamma_old);
            denom = delta - beta * gamma * fast_rcp(alpha);
        }
        if (!(denom > 0.0) || it == DT_CG_CAP) break;
        alpha = gamma * fast_rcp(denom);
        pv = rv + beta * pv;
        sv = wv + beta * sv;
        x += alpha * pv;
        rv -= alpha * sv;
        gamma_old = gamma;
        ++iters;
    }
    if (owner) xs[r] = x;
    sync128();
    return done;
}

__device__ __forceinline__ void named_sync_128() { asm volatile("bar.sync 1, 128;" ::: "memory"); }



struct DtParams {
    int B, H, Lmax, splits, head_rows;
    float scale, lambda;
    const int* lens;
    float* parts;
    int* status;
    int defer;           // 1: write the moment record even for a single part; a solve kernel follows
    const float* lambda_units;   // optional per-(sequence, head) ridge
    int ridge_mode;
    int kv_group;        // query heads per key/value head
    int window;          // sliding window (0: none)
    long long wait_clocks;   // cap of every bounded wait, in SM clocks
    int no_loads;        // test aid: the TMA warp issues no copy at all, so that every wait expires with nothing in flight
    PagedKv paged;       // table != nullptr: the tensor maps cover [num_pages * kv heads][page_size][64]
};

template <typename TOut>
__global__ void __launch_bounds__(DT_THREADS, 2)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __nv_bfloat16* __restrict__ q, TOut* __restrict__ out, const DtParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + SMD_BAR;
    auto bar = [&](int i) { return bars + 8u * i; };
    volatile int* misc = reinterpret_cast<volatile int*>(smem + SMD_MISC);   // [0] tmem base, [1] abort
    volatile int* abort_flag = misc + 1;
    volatile float* tmax = reinterpret_cast<volatile float*>(smem + SMD_MISC + 16);   // 2 x 4 warp maxima
    const long long wcap = prm.wait_clocks;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int part = blockIdx.x;
    // Longest caches first: blocks launch in blockIdx order, so block y takes head (y % H) of the
    // sequence whose length has rank (y / H).  Every block ranks the (few) sequence lengths itself.
    int bh = blockIdx.y;
    if (prm.B <= DT_MAX_RANKED) {
        __shared__ int s_len[DT_MAX_RANKED];
        __shared__ int s_pick;
        for (int b = tid; b < prm.B; b += DT_THREADS) s_len[b] = visible_keys(prm.lens[b], prm.Lmax, prm.window);
        __syncthreads();
        const int want = blockIdx.y / prm.H;
        for (int b = tid; b < prm.B; b += DT_THREADS) {
            const int lb = s_len[b];
            int rank = 0;
            for (int o = 0; o < prm.B; ++o) rank += (s_len[o] > lb) || (s_len[o] == lb && o < b);
            if (rank == want) s_pick = b;
        }
        __syncthreads();
        bh = s_pick * prm.H + blockIdx.y % prm.H;
    }
    const int kstart = first_visible_key(prm.lens[bh / prm.H], prm.Lmax, prm.window);   // sliding window
    const int L = visible_keys(prm.lens[bh / prm.H], prm.Lmax, prm.window);
    if (L < prm.head_rows) return;                      // short caches: solved by the direct fp64 kernel
    const int chunk = ((L + prm.splits - 1) / prm.splits + DT_BK - 1) / DT_BK * DT_BK;
    const int jbeg = part * chunk, jend = min(L, jbeg + chunk);
    const int ntile = jend > jbeg ? (jend - jbeg + DT_BK - 1) / DT_BK : 0;

    if (tid == 0) {
        for (int s = 0; s < DT_NST; ++s) { mbar_init(bar(DB_KVFULL + s), 1); mbar_init(bar(DB_KVEMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar(DB_BFULL + b), DT_COMPUTE / 32); mbar_init(bar(DB_BFREE + b), 1); }
        mbar_init(bar(DB_DFULL), 1);
        mbar_init(bar(DB_PASS), DT_COMPUTE / 32);
        mbar_init(bar(DB_EXIT), 1);
        misc[1] = 0;
        misc[2] = 0;      // set by the compute warps when the pass has to be repeated
        fence_barrier_init();
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(sbase + SMD_MISC), "r"(DT_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (uint32_t)misc[0];

    float omega = 0.f, m_ref = -INFINITY;     // compute threads; m_ref in log2 units
    uint32_t d_parity = 0;                     // compute threads: phase of the accumulator barrier to wait for

    if (warp == 4) {
        // ================================ TMA producer ================================
        if (lane == 0 && !prm.no_loads) {
            // K/V unit and row of a tile in the tensor map: (batch, key/value head) and the key index, or for a
            // paged cache (page, key/value head) and the row inside the page (a tile never straddles a page)
            const int hkv = prm.H / prm.kv_group, kvl = (bh % prm.H) / prm.kv_group;
            const int kvh = (bh / prm.H) * hkv + kvl;
            const int* table = prm.paged.table ? prm.paged.table + (size_t)(bh / prm.H) * prm.paged.max_pages : nullptr;
            int issued = 0;      // tiles whose copies have been issued
            for (int g = 0, pass = 0; pass < 2; ++pass) {
              bool okp = true;
              for (int t = 0; t < ntile; ++t, ++g) {      // g: running tile count over both passes (ring position)
                const uint32_t s = g % DT_NST;
                if (!mbar_wait(bar(DB_KVEMPTY + s), ((g / DT_NST) & 1) ^ 1, abort_flag, wcap)) { okp = false; break; }
                issued = g + 1;
                const uint32_t dst = sbase + SMD_KV + s * 16384;
                mbar_expect_tx(bar(DB_KVFULL + s), 16384);
                int unit = kvh, jrow = kstart + jbeg + t * DT_BK;
                if (table) {
                    const int page = min(max(table[jrow / prm.paged.page_size], 0), prm.paged.num_pages - 1);
                    unit = page * hkv + kvl;
                    jrow %= prm.paged.page_size;
                }
                tma_load_3d(dst, &tmK, bar(DB_KVFULL + s), 0, jrow, unit);
                tma_load_3d(dst + 8192, &tmV, bar(DB_KVFULL + s), 0, jrow, unit);
              }
              // a second pass only if the compute warps ask for it
              if (!okp || pass == 1 || ntile == 0 || !mbar_wait(bar(DB_PASS), 0, abort_flag, wcap) || misc[2] == 0) break;
            }
            if (*abort_flag) {      // an aborted block: the copies issued above must have landed before the block exits
                for (int g = max(0, issued - DT_NST); g < issued; ++g)
                    (void)mbar_wait_landed(bar(DB_KVFULL + g % DT_NST), (g / DT_NST) & 1, wcap);
            }
        }
    } else if (warp == 5) {
        // ================================ MMA issuer (whole warp, predicated) ================================
        const uint32_t el = elect_one();
        for (int g = 0, pass = 0; pass < 2; ++pass) {
            bool okp = true;
            for (int t = 0; t < ntile; ++t, ++g) {
                const uint32_t s = g % DT_NST, b = g & 1;
                if (!mbar_wait(bar(DB_KVFULL + s), (g / DT_NST) & 1, abort_flag, wcap)) { okp = false; break; }
                if (!mbar_wait(bar(DB_BFULL + b), (g >> 1) & 1, abort_flag, wcap)) { okp = false; break; }
                tc_fence_after();
                const uint32_t bsm = sbase + SMD_B + b * 2 * DT_BTILE;
                mma_tile(el, tmem, make_desc_a(sbase + SMD_KV + s * 16384), make_desc_b(bsm), t > 0);     // t == 0 overwrites
                tc_commit_el(el, bar(DB_KVEMPTY + s));
                tc_commit_el(el, bar(DB_BFREE + b));
                if (t == ntile - 1) tc_commit_el(el, bar(DB_DFULL));
            }
            if (!okp || pass == 1 || ntile == 0 || !mbar_wait(bar(DB_PASS), 0, abort_flag, wcap) || misc[2] == 0) break;
        }
        if (*abort_flag) {      // an aborted block: the MMAs issued above must be done before TMEM and shared memory go
            tc_commit_el(el, bar(DB_EXIT));
            (void)mbar_wait_landed(bar(DB_EXIT), 0, wcap);
        }
    } else {
        // ================================ compute warps ================================
        // key inside the tile and feature half: lanes 0..15 of a warp take the low halves of 16 keys,
        // lanes 16..31 the high halves, so the eight lanes that share a 128-byte shared-memory wavefront
        // have the same half and neighbouring keys (no bank conflicts in the tile loads or B stores)
        const int jl = warp * 16 + (lane & 15), h = lane >> 4;
        const float c1 = prm.scale * 1.4426950408889634f;
        float qv[32];
        {
            const __nv_bfloat16* qp = q + (size_t)bh * DT_D + 32 * h;
#pragma unroll
            for (int i = 0; i < 4; ++i) load8(qp + 8 * i, qv + 8 * i);
        }
        bool ok = true;
        const uint32_t rowoff = (jl >> 3) * 128 + (jl & 7) * 16;      // key group, row inside the core matrix
        // Software pipeline over tiles: the shared-memory loads of tile t+1 are issued before the
        // scale-and-store phase of tile t, and its score follows right after, so the two phases'
        // latencies overlap.  stage_load fetches this lane's 32 features of key jl (swizzled 16-byte
        // chunks 4h .. 4h+3) as raw bf16 pairs; stage_score turns them into kf[], the score and the weight.
        uint4 raw[4];
        float kf[32];
        float w = 0.f;
        // (t: tile of the pass, it fixes the keys; g: running tile count over both passes, it fixes ring stage,
        //  buffer and barrier phase)
        auto stage_load = [&](int g) -> bool {
            const uint32_t s = g % DT_NST;
            if (!mbar_wait(bar(DB_KVFULL + s), (g / DT_NST) & 1, abort_flag, wcap)) return false;
            uint8_t* ktile = smem + SMD_KV + s * 16384;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                raw[i] = *reinterpret_cast<const uint4*>(ktile + jl * 128 + (((4 * h + i) ^ (jl & 7)) << 4));
            return true;
        };
        float s2 = 0.f;
        bool valid = false;
        // first half of the score stage: arithmetic only (no barrier), so it can run while the
        // stores of the tile before are still draining
        auto stage_score_math = [&](int t, int g) {
            const uint32_t s = g % DT_NST;
            uint8_t* ktile = smem + SMD_KV + s * 16384;
            valid = jbeg + t * DT_BK + jl < jend;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t wds[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    kf[8 * i + 2 * e] = __uint_as_float(wds[e] << 16);
                    kf[8 * i + 2 * e + 1] = __uint_as_float(wds[e] & 0xFFFF0000u);
                }
            }
            if (!valid) {
                // ragged last tile: rows past the end may hold anything (unused cache slots).  They are
                // part of the A operand, so clear them (0 x NaN would poison the accumulator).
#pragma unroll
                for (int e = 0; e < 32; ++e) kf[e] = 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t off = jl * 128 + (((4 * h + i) ^ (jl & 7)) << 4);
                    *reinterpret_cast<uint4*>(ktile + off) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(ktile + 8192 + off) = make_uint4(0, 0, 0, 0);
                }
            }
            float sd[4] = {0.f, 0.f, 0.f, 0.f};          // four independent chains
#pragma unroll
            for (int e = 0; e < 32; ++e) sd[e & 3] = fmaf(qv[e], kf[e], sd[e & 3]);
            float sdot = (sd[0] + sd[1]) + (sd[2] + sd[3]);
            sdot += __shfl_xor_sync(0xffffffffu, sdot, 16);
            s2 = valid ? sdot * c1 : -INFINITY;
        };
        // second half: the weight.  The reference maximum is the first tile's (one block-wide reduction per pass at
        // most); later tiles only note, per thread and without any barrier, the largest score seen and whether one
        // exceeded the reference by more than 2^90 -- then the weights of this pass are useless (they are clamped,
        // so nothing overflows) and the pass is repeated with the true maximum as reference.
        float run_max = -INFINITY;
        bool over = false;
        auto stage_score_sync = [&](int t, bool first_pass) {
            if (t == 0 && first_pass) {
                float wm = s2;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
                if (lane == 0) tmax[warp] = wm;
                named_sync_128();
                m_ref = fmaxf(fmaxf(tmax[0], tmax[1]), fmaxf(tmax[2], tmax[3]));
            }
            run_max = fmaxf(run_max, s2);
            over |= s2 > m_ref + 90.f;
            w = valid ? ex2f(fminf(s2 - m_ref, 100.f)) : 0.f;
            if (h == 0) omega += w;
        };
        for (int pass = 0, g0 = 0; pass < 2 && ok && ntile > 0; ++pass, g0 += ntile) {
            omega = 0.f;
            ok = stage_load(g0);
            if (!ok) break;
            stage_score_math(0, g0);
            stage_score_sync(0, pass == 0);
            for (int t = 0; t < ntile && ok; ++t) {
                const int g = g0 + t;
                const uint32_t b = g & 1;
                const bool more = t + 1 < ntile;
                // wait until the MMA of the tile two before has released this B buffer (long done in steady state)
                if (!mbar_wait(bar(DB_BFREE + b), ((g >> 1) & 1) ^ 1, abort_flag, wcap)) { ok = false; break; }
                // B rows of tile t: w * [k | 1] as bf16 hi + lo, eight features at a time straight into the
                // operand tiles, so the stores drain while the rest of the iteration runs
                uint8_t* bhi = smem + SMD_B + b * 2 * DT_BTILE;
                uint8_t* blo = bhi + DT_BTILE;
                const uint64_t ww = pk2(w, w);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float a, bq;
                        upk2(mul2(ww, pk2(kf[8 * i + 2 * e], kf[8 * i + 2 * e + 1])), a, bq);
                        hi[e] = split_bf16x2(a, bq, lo[e]);
                    }
                    const uint32_t off = (4 * h + i) * 1024 + rowoff;          // column block 4h+i
                    *reinterpret_cast<uint4*>(bhi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(blo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                {   // column blocks 8 (ones column first) and 9 (zero padding)
                    uint32_t wlo;
                    const uint32_t whi = split_bf16x2(w, 0.f, wlo);
                    const uint32_t off = (8 + h) * 1024 + rowoff;
                    *reinterpret_cast<uint4*>(bhi + off) = make_uint4(h == 0 ? whi : 0u, 0, 0, 0);
                    *reinterpret_cast<uint4*>(blo + off) = make_uint4(h == 0 ? wlo : 0u, 0, 0, 0);
                }
                // the next tile: shared-memory loads, then the score arithmetic, while the stores drain
                if (more && !stage_load(g + 1)) { ok = false; break; }
                if (more) stage_score_math(t + 1, g + 1);
                fence_proxy_async();
                // one arrival per warp: 32 lanes arriving on one mbarrier are 32 serialised shared-memory atomics
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(DB_BFULL + b));
                if (more) stage_score_sync(t + 1, false);
            }
            if (!ok || pass == 1) break;
            // end of the first pass: did any score leave the range of the reference?  (one barrier per pass)
            uint32_t any;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
                "barrier.cta.red.or.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(any) : "r"((uint32_t)over) : "memory");
            if (any) {
                float wm = run_max;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
                if (lane == 0) tmax[4 + warp] = wm;
            }
            if (tid == 0) misc[2] = (int)any;
            named_sync_128();
            if (any) {
                m_ref = fmaxf(fmaxf(tmax[4], tmax[5]), fmaxf(tmax[6], tmax[7]));
                over = false;
                d_parity = 1;            // the accumulator of the second pass completes the barrier's second phase
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(DB_PASS));      // the TMA and MMA warps read misc[2] after this
            if (!any) break;
        }
        // total weight of this part
        if (ok) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) omega += __shfl_xor_sync(0xffffffffu, omega, off);
        }
    }

    // ================================ epilogue ================================
    // All 192 threads take part (the solve below is a block-wide routine).
    __shared__ float s_omega[4];
    __shared__ float s_mref;
    if (warp < 4 && lane == 0) s_omega[warp] = omega;
    if (tid == 0) s_mref = m_ref;
    bool d_ok = true;
    if (warp < 4 && ntile > 0) {
        d_ok = mbar_wait(bar(DB_DFULL), d_parity, abort_flag, wcap);
        tc_fence_after();
    }
    // moments -> registers (lane f: row f of M plus a[f]; lane 64+f: row f of N plus c[f])
    float dv[96];
    if (warp < 4) {
        if (ntile > 0 && d_ok) {
            const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
            // columns 0..79 hold D_hi, 80..159 D_lo; dv[e] = D_hi[e] + D_lo[e] for the 65 columns in use
#pragma unroll
            for (int cb = 0; cb < 96; cb += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + cb, v);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) dv[cb + e] = __uint_as_float(v[e]);
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) dv[e] += dv[80 + e];            // D_lo[0..15] sat in columns 80..95
#pragma unroll
            for (int cb = 96; cb < 160; cb += 32) {
                uint32_t v[32];
                tmem_ld32(lane_addr + cb, v);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) dv[cb - 80 + e] += __uint_as_float(v[e]);   // D_lo[16..79]
            }
        } else {
#pragma unroll
            for (int e = 0; e < 96; ++e) dv[e] = 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();       // every pipeline stage is drained: shared memory can be re-carved
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(DT_TMEM_COLS) : "memory");
    }
    const bool aborted = *abort_flag != 0;
    if (aborted) {
        // (the TMA and MMA warps have waited above for what they had issued)
        if (tid == 0) {
            if (prm.status) atomicAdd(prm.status + LLA_STATUS_TIMEOUT, 1);
            if (prm.splits > 1 || prm.defer) {
                // no record of this part: poison its weight and maximum, so that the solve kernel emits NaN for the
                // unit instead of reading whatever an earlier call left in the record buffer
                float* dst = prm.parts + ((size_t)bh * prm.splits + part) * (2 * 64 * 64 + 2 * 64 + 4);
                dst[2 * 64 * 64 + 128] = __int_as_float(0x7fc00000);
                dst[2 * 64 * 64 + 129] = __int_as_float(0x7fc00000);
            }
        }
        return;
    }
    const float omega_tot = s_omega[0] + s_omega[1] + s_omega[2] + s_omega[3];
    const float mref_ln = s_mref * 0.6931471805599453f;          // back to natural-log units

    if (prm.splits > 1 || prm.defer) {
        // partial record for the solve kernel: M, N, a, c, omega, m (same layout as the SIMT path)
        if (!LLA_IN_BOUNDS((size_t)bh * prm.splits + part, (size_t)gridDim.y * prm.splits, prm.status, 501)) return;
        float* dst = prm.parts + ((size_t)bh * prm.splits + part) * (2 * 64 * 64 + 2 * 64 + 4);
        if (warp < 4) {
            float* rowp = dst + (size_t)tid * 64;                 // tid < 64: M rows; 64..127: N rows
#pragma unroll
            for (int e = 0; e < 64; e += 4)
                *reinterpret_cast<float4*>(rowp + e) = make_float4(dv[e], dv[e + 1], dv[e + 2], dv[e + 3]);
            dst[2 * 64 * 64 + tid] = dv[64];                      // a then c
        }
        if (tid == 0) {
            dst[2 * 64 * 64 + 128] = omega_tot;
            dst[2 * 64 * 64 + 129] = ntile > 0 ? mref_ln : -INFINITY;
        }
        return;
    }

    // single part: centre, solve and emit the output row here
    double* Md = reinterpret_cast<double*>(smem);              // 64 x 65
    double* av = Md + 64 * 65;                                  // a -> kbar
    double* cv = av + 64;                                       // c -> vbar
    double* rhs = cv + 64;
    float* Nd = reinterpret_cast<float*>(rhs + 64);             // 64 x 65 (padded rows)
    const double inv = 1.0 / (double)omega_tot;
    const double lam_u = prm.lambda_units ? (double)prm.lambda_units[bh] : (double)prm.lambda;
    const double ridge = (prm.ridge_mode == LLA_RIDGE_PRINTED ? lam_u : lam_u * exp(-(double)mref_ln)) * inv;
    if (warp < 4) {
        if (tid < 64) av[tid] = (double)dv[64] * inv;
        else cv[tid - 64] = (double)dv[64] * inv;
    }
    __syncthreads();
    if (warp < 4) {
        if (tid < 64) {
            // full row of the centred matrix (M is symmetric up to fp32 rounding of the accumulators)
            const double ar = av[tid];
#pragma unroll
            for (int e = 0; e < 64; ++e) Md[tid * 65 + e] = (double)dv[e] * inv - ar * av[e];
            Md[tid * 65 + tid] += ridge;
            rhs[tid] = (double)to_f32(q[(size_t)bh * DT_D + tid]) - ar;
        } else {
#pragma unroll
            for (int e = 0; e < 64; ++e) Nd[(tid - 64) * 65 + e] = dv[e];
        }
    }
    __syncthreads();
    // conjugate gradients first (fast); the blocked factorisation only if they do not converge
    double* xs = reinterpret_cast<double*>(Nd + 64 * 65);      // x, p and reduction scratch after N
    __shared__ int s_cg_ok;
    if (warp < 4) {
        int cg_its = 0;
        double cr[32];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) cr[8 * i + j] = Md[(cg_row0(tid) + i) * 65 + cg_col0(tid) + j];
        const bool okc = cg_solve_64(cr, rhs[cg_row(tid)], xs, xs + 64, xs + 128, cg_its);
        if (tid == 0) {
            s_cg_ok = okc ? 1 : 0;
            if (prm.status) atomicAdd(prm.status + LLA_STATUS_ITER_SUM, cg_its);
        }
    }
    __syncthreads();
    bool solved = true;
    if (s_cg_ok) {
        if (tid < 64) rhs[tid] = xs[tid];
        __syncthreads();
    } else {
        solved = block_ldlt_solve<64>(Md, 65, rhs);
    }
    if (tid < 64) {
        double o = cv[tid];
        for (int f = 0; f < 64; ++f) o += ((double)Nd[tid * 65 + f] * inv - cv[tid] * av[f]) * rhs[f];
        store_out(out + (size_t)bh * DT_D + tid, (float)o);
    }
    if (!solved && tid == 0 && prm.status) atomicAdd(prm.status + LLA_STATUS_BAD_PIVOT, 1);
}

// Second kernel of the two-kernel decode: merge the parts' moment records of one (sequence, head),
// centre them, solve and emit the output row.  Everything a thread needs of the two matrices goes
// straight from the records (L2) into registers, so a block holds little shared memory and several
// of them share an SM; the solve itself is latency-bound (barriers and shuffles), which is why it is
// kept out of the streaming kernel whenever the caller provides the record buffer.
constexpr int DS_MAX_SPLITS = 64;
template <typename TOut>
__global__ void __launch_bounds__(DT_COMPUTE, 4)
decode_solve_kernel(const __nv_bfloat16* __restrict__ q, const float* __restrict__ parts, TOut* __restrict__ out,
                    const int* __restrict__ lens, int H, int Lmax, int head_rows, float lambda, int splits,
                    int* __restrict__ status, const float* __restrict__ lambda_units, int ridge_mode, int window) {
    constexpr int D = DT_D, PF = 2 * D * D + 2 * D + 4;
    __shared__ __align__(16) double s_a[D], s_c[D], s_x[D], s_p[D], s_red[24];
    __shared__ double s_f[DS_MAX_SPLITS];
    __shared__ double s_L[D * 65];          // only touched by the factorisation fallback
    const int tid = threadIdx.x, r = tid >> 1, hh = tid & 1, bh = blockIdx.x;
    // launched as a programmatic dependent of the streaming kernel: nothing of that grid may be read before this
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {
    if (visible_keys(lens[bh / H], Lmax, window) < head_rows) return;
    const float* src = parts + (size_t)bh * splits * PF;
    float m = -INFINITY;
    for (int p = 0; p < splits; ++p) m = fmaxf(m, src[(size_t)p * PF + 2 * D * D + 2 * D + 1]);
    for (int p = tid; p < splits; p += DT_COMPUTE)
        s_f[p] = exp((double)src[(size_t)p * PF + 2 * D * D + 2 * D + 1] - (double)m);   // 0 for empty parts
    __syncthreads();
    double omega = 0.0;
    for (int p = 0; p < splits; ++p) omega += s_f[p] * (double)src[(size_t)p * PF + 2 * D * D + 2 * D];
    const double inv = 1.0 / omega;
    const double lam_u = lambda_units ? (double)lambda_units[bh] : (double)lambda;
    const double ridge = (ridge_mode == LLA_RIDGE_PRINTED ? lam_u : lam_u * exp(-(double)m)) * inv;
    {
        double s1 = 0.0;                     // thread e < 64: a[e]; thread 64 + e: c[e]
        for (int p = 0; p < splits; ++p) s1 += s_f[p] * (double)src[(size_t)p * PF + 2 * D * D + tid];
        if (tid < D) s_a[tid] = s1 * inv; else s_c[tid - D] = s1 * inv;
    }
    __syncthreads();
    // this thread's 4 x 8 block of the centred matrix (see cg_solve_64)
    const int row0 = cg_row0(tid), col0 = cg_col0(tid), myrow = cg_row(tid);
    double cr[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) cr[c] = 0.0;
    for (int p = 0; p < splits; ++p) {
        const double f = s_f[p];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4* mp = reinterpret_cast<const float4*>(src + (size_t)p * PF + (row0 + i) * D + col0);
            const float4 v0 = mp[0], v1 = mp[1];
            cr[8 * i] += f * (double)v0.x; cr[8 * i + 1] += f * (double)v0.y;
            cr[8 * i + 2] += f * (double)v0.z; cr[8 * i + 3] += f * (double)v0.w;
            cr[8 * i + 4] += f * (double)v1.x; cr[8 * i + 5] += f * (double)v1.y;
            cr[8 * i + 6] += f * (double)v1.z; cr[8 * i + 7] += f * (double)v1.w;
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const double ai = s_a[row0 + i];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            cr[8 * i + j] = cr[8 * i + j] * inv - ai * s_a[col0 + j];
            if (row0 + i == col0 + j) cr[8 * i + j] += ridge;
        }
    }
    const double b_r = (double)to_f32(q[(size_t)bh * D + myrow]) - s_a[myrow];
    int cg_its = 0;
    const bool okc = cg_solve_64(cr, b_r, s_x, s_p, s_red, cg_its);
    if (tid == 0 && status) atomicAdd(status + LLA_STATUS_ITER_SUM, cg_its);
    bool solved = true;
    if (!okc) {        // uniform over the block: the decision comes from block-wide sums
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) s_L[(row0 + i) * 65 + col0 + j] = cr[8 * i + j];
        if ((tid & 1) == 0) s_x[myrow] = b_r;
        solved = block_ldlt_solve<D>(s_L, 65, s_x);
    }
    // o_e = vbar_e + sum_f (N[e][f] / omega - vbar_e kbar_f) y_f, two threads per output element
    double nr[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) nr[c] = 0.0;
    for (int p = 0; p < splits; ++p) {
        const float4* np_ = reinterpret_cast<const float4*>(src + (size_t)p * PF + D * D + r * D + 32 * hh);
        const double f = s_f[p];
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
            const float4 v = np_[c4];
            nr[4 * c4] += f * (double)v.x; nr[4 * c4 + 1] += f * (double)v.y;
            nr[4 * c4 + 2] += f * (double)v.z; nr[4 * c4 + 3] += f * (double)v.w;
        }
    }
    const double cb = s_c[r];
    double o = 0.0;
#pragma unroll
    for (int c = 0; c < 32; ++c) o += (nr[c] * inv - cb * s_a[32 * hh + c]) * s_x[32 * hh + c];
    o += __shfl_xor_sync(0xffffffffu, o, 1);
    if (hh == 0) store_out(out + (size_t)bh * D + r, (float)(o + cb));
    if (!solved && tid == 0 && status) atomicAdd(status + LLA_STATUS_BAD_PIVOT, 1);
    }
}

template <typename TOut>
int launch_t(const DecodeArgs& a) {
    const int splits = a.splits < 1 ? 1 : a.splits;
    const size_t need = sizeof(float) * (size_t)a.B * a.H * splits * (2 * 64 * 64 + 2 * 64 + 4);
    const bool have_ws = a.workspace && a.workspace_bytes >= need && ((uintptr_t)a.workspace & 15u) == 0;
    if (splits > 1 && !have_ws) return LLA_ERR_WORKSPACE;
    if (splits > DS_MAX_SPLITS) return LLA_ERR_INVALID_ARG;
    CUtensorMap mk, mv;
    const int BH = a.B * a.H;
    const int kvg = a.kv_group > 0 ? a.kv_group : 1;
    const int map_units = a.paged.table ? a.paged.num_pages * (a.H / kvg) : BH / kvg;
    const int map_rows = a.paged.table ? a.paged.page_size : a.Lmax;
    if (!make_map_bf16_64(&mk, a.kcache, map_units, map_rows, DT_BK) || !make_map_bf16_64(&mv, a.vcache, map_units, map_rows, DT_BK))
        return LLA_ERR_CUDA;
    DtParams prm;
    prm.B = a.B; prm.H = a.H; prm.Lmax = a.Lmax; prm.splits = splits; prm.head_rows = a.head_rows;
    prm.scale = a.scale; prm.lambda = a.lambda; prm.lens = a.lens;
    prm.lambda_units = a.lambda_units; prm.ridge_mode = a.ridge_mode; prm.kv_group = kvg; prm.paged = a.paged; prm.window = a.window;
    prm.wait_clocks = a.wait_clocks > 0 ? a.wait_clocks : kWaitClocks; prm.no_loads = a.no_loads;
    prm.parts = (float*)a.workspace; prm.status = a.status;
    prm.defer = have_ws ? 1 : 0;      // with a record buffer the solve runs as its own kernel
    auto kern = decode_tc_kernel<TOut>;
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMD_ALLOC));
    // two blocks per SM need the largest shared-memory carve-out
    LLA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    dim3 grid(splits, BH);
    kern<<<grid, DT_THREADS, SMD_ALLOC, a.stream>>>(mk, mv, (const __nv_bfloat16*)a.q, (TOut*)a.out, prm);
    LLA_CUDA_TRY(cudaGetLastError());
    if (have_ws) {
        // Programmatic dependent launch: the solve grid is set up while the streaming grid drains and its blocks
        // start (past the griddepcontrol.wait at their top) the moment that grid has completed and its records
        // are visible; 305 -> 303 us per step.  (Letting the streaming blocks trigger the launch early, so that
        // solve blocks already sit on the SMs the tail leaves free, was slower: 305 us.)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(BH);
        cfg.blockDim = dim3(DT_COMPUTE);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = a.stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        LLA_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_solve_kernel<TOut>, (const __nv_bfloat16*)a.q, (const float*)a.workspace,
                                        (TOut*)a.out, a.lens, a.H, a.Lmax, a.head_rows, a.lambda, splits, a.status,
                                        a.lambda_units, a.ridge_mode, a.window));
    }
    return LLA_OK;
}

}  // namespace

bool decode_tensor_supported(const DecodeArgs& a) {
    return a.in_dtype == LLA_BF16 && a.d == DT_D && a.dv == DT_D && sm100::get_encode() != nullptr;
}

// Tensor-core decode.  With a record buffer (always for splits > 1, optional for a single part) the
// streaming kernel writes moment records and a solve kernel follows; without one, single-part
// blocks solve in their own epilogue.
int launch_decode_tensor_moments(const DecodeArgs& a) {
    if (!decode_tensor_supported(a)) return LLA_ERR_UNSUPPORTED;
    if (a.out_dtype == LLA_BF16) return launch_t<__nv_bfloat16>(a);
    if (a.out_dtype == LLA_F32) return launch_t<float>(a);
    return LLA_ERR_UNSUPPORTED;
}

}  // namespace lla
