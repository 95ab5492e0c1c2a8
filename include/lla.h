/*
 * lla.h - C ABI of the B200 (sm_100a) Local Linear Attention library.
 *
 * One hot path: the causal LLA forward pass, its single-query decode variant, and the backward pass.
 * For every query i the pass forms kernel weights w_ij = exp(scale * q_i.k_j) over the
 * visible keys (j <= i when causal), the query-centred moments
 *     omega_i = sum_j w_ij,  mu_i = sum_j w_ij (k_j - q_i),
 *     Sigma_i = sum_j w_ij (k_j - q_i)(k_j - q_i)^T + lambda I        (Eq. "query_specific"),
 * solves Sigma_i rho_i = mu_i without ever storing Sigma_i (matrix-free conjugate gradients,
 * Section 3.1 / Algorithm 2; rows with very few visible keys are solved directly), and emits
 *     o_i = sum_j w_ij (1 - (k_j - q_i)^T rho_i) v_j / (omega_i - mu_i^T rho_i)   (Eq. "lla").
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers unless a comment says "host".  Tensors are
 *     contiguous, row-major, innermost index fastest, base address 16-byte aligned.
 *   - The caller owns every buffer.  The library reads inputs, writes outputs (outputs must
 *     not alias inputs), and keeps no pointer once the enqueued work has completed.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work
 *     is ordered after what `stream` holds at the call and before anything enqueued on it later; part
 *     of it (the directly-solved rows) may run on a library-owned side stream that is forked from and
 *     joined back to `stream` with events.  No entry point synchronises the device (the *_host forms
 *     synchronise `stream`).  Calls may come from several host threads.
 *   - Return value: an lla_status as int.  Argument errors are detected on the host before any
 *     launch.  Nothing throws or aborts.  Conditions that only the device can see (rows that hit
 *     the iteration cap, a failed pivot in a directly-solved row) are counted in the optional
 *     `device_status` words, readable after the caller synchronises the stream.
 *   - The library is CUDA only: there is no host fallback.  On a machine without a usable
 *     device every launch returns LLA_ERR_CUDA.
 *   - Supported head sizes: d = dv in {16, 64, 128}; other values return LLA_ERR_UNSUPPORTED.
 *   - lambda must be >= 0.  With lambda == 0 rows that see fewer than d+1 keys have a singular
 *     system; their output is unspecified (the paper's definition has no unique answer there).
 */
#ifndef LLA_H_
#define LLA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lla_status {
    LLA_OK = 0,
    LLA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, negative lambda, non-finite scale */
    LLA_ERR_UNSUPPORTED = 2, /* head size or dtype combination not compiled in */
    LLA_ERR_WORKSPACE = 3,   /* caller workspace missing or too small */
    LLA_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed */
    LLA_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (reported via device_status) */
} lla_status;

typedef enum lla_dtype { LLA_BF16 = 0, LLA_F32 = 1 } lla_dtype;

/* Implementation selector for lla_forward_ex. */
typedef enum lla_impl {
    LLA_IMPL_AUTO = 0,   /* tensor-core kernel where compiled for the shape, else SIMT */
    LLA_IMPL_SIMT = 1,   /* fp32 CUDA-core kernel (every supported shape and dtype) */
    LLA_IMPL_TENSOR = 2  /* tcgen05/TMEM kernel (bf16 inputs, d = dv = 64 or 128) */
} lla_impl;

/* How the ridge enters (lla_forward_params / lla_decode_params.ridge_mode).
 * DEFINITION: Sigma_i = sum_j exp(s_ij) z z^T + lambda I with the raw weights of Eq. "query_specific";
 *             computed with max-subtracted weights and the ridge lambda * exp(-m_i).
 * PRINTED:    Algorithm 1/2 as printed: lambda is added to the moments of the max-subtracted weights
 *             exp(s_ij - m_i) as it is, i.e. an effective ridge lambda * exp(m_i) in the raw frame. */
typedef enum lla_ridge_mode { LLA_RIDGE_DEFINITION = 0, LLA_RIDGE_PRINTED = 1 } lla_ridge_mode;

/* Row groups for lla_forward_params.phases. */
enum { LLA_PHASE_ALL = 0, LLA_PHASE_DIRECT = 1, LLA_PHASE_ITERATIVE = 2 };

/* Words of the optional device_status array (int[LLA_STATUS_WORDS], zeroed by the call). */
enum {
    LLA_STATUS_ROWS_AT_CAP = 0,  /* rows whose CG stopped at max_iters above the tolerance */
    LLA_STATUS_BAD_PIVOT = 1,    /* directly-solved rows whose Cholesky met a pivot <= 0 */
    LLA_STATUS_TIMEOUT = 2,      /* bounded waits that expired (0 in a healthy run) */
    LLA_STATUS_ITER_SUM = 3,     /* low 31 bits of the sum over CG rows of iterations executed */
    LLA_STATUS_BOUNDS = 4,       /* debug build only (liblla_debug.so): stores skipped because their index was out of range */
    LLA_STATUS_BOUNDS_SITE = 5,  /* debug build only: id of the first such store (0: none) */
    LLA_STATUS_WORDS = 8
};

/*
 * Causal LLA forward, bf16 in / bf16 out, fp32 accumulation (Section 3.2, matrix form and
 * Algorithm 1; solver per Algorithm 2).
 *   q, k : [B, H, n, d]  bf16      v : [B, H, n, dv] bf16      out : [B, H, n, dv] bf16
 *   scale  : multiplies q.k inside exp (the paper's 1/h); lambda : ridge, >= 0
 *   causal : nonzero -> row i sees keys 0..i (diagonal included); zero -> every row sees all n
 * Uses the default solver settings (see lla_forward_ex) and no caller workspace.
 */
int lla_forward(const void *q, const void *k, const void *v, void *out, int B, int H, int n, int d,
                int dv, float scale, float lambda, int causal, void *stream);

/* Same operation with fp32 inputs and fp32 output (fp32 arithmetic, tighter solver tolerance). */
int lla_forward_f32(const void *q, const void *k, const void *v, void *out, int B, int H, int n,
                    int d, int dv, float scale, float lambda, int causal, void *stream);

/*
 * Single-query decode over a KV cache: Eq. "lla" for one query per (sequence, head).  The paper
 * only names an inference kernel; the semantics are its definition at one row.
 *   q      : [B, H, d]                 bf16
 *   kcache : [B, H, Lmax, d]           bf16     vcache : [B, H, Lmax, dv] bf16
 *   lens   : [B] int32, DEVICE pointer, 1 <= lens[b] <= Lmax.  lens[b] counts the current token,
 *            whose key and value are already stored in the cache (this matches j <= i).
 *            A length outside [1, Lmax] is clamped into that range on the device.
 *   out    : [B, H, dv]                bf16
 */
int lla_decode(const void *q, const void *kcache, const void *vcache, const int *lens, void *out,
               int B, int H, int Lmax, int d, int dv, float scale, float lambda, void *stream);

/* Decode with fp32 caches, query and output. */
int lla_decode_f32(const void *q, const void *kcache, const void *vcache, const int *lens,
                   void *out, int B, int H, int Lmax, int d, int dv, float scale, float lambda,
                   void *stream);

/*
 * Full-control forward.  Zero-initialise the struct, then set fields; zero / NULL means default.
 *   in_dtype / out_dtype : lla_dtype of q,k,v and of out (bf16 inputs may write an fp32 output)
 *   max_iters : CG iteration cap per row (default 64; Algorithm 2's T)
 *   tol       : CG stops a row when |residual| <= tol * |right-hand side| (Algorithm 2's
 *               epsilon; default 1e-4 for bf16 inputs, 1e-6 for fp32 inputs)
 *   head_rows : rows that see fewer than this many keys are solved directly in fp64 from the
 *               explicit d x d system instead of by CG (0 = default: 1.5*d for bf16 inputs, 2*d for
 *               fp32 inputs; negative disables).  Those early systems are too ill-conditioned for fp32 CG.
 *   impl      : lla_impl
 *   phases    : which groups of rows to compute: 0 = all; LLA_PHASE_DIRECT = only the rows
 *               solved directly; LLA_PHASE_ITERATIVE = only the rows solved by CG (profiling aid:
 *               the other rows of `out` are left untouched)
 *   rho       : optional [B, H, n, d] fp32, the solutions Sigma_i^{-1} mu_i (Algorithm 1 keeps
 *               them for the backward pass)
 *   stats     : optional [B, H, n, 3] fp32: a shift m_i of the scaled scores, omega_i and
 *               delta_i = omega_i - mu_i^T rho_i, the last two for weights exp(score - m_i).  m_i is the row
 *               maximum in the directly-solved rows and in the CUDA-core kernel; the tensor-core kernel uses
 *               shift zero whenever every maximum of the row tile lies within 2^+-8 (Eq. "lla" does not depend on
 *               the shift; m_i + log omega_i and m_i + log delta_i are the shift-free quantities)
 *   iters     : optional [B, H, n] int32, CG iterations executed for the row (-1 for rows solved
 *               directly)
 *   device_status : optional int[LLA_STATUS_WORDS] on the device
 *   q_rows    : 0 (or n) for the plain forward; 0 < q_rows < n for a chunk of queries at the last
 *               q_rows positions against all n keys (see the field's comment below)
 *   lambda_rows : optional [B, H, n] fp32 on the device, one ridge per query row (the paper's
 *               per-token regularisation); when not NULL it replaces `lambda`
 *   ridge_mode : lla_ridge_mode (0 = the definition; 1 = Algorithm 1/2 as printed)
 *   workspace / workspace_bytes : device scratch of at least lla_forward_workspace_bytes(...)
 *               bytes, 256-byte aligned; may be NULL when that function returns 0
 */
typedef struct lla_forward_params {
    const void *q, *k, *v;
    void *out;
    int B, H, n, d, dv;
    int in_dtype, out_dtype;
    float scale, lambda;
    int causal;
    int max_iters;
    float tol;
    int head_rows;
    int impl;
    int phases;
    float *rho;
    float *stats;
    int *iters;
    int *device_status;
    void *workspace;
    size_t workspace_bytes;
    void *stream;
    const float *lambda_rows;   /* optional [B, H, n] fp32 on the device: one ridge per query row
                                   (per-token regularisation); replaces `lambda` when not NULL */
    int ridge_mode;             /* lla_ridge_mode */
    int q_rows;                 /* 0 or n: one query per key position.  0 < q_rows < n: prefill of the
                                   LAST q_rows positions against all n keys (a chunk appended to an
                                   existing cache): q, out, rho, stats, iters and lambda_rows then have
                                   q_rows rows per head; query row r sits at position n - q_rows + r and,
                                   when causal, sees keys 0 .. n - q_rows + r */
    int kv_heads;   /* 0 or H: every query head has its own k, v.  Otherwise H must be a multiple of kv_heads and
                       k, v are [B, kv_heads, n, d]: query head h reads key/value head h / (H / kv_heads)
                       (grouped-query sharing) */
    int window;     /* causal sliding window: 0 = a row sees every earlier position; W > 0 = only its last W
                       positions (itself included).  Needs causal != 0 and W >= the direct-row threshold
                       (head_rows; 1.5 d for bf16, 2 d for fp32 by default), else LLA_ERR_UNSUPPORTED */
    int cg_precise_iters; /* tensor-core kernel only.  The operands formed on the fly in a CG iteration (the search
                       direction P and the weighted products W .* (P K^T) of Algorithm 2) enter the tensor cores
                       as bf16 hi + lo pairs (16 mantissa bits, two products each) during the first
                       cg_precise_iters iterations of a row tile and as single fp16 values (11 bits, one product)
                       afterwards: an iteration's products are scaled by the size of its search direction,
                       which has fallen by then, so the coarser operands of the later iterations add less
                       error than the tolerance leaves.  The fp16 sweeps read an fp16 copy of k made by a
                       pre-pass into `workspace` (without room for it there, or with an entry of q or k beyond
                       6e4 in magnitude, every iteration uses pairs).  0 = default (1 iteration; 4 for the row
                       tiles within the first 8 d positions, which converge more slowly); n > 0 = n
                       iterations for every tile; LLA_CG_PRECISE_ALL = every iteration with pairs;
                       LLA_CG_PRECISE_NONE = fp16 from the first iteration on */
    long long q_strides[3], k_strides[3], v_strides[3], out_strides[3];
                          /* element strides (batch, head, row) of q [B, H, rows, d], k and v [B, kv heads, n, d] and
                       out; the innermost index always has stride 1.  All zero = contiguous in that order.  Any other
                       layout whose strides are positive multiples of 8 elements is read in place, e.g. tensors kept
                       as [B, n, H, d]: strides (n H d, d, H d).  The caller guarantees that the strides address
                       memory it owns and that rows of `out` do not overlap.  The optional per-row outputs (rho,
                       stats, iters) and lambda_rows stay contiguous [B, H, rows, ...].  Forward only */
    const unsigned char *block_mask; /* block sparsity (tensor-core kernel, causal, no window): device array
                       [ceil(q_rows / 128)][ceil(n / 64)] of bytes, row t for the query rows 128 t .. 128 t + 127,
                       entry c for the keys 64 c .. 64 c + 63; nonzero = the rows of that tile attend to the keys
                       of that block (those at or before their own position).  Always attended whatever the mask
                       says: the blocks of the first head_rows keys (so that every row's system stays well posed
                       and the directly-solved rows are untouched) and the blocks on the tile's diagonal.  NULL =
                       dense.  n <= 65536.  Shapes the tensor-core kernel does not cover: LLA_ERR_UNSUPPORTED */
    long long block_mask_stride;     /* bytes from one (batch, head) unit's mask to the next; 0 = one mask for all */
    int cg_precondition;  /* tensor-core kernel only.  0 = plain conjugate gradients as in Algorithm 2 (default).
                       1 = preconditioned with the inverse covariance of the visible keys: one d x d matrix per
                       block of 128 keys, built by a pre-pass into `workspace` (plain CG without room for it
                       there).  The system of a row is that covariance under the row's attention weights, so the
                       closer the weights are to uniform the fewer iterations remain -- about half on the
                       synthetic workloads; with sharply peaked weights it may not pay for its pre-pass.  The
                       solution is the same within the tolerance; a row on which the rounded matrix turns out
                       not to be positive definite carries on with plain CG */
    long long debug_wait_clocks; /* tensor-core kernel only: cap, in SM clocks, of every bounded wait on a barrier
                       inside the kernel (0 = default, about 2^31).  A wait that runs out makes its thread block
                       stop: the block waits for the copies and MMAs it has issued itself, releases its tensor
                       memory and returns without writing its rows; the call still returns LLA_OK and
                       device_status[LLA_STATUS_TIMEOUT] counts the blocks that gave up */
    int debug_flags;          /* LLA_DEBUG_NO_LOADS: the kernel's copy-issuing warp issues nothing, so that every
                       wait of every block expires with no copy or MMA in flight.  For testing the path above
                       without faulting or hanging anything; the output is left unwritten */
} lla_forward_params;
enum { LLA_CG_PRECISE_ALL = -1, LLA_CG_PRECISE_NONE = -2 };
enum { LLA_DEBUG_NO_LOADS = 1 };

int lla_forward_ex(const lla_forward_params *p);

/*
 * Full-control decode.  Fields as in lla_decode; additionally
 *   in_dtype / out_dtype : lla_dtype of q and the caches, and of out
 *   splits    : number of key-range parts each (sequence, head) is divided into so that long
 *               caches spread over more thread blocks (0 = chosen from B*H and Lmax; 1 = none).
 *               With splits > 1 partial moments go through `workspace`.
 *   lambda_units : optional [B, H] fp32 on the device, one ridge per (sequence, head)
 *   ridge_mode : lla_ridge_mode; LLA_RIDGE_PRINTED runs on the CUDA-core decode kernels
 *   workspace : device scratch of at least lla_decode_workspace_bytes(...) bytes, 256-byte
 *               aligned; required when the effective number of splits exceeds 1.  Unsplit, it
 *               is optional: given one, the tensor-core path (bf16, d = dv = 64) writes each
 *               (sequence, head)'s moments there and solves in a second kernel, which is faster
 *               than solving at the end of the streaming kernel; the result is the same.
 */
typedef struct lla_decode_params {
    const void *q, *kcache, *vcache;
    const int *lens;
    void *out;
    int B, H, Lmax, d, dv;
    int in_dtype, out_dtype;
    float scale, lambda;
    int splits;
    int impl;
    int *device_status;
    void *workspace;
    size_t workspace_bytes;
    void *stream;
    const float *lambda_units;  /* optional [B, H] fp32 on the device: one ridge per (sequence, head) */
    int ridge_mode;             /* lla_ridge_mode */
    int kv_heads;   /* as in lla_forward_params: the caches are [B, kv_heads, Lmax, d] */
    /* Paged cache (block_table != NULL): kcache, vcache are [num_pages, kv heads, page_size, d] and the keys
       j of sequence b are rows j % page_size of page block_table[b * max_pages + j / page_size]
       (int32 on the device, entries in [0, num_pages)).  page_size must be a multiple of 128 and
       max_pages * page_size >= Lmax; Lmax then only bounds lens.  bf16 and fp32 caches alike. */
    const int *block_table;
    int page_size, max_pages, num_pages;
    int window;     /* sliding window: 0 = the query sees all lens[b] cached keys; W > 0 = only the last
                       min(W, lens[b]) of them (positions lens[b] - W .. lens[b] - 1).  Not with a paged cache */
    long long debug_wait_clocks; /* as in lla_forward_params, for the tensor-core streaming kernel (bf16, d = 64) */
    int debug_flags;             /* LLA_DEBUG_NO_LOADS: its copy-issuing warp issues nothing, every bounded wait expires
                                    with nothing in flight, device_status[LLA_STATUS_TIMEOUT] counts the blocks and
                                    their units' outputs are NaN (the record of a block that gave up is poisoned) */
} lla_decode_params;

int lla_decode_ex(const lla_decode_params *p);

/*
 * Host-buffer convenience forms of the two operations above (same mathematics, Eq. "lla").
 * q, k, v, lens and out are HOST pointers (pinned memory gives the fastest copies; pageable
 * memory works).  The call allocates device buffers from the stream-ordered pool, copies the
 * inputs up, runs the device path on `stream`, copies the result back and SYNCHRONISES the
 * stream before returning, so `out` is valid on return.  dtypes are lla_dtype values.
 * lla_forward_host cuts larger problems into four chunks of (batch, head) units whose upload,
 * kernels and download run on library-owned streams, so copies and kernels overlap (with pinned
 * buffers); `stream` is joined with them before the call returns.
 * lla_decode_host reads lens[] on the host and uploads only the first lens[b] rows of every
 * (sequence, head) cache.
 * Side effect on the process: the entry points that take scratch from the pool (these two, lla_forward and
 * lla_decode) set the release threshold of the current device's DEFAULT stream-ordered memory pool to
 * "keep everything", once per device, so that repeated calls do not return their scratch to the driver.
 * A host program that trims that pool itself should use the _ex forms with its own workspace instead.
 */
int lla_forward_host(const void *q, const void *k, const void *v, void *out, int B, int H, int n,
                     int d, int dv, int in_dtype, int out_dtype, float scale, float lambda,
                     int causal, void *stream);
int lla_decode_host(const void *q, const void *kcache, const void *vcache, const int *lens,
                    void *out, int B, int H, int Lmax, int d, int dv, int in_dtype, int out_dtype,
                    float scale, float lambda, void *stream);

/*
 * Decode for callers that must not allocate.  (The paper has no counterpart; this is a packaging
 * variant of the split-key decode, same arithmetic as lla_decode_ex with `splits` parts.)
 *
 * Who needs it: code that runs where the CUDA allocator is off limits - inside a serving loop
 * whose memory is fully pre-planned, under a framework that forbids cudaMalloc after start-up
 * (a synchronising allocation would stall every stream of the process), or in a plug-in that is
 * handed device buffers but owns no allocator.  Such callers cannot provide the partial-moment
 * workspace that a split decode needs, and the library may not allocate it for them either.
 *
 * Instead the partial moments go to a fixed array of LLA_NOALLOC_SCRATCH_BYTES that is part of the
 * library image: every GPU that loads the library holds those bytes until the library is unloaded.
 * The call performs no cudaMalloc, cudaFree or other allocating call.  Its first use on a device
 * looks up the array's device address (with that device current); make that first call outside
 * any stream capture.
 *
 * Arguments are those of lla_decode plus the dtypes and `splits` (0 = the default of
 * lla_decode_default_splits; 1 = no split, which uses the array only if the records fit).  All tensor pointers are
 * device pointers owned by the caller.
 * Errors: LLA_ERR_WORKSPACE if an explicit `splits` > 1 needs more than the fixed array holds
 * (lla_decode_workspace_bytes(...) > LLA_NOALLOC_SCRATCH_BYTES): use fewer splits or lla_decode_ex
 * with a caller workspace.  With splits = 0 a default split count that does not fit runs unsplit instead.
 * Other codes as for lla_decode_ex.  The array's device address is looked up once per device and kept for
 * the life of the process: after cudaDeviceReset on that device the entry point must not be used again.
 * Sharing: all calls on a device use the same array.  Each call overwrites every record it later
 * reads, so nothing needs clearing between calls, but two calls whose kernels may run at the same
 * time (different streams, or different host threads) race on it: serialise them.
 */
#define LLA_NOALLOC_SCRATCH_BYTES (64u << 20)
int lla_decode_noalloc(const void *q, const void *kcache, const void *vcache, const int *lens,
                       void *out, int B, int H, int Lmax, int d, int dv, int in_dtype,
                       int out_dtype, float scale, float lambda, int splits, void *stream);

/* Scratch bytes lla_forward_ex can use for this problem (0 when none).  Only the d = 128 tensor-core
 * kernel has any (2 x SM count x 192 KiB: per-SM slots for the CG row vectors; the call queries the
 * current device's SM count).  It is optional: given a workspace of that size the call allocates
 * nothing (two calls that may run at the same time need separate workspaces); without one the
 * library keeps its own buffer per GPU, allocated with cudaMalloc by the first such call and shared
 * safely by all later ones (blocks address it by SM id and one block fills an SM). */
size_t lla_forward_workspace_bytes(int B, int H, int n, int d, int dv, int in_dtype, int impl);

/* Scratch bytes lla_decode_ex uses for this problem and split count: required when splits > 1,
 * optional (see lla_decode_params.workspace; 0 where it would not be used) when splits <= 1. */
size_t lla_decode_workspace_bytes(int B, int H, int Lmax, int d, int dv, int in_dtype, int splits);

/* Number of key-range parts lla_decode / lla_decode_ex(splits = 0) would use. */
int lla_decode_default_splits(int B, int H, int Lmax);

/*
 * Backward pass (the paper's backward appendix): gradients of a scalar loss L with respect to Q, K and
 * V, given g_i = dL/do_i and the tensors the forward saved (Section 3.2 keeps R and delta next to the
 * output for this purpose).  Causal, ridge as in the definition (LLA_RIDGE_DEFINITION), one scalar lambda,
 * q_rows = n.  Supported: bf16 q, k, v with d = dv in {64, 128}; anything else is LLA_ERR_UNSUPPORTED.
 *
 * Per query row the appendix's quantities are gamma_ij = g_i . v_j, one further linear solve with the
 * row's Sigma_i (its u_i; the forward's conjugate-gradient kernel is run on it, rows that see fewer than
 * head_rows keys are solved directly in fp64 like in the forward), and then
 *     Delta_V = S^T G,  Delta_K = Delta_W^K + Delta_Z^K,  Delta_Q = Delta_W^Q + Delta_Z^Q.
 *
 *   q, k, v   : [B, H, n, d] bf16 on the device, as given to the forward
 *   out       : [B, H, n, d] the forward's output, out_dtype (LLA_BF16 or LLA_F32).  Only g_i . o_i is
 *               taken from it; a bf16 `out` limits the accuracy of dq and dk to its rounding
 *   dout      : [B, H, n, d] g, dout_dtype (LLA_BF16 or LLA_F32)
 *   rho, stats: [B, H, n, d] and [B, H, n, 3] fp32, written by lla_forward_ex for the same inputs,
 *               scale, lambda, head_rows and window (a causal forward with q_rows = n and the ridge of the
 *               definition; the call cannot tell and would return the gradient of that forward)
 *   dq, dk, dv: [B, H, n, d] fp32 on the device, overwritten
 *   max_iters, tol, head_rows : as in lla_forward_params (0 = defaults)
 *   device_status : optional int[LLA_STATUS_WORDS], zeroed by the call
 *   workspace / workspace_bytes : device scratch of at least lla_backward_workspace_bytes(B, H, n, d)
 *               bytes, 256-byte aligned (required; LLA_ERR_WORKSPACE otherwise)
 * All pointers 16-byte aligned; no output may alias an input.  Work is enqueued on `stream`; the call
 * does not synchronise and keeps no pointer.
 * Reproducibility: dq is bit-identical from run to run (each query tile owns its rows and stores them; with
 * impl = LLA_IMPL_SIMT the key tiles add their shares atomically instead and it is not).  So are the rows of dk and
 * dv from position 128 * ceil((head_rows - 1) / 128) on, unless heads are grouped: a key tile owns and stores them.
 * The earlier rows also receive the directly-solved query rows' shares, and with grouped heads every row receives
 * one share per query head of its group; those are summed with fp32 atomic adds, whose order varies, and agree
 * between runs to rounding (about 1e-6 relative), not bit for bit.
 */
typedef struct lla_backward_params {
    const void *q, *k, *v, *out, *dout;
    const float *rho, *stats;
    float *dq, *dk, *dv;
    int B, H, n, d;
    int out_dtype, dout_dtype;
    float scale, lambda;
    int max_iters;
    float tol;
    int head_rows;
    int *device_status;
    void *workspace;
    size_t workspace_bytes;
    void *stream;
    int *iters;   /* optional [B, H, n] on the device: CG iterations of the extra solve per row (rows that are
                     solved directly are left untouched) */
    float *dlambda; /* optional [B, H, n] fp32 on the device: dL/d(lambda_i), the derivative with respect to a
                       ridge of its own per query row (the paper's learnable regularisation), evaluated at
                       lambda; their sum over i is the derivative with respect to the scalar */
    int impl;     /* LLA_IMPL_AUTO: moments and pair kernels on the tensor cores; LLA_IMPL_SIMT: on the CUDA cores */
    int kv_heads; /* as in lla_forward_params: k, v, dk, dv are [B, kv_heads, n, d]; a key/value head's gradient
                     sums over the query heads that read it */
    int window;   /* as in lla_forward_params: the forward being differentiated ran with this causal sliding window
                     (0: none).  At least head_rows, and not with impl = LLA_IMPL_SIMT: LLA_ERR_UNSUPPORTED otherwise */
    int cg_precondition; /* as in lla_forward_params: 1 = the extra solve runs the preconditioned conjugate gradients
                     (about half the iterations; same result within the tolerance) */
    const unsigned char *block_mask; /* as in lla_forward_params: the forward being differentiated ran with this block
                     mask (same layout, same always-attended blocks; NULL = dense).  Not with a window, n > 65536 or
                     impl = LLA_IMPL_SIMT: LLA_ERR_UNSUPPORTED */
    long long block_mask_stride;
    int q_rows;   /* as in lla_forward_params: the forward being differentiated had only the queries of the last q_rows
                     positions (0 = n); q, out, dout, rho, stats, dq, iters and dlambda are then [B, H, q_rows, ..],
                     k, v, dk, dv keep n rows.  Not with a block mask or impl = LLA_IMPL_SIMT: LLA_ERR_UNSUPPORTED */
    long long debug_wait_clocks; /* as in lla_forward_params, for the solve and the tensor-core kernels of this pass */
    int debug_flags;             /* LLA_DEBUG_NO_LOADS: their copy-issuing warps issue nothing, every bounded wait
                                    expires with nothing in flight, the blocks leave without results and
                                    device_status[LLA_STATUS_TIMEOUT] counts them; the call still returns LLA_OK */
} lla_backward_params;

int lla_backward_ex(const lla_backward_params *p);
size_t lla_backward_workspace_bytes(int B, int H, int n, int d);

/* Static, NUL-terminated description of a status code. */
const char *lla_status_string(int status);

/* Library version: major*10000 + minor*100 + patch. */
int lla_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LLA_H_ */
