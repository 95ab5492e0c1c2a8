// C-ABI entry points: argument validation, defaults, dispatch.  See include/lla.h for the contract.
#include <math.h>

#include <mutex>

#include "lla_common.cuh"

namespace {

using lla::DecodeArgs;
using lla::ForwardArgs;
using lla::BackwardArgs;

// Side stream on which the directly-solved rows run next to the iterative kernel (fork/join with
// events, so the caller's stream semantics are unchanged).  One per device, created on first use.
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool ok = false;
    // held while a call enqueues its fork / side work / join: a wait captures the event's latest record, so two
    // host threads interleaving their records on the shared events would wait on each other's points
    std::mutex use;
};
SideStream* side_stream() {
    static std::mutex mu;
    static SideStream per_dev[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    SideStream& s = per_dev[dev];
    if (!s.ok) {
        if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        s.ok = true;
    }
    return &s;
}

// Worker streams of the host-buffer forward: the (batch, head) units are cut into a few chunks and
// each chunk's upload, kernels and download run on their own stream, so the copies of one chunk
// overlap the kernels of another.
constexpr int kHostChunks = 4;
struct HostPipe {
    cudaStream_t stream[kHostChunks] = {};
    cudaEvent_t ready = nullptr, done[kHostChunks] = {};
    bool ok = false;
    // held for a whole call: the events and worker streams are shared by every caller on the device, and a wait
    // takes an event's latest record, so two host threads must not interleave their record/wait sequences
    std::mutex use;
};
HostPipe* host_pipe() {
    static std::mutex mu;
    static HostPipe per_dev[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    HostPipe& h = per_dev[dev];
    if (!h.ok) {
        if (cudaEventCreateWithFlags(&h.ready, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        for (int c = 0; c < kHostChunks; ++c) {
            if (cudaStreamCreateWithFlags(&h.stream[c], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&h.done[c], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        h.ok = true;
    }
    return &h;
}

bool head_size_ok(int d, int dv) { return d == dv && (d == 16 || d == 64 || d == 128); }

int check_forward(const lla_forward_params* p) {
    if (!p) return LLA_ERR_INVALID_ARG;
    if (!p->q || !p->k || !p->v || !p->out) return LLA_ERR_INVALID_ARG;
    if (p->B < 1 || p->H < 1 || p->n < 1 || p->d < 1 || p->dv < 1) return LLA_ERR_INVALID_ARG;
    if (!(p->lambda >= 0.f) || !isfinite(p->lambda) || !isfinite(p->scale)) return LLA_ERR_INVALID_ARG;
    if (p->ridge_mode != LLA_RIDGE_DEFINITION && p->ridge_mode != LLA_RIDGE_PRINTED) return LLA_ERR_INVALID_ARG;
    if (p->q_rows < 0 || p->q_rows > p->n) return LLA_ERR_INVALID_ARG;
    if (p->kv_heads < 0 || (p->kv_heads > 0 && p->H % p->kv_heads != 0)) return LLA_ERR_INVALID_ARG;
    if (p->max_iters < 0 || p->tol < 0.f || !isfinite(p->tol)) return LLA_ERR_INVALID_ARG;
    if (p->cg_precondition < 0 || p->cg_precondition > 1) return LLA_ERR_INVALID_ARG;
    for (const long long* st : {p->q_strides, p->k_strides, p->v_strides, p->out_strides}) {
        const bool set = st[0] || st[1] || st[2];
        // given strides: positive, and multiples of 8 elements so that every row starts on a 16-byte boundary
        // (vector loads, TMA); the innermost index always has stride 1
        if (set && (st[0] <= 0 || st[1] <= 0 || st[2] <= 0 || (st[0] | st[1] | st[2]) % 8 != 0)) return LLA_ERR_INVALID_ARG;
    }
    if (p->debug_wait_clocks < 0 || (p->debug_flags & ~LLA_DEBUG_NO_LOADS)) return LLA_ERR_INVALID_ARG;
    if ((long long)p->B * p->H > 65535 || (p->n + 127) / 128 > 65535) return LLA_ERR_UNSUPPORTED;
    if (!head_size_ok(p->d, p->dv)) return LLA_ERR_UNSUPPORTED;
    const bool dt_ok = (p->in_dtype == LLA_BF16 && (p->out_dtype == LLA_BF16 || p->out_dtype == LLA_F32)) ||
                       (p->in_dtype == LLA_F32 && p->out_dtype == LLA_F32);
    if (!dt_ok) return LLA_ERR_UNSUPPORTED;
    if (p->impl != LLA_IMPL_AUTO && p->impl != LLA_IMPL_SIMT && p->impl != LLA_IMPL_TENSOR)
        return LLA_ERR_INVALID_ARG;
    if (p->phases < LLA_PHASE_ALL || p->phases > LLA_PHASE_ITERATIVE) return LLA_ERR_INVALID_ARG;
    const uintptr_t align = (uintptr_t)p->q | (uintptr_t)p->k | (uintptr_t)p->v | (uintptr_t)p->out;
    if (align & 15u) return LLA_ERR_INVALID_ARG;
    return LLA_OK;
}

ForwardArgs to_args(const lla_forward_params* p) {
    ForwardArgs a;
    a.q = p->q; a.k = p->k; a.v = p->v; a.out = p->out;
    a.B = p->B; a.H = p->H; a.n = p->n; a.d = p->d; a.dv = p->dv;
    a.in_dtype = p->in_dtype; a.out_dtype = p->out_dtype;
    a.scale = p->scale; a.lambda = p->lambda; a.causal = p->causal ? 1 : 0;
    a.max_iters = p->max_iters > 0 ? p->max_iters : 64;
    a.tol = p->tol > 0.f ? p->tol : (p->in_dtype == LLA_F32 ? 1e-6f : 1e-4f);
    a.head_rows = p->head_rows == 0 ? (p->in_dtype == LLA_F32 ? 2 * p->d : p->d + p->d / 2)
                                   : (p->head_rows < 0 ? 0 : p->head_rows);
    a.rho = p->rho; a.stats = p->stats; a.iters = p->iters; a.status = p->device_status;
    a.workspace = p->workspace; a.workspace_bytes = p->workspace_bytes;
    a.stream = (cudaStream_t)p->stream;
    a.lambda_rows = p->lambda_rows;
    a.ridge_mode = p->ridge_mode;
    a.nq = p->q_rows > 0 ? p->q_rows : p->n;
    a.kv_group = p->kv_heads > 0 ? p->H / p->kv_heads : 1;
    a.window = p->window;
    a.wait_clocks = p->debug_wait_clocks;
    a.block_mask = p->block_mask; a.block_mask_stride = p->block_mask_stride;
    // layouts: all-zero strides mean contiguous [B, heads, rows, width]
    a.set_contiguous();
    auto take = [](lla::Strides& dst, const long long* src) {
        if (src[0] || src[1] || src[2]) dst = lla::Strides{src[0], src[1], src[2]};
    };
    take(a.sq, p->q_strides); take(a.sk, p->k_strides); take(a.sv, p->v_strides); take(a.so, p->out_strides);
    a.precondition = p->cg_precondition > 0 ? 1 : 0;
    a.no_loads = (p->debug_flags & LLA_DEBUG_NO_LOADS) ? 1 : 0;
    if (p->cg_precise_iters != 0) {
        a.precise_iters = p->cg_precise_iters == LLA_CG_PRECISE_NONE ? 0 : p->cg_precise_iters < 0 ? (1 << 30) : p->cg_precise_iters;
        a.precise_iters_early = a.precise_iters;
    }
    return a;
}

int check_decode(const lla_decode_params* p) {
    if (!p) return LLA_ERR_INVALID_ARG;
    if (!p->q || !p->kcache || !p->vcache || !p->lens || !p->out) return LLA_ERR_INVALID_ARG;
    if (p->B < 1 || p->H < 1 || p->Lmax < 1 || p->d < 1 || p->dv < 1 || p->splits < 0) return LLA_ERR_INVALID_ARG;
    if (p->impl != LLA_IMPL_AUTO && p->impl != LLA_IMPL_SIMT && p->impl != LLA_IMPL_TENSOR) return LLA_ERR_INVALID_ARG;
    if (!(p->lambda >= 0.f) || !isfinite(p->lambda) || !isfinite(p->scale)) return LLA_ERR_INVALID_ARG;
    if (p->ridge_mode != LLA_RIDGE_DEFINITION && p->ridge_mode != LLA_RIDGE_PRINTED) return LLA_ERR_INVALID_ARG;
    if ((long long)p->B * p->H > 65535) return LLA_ERR_UNSUPPORTED;
    if (!head_size_ok(p->d, p->dv)) return LLA_ERR_UNSUPPORTED;
    const bool dt_ok = (p->in_dtype == LLA_BF16 && (p->out_dtype == LLA_BF16 || p->out_dtype == LLA_F32)) ||
                       (p->in_dtype == LLA_F32 && p->out_dtype == LLA_F32);
    if (!dt_ok) return LLA_ERR_UNSUPPORTED;
    const uintptr_t align = (uintptr_t)p->q | (uintptr_t)p->kcache | (uintptr_t)p->vcache | (uintptr_t)p->out;
    if (align & 15u) return LLA_ERR_INVALID_ARG;
    return LLA_OK;
}

void keep_pool_memory() {
    // Let the current device's default stream-ordered pool keep freed blocks, so that repeated calls of the
    // entry points that take their scratch from it do not go back to the driver every time.  Once per device.
    // (A process-wide setting of that pool: include/lla.h says so.)
    static std::once_flag once[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    std::call_once(once[dev], [dev]() {
        cudaMemPool_t pool;
        if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess) {
            unsigned long long keep = ~0ull;
            cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        }
    });
}

}  // namespace

extern "C" {

int lla_forward_ex(const lla_forward_params* p) {
    const int rc = check_forward(p);
    if (rc != LLA_OK) return rc;
    ForwardArgs a = to_args(p);
    if (a.window < 0) return LLA_ERR_INVALID_ARG;
    if (a.window > 0 && (!a.causal || a.window < a.head_rows)) return LLA_ERR_UNSUPPORTED;
    const bool tensor_ok = lla::forward_tensor_supported(a);
    if (p->impl == LLA_IMPL_TENSOR && !tensor_ok) return LLA_ERR_UNSUPPORTED;
    const bool use_tensor = tensor_ok && p->impl != LLA_IMPL_SIMT;
    if (p->block_mask && (!use_tensor || !a.causal || a.window > 0 || a.n > 65536 || p->block_mask_stride < 0)) return LLA_ERR_UNSUPPORTED;
    // the forward workspace is optional (see lla_forward_workspace_bytes); a misaligned one is an error
    if (a.workspace && a.workspace_bytes > 0 && ((uintptr_t)a.workspace & 255u)) return LLA_ERR_WORKSPACE;
    (void)use_tensor;
    if (a.status) LLA_CUDA_TRY(cudaMemsetAsync(a.status, 0, sizeof(int) * LLA_STATUS_WORDS, a.stream));
    // The two row groups write disjoint rows of `out`; when both run, the direct rows go to a side
    // stream so they fill the SMs the iterative kernel's last wave leaves idle.
    // (the pre-pass of the tensor-core kernel goes first so that the fork below comes after it: the direct rows
    // then start beside the iterative kernel, not ahead of it, and fill the SMs its last wave leaves idle)
    if (use_tensor && p->phases != LLA_PHASE_DIRECT) {
        const int rc_pre = lla::forward_tensor_prepass(a);
        if (rc_pre != LLA_OK) return rc_pre;
    }
    const bool both = p->phases == LLA_PHASE_ALL && lla::head_rows_count(a) > 0;
    SideStream* side = both ? side_stream() : nullptr;
    if (side) {
        std::lock_guard<std::mutex> lock(side->use);
        LLA_CUDA_TRY(cudaEventRecord(side->fork, a.stream));
        LLA_CUDA_TRY(cudaStreamWaitEvent(side->stream, side->fork, 0));
        const int rc_main = use_tensor ? lla::launch_forward_tensor(a) : lla::launch_forward_simt(a);
        ForwardArgs h = a;
        h.stream = side->stream;
        const int rc_head = lla::launch_head_rows(h);
        LLA_CUDA_TRY(cudaEventRecord(side->join, side->stream));
        LLA_CUDA_TRY(cudaStreamWaitEvent(a.stream, side->join, 0));
        return rc_main != LLA_OK ? rc_main : rc_head;
    }
    if (p->phases != LLA_PHASE_ITERATIVE) {
        const int st = lla::launch_head_rows(a);
        if (st != LLA_OK) return st;
    }
    if (p->phases == LLA_PHASE_DIRECT) return LLA_OK;
    return use_tensor ? lla::launch_forward_tensor(a) : lla::launch_forward_simt(a);
}

int lla_forward(const void* q, const void* k, const void* v, void* out, int B, int H, int n, int d, int dv,
                float scale, float lambda, int causal, void* stream) {
    lla_forward_params p = {};
    p.q = q; p.k = k; p.v = v; p.out = out;
    p.B = B; p.H = H; p.n = n; p.d = d; p.dv = dv;
    p.in_dtype = LLA_BF16; p.out_dtype = LLA_BF16;
    p.scale = scale; p.lambda = lambda; p.causal = causal;
    p.stream = stream;
    // scratch from the stream-ordered pool (kept warm between calls); without it the call still works
    // (see lla_forward_workspace_bytes)
    const size_t ws = lla_forward_workspace_bytes(B, H, n, d, dv, LLA_BF16, LLA_IMPL_AUTO);
    void* scratch = nullptr;
    if (ws > 0 && check_forward(&p) == LLA_OK) {
        keep_pool_memory();
        if (cudaMallocAsync(&scratch, ws, (cudaStream_t)stream) != cudaSuccess) {
            (void)cudaGetLastError();
            scratch = nullptr;
        }
    }
    p.workspace = scratch;
    p.workspace_bytes = scratch ? ws : 0;
    const int rc = lla_forward_ex(&p);
    if (scratch) (void)cudaFreeAsync(scratch, (cudaStream_t)stream);
    return rc;
}

int lla_forward_f32(const void* q, const void* k, const void* v, void* out, int B, int H, int n, int d,
                    int dv, float scale, float lambda, int causal, void* stream) {
    lla_forward_params p = {};
    p.q = q; p.k = k; p.v = v; p.out = out;
    p.B = B; p.H = H; p.n = n; p.d = d; p.dv = dv;
    p.in_dtype = LLA_F32; p.out_dtype = LLA_F32;
    p.scale = scale; p.lambda = lambda; p.causal = causal;
    p.stream = stream;
    return lla_forward_ex(&p);
}

int lla_decode_default_splits(int B, int H, int Lmax) {
    // enough thread blocks to fill 148 SMs twice over, but no part shorter than 512 keys
    const long long bh = (long long)B * H;
    if (bh <= 0 || Lmax <= 0) return 1;
    long long s = (2 * 148 + bh - 1) / bh;
    const long long cap = Lmax / 512 > 1 ? Lmax / 512 : 1;
    if (s > cap) s = cap;
    if (s > 32) s = 32;
    return s < 1 ? 1 : (int)s;
}

int lla_decode_ex(const lla_decode_params* p) {
    const int rc = check_decode(p);
    if (rc != LLA_OK) return rc;
    DecodeArgs a;
    a.q = p->q; a.kcache = p->kcache; a.vcache = p->vcache; a.lens = p->lens; a.out = p->out;
    a.B = p->B; a.H = p->H; a.Lmax = p->Lmax; a.d = p->d; a.dv = p->dv;
    a.in_dtype = p->in_dtype; a.out_dtype = p->out_dtype;
    a.scale = p->scale; a.lambda = p->lambda;
    a.splits = p->splits > 0 ? p->splits : lla_decode_default_splits(p->B, p->H, p->Lmax);
    if (p->splits == 0 && a.splits > 1) {
        // default split count, but the caller gave no (or too small a) workspace: run unsplit
        const size_t need = lla::decode_workspace_bytes(a.B, a.H, a.d, a.dv, a.splits);
        if (!p->workspace || p->workspace_bytes < need) a.splits = 1;
    }
    if (a.splits > 1 && ((uintptr_t)p->workspace & 255u)) return LLA_ERR_WORKSPACE;
    a.head_rows = 2 * p->d;
    a.impl = p->impl;
    a.status = p->device_status;
    a.workspace = p->workspace; a.workspace_bytes = p->workspace_bytes;
    a.stream = (cudaStream_t)p->stream;
    a.lambda_units = p->lambda_units;
    a.ridge_mode = p->ridge_mode;
    if (p->kv_heads < 0 || (p->kv_heads > 0 && p->H % p->kv_heads != 0)) return LLA_ERR_INVALID_ARG;
    a.kv_group = p->kv_heads > 0 ? p->H / p->kv_heads : 1;
    if (p->block_table) {
        if (p->page_size < 128 || p->page_size % 128 != 0 || p->max_pages < 1 || p->num_pages < 1 ||
            (long long)p->max_pages * p->page_size < p->Lmax)
            return LLA_ERR_INVALID_ARG;
        a.paged = lla::PagedKv{p->block_table, p->page_size, p->max_pages, p->num_pages};
    }
    if (p->window < 0 || (p->window > 0 && p->block_table)) return LLA_ERR_INVALID_ARG;
    a.window = p->window;
    if (p->debug_wait_clocks < 0 || (p->debug_flags & ~LLA_DEBUG_NO_LOADS)) return LLA_ERR_INVALID_ARG;
    a.wait_clocks = p->debug_wait_clocks;
    a.no_loads = (p->debug_flags & LLA_DEBUG_NO_LOADS) ? 1 : 0;
    if (a.status) LLA_CUDA_TRY(cudaMemsetAsync(a.status, 0, sizeof(int) * LLA_STATUS_WORDS, a.stream));
    // The units with short caches go to the direct kernel, which writes rows of `out` nobody else writes and
    // returns at once for every other unit: it runs on the side stream beside the streaming kernel instead of
    // behind the solve (its launch alone is 2-3 us of a 300 us step).
    SideStream* side = side_stream();
    if (side) {
        std::lock_guard<std::mutex> lock(side->use);
        LLA_CUDA_TRY(cudaEventRecord(side->fork, a.stream));
        LLA_CUDA_TRY(cudaStreamWaitEvent(side->stream, side->fork, 0));
        DecodeArgs h = a;
        h.stream = side->stream;
        const int rc_head = lla::launch_head_rows_decode(h);
        LLA_CUDA_TRY(cudaEventRecord(side->join, side->stream));
        const int st = lla::launch_decode(a);
        LLA_CUDA_TRY(cudaStreamWaitEvent(a.stream, side->join, 0));
        return st != LLA_OK ? st : rc_head;
    }
    const int st = lla::launch_decode(a);
    if (st != LLA_OK) return st;
    return lla::launch_head_rows_decode(a);
}

int lla_decode(const void* q, const void* kcache, const void* vcache, const int* lens, void* out, int B,
               int H, int Lmax, int d, int dv, float scale, float lambda, void* stream) {
    lla_decode_params p = {};
    p.q = q; p.kcache = kcache; p.vcache = vcache; p.lens = lens; p.out = out;
    p.B = B; p.H = H; p.Lmax = Lmax; p.d = d; p.dv = dv;
    p.in_dtype = LLA_BF16; p.out_dtype = LLA_BF16;
    p.scale = scale; p.lambda = lambda;
    p.stream = stream;
    // scratch for the moment records comes from the stream-ordered pool (kept warm between calls)
    p.splits = 1;
    const size_t ws = lla_decode_workspace_bytes(B, H, Lmax, d, dv, LLA_BF16, 1);
    void* scratch = nullptr;
    if (ws > 0 && B > 0 && H > 0) {
        keep_pool_memory();
        if (cudaMallocAsync(&scratch, ws, (cudaStream_t)stream) != cudaSuccess) {
            (void)cudaGetLastError();
            scratch = nullptr;          // fall back to the fused epilogue
        }
    }
    p.workspace = scratch;
    p.workspace_bytes = scratch ? ws : 0;
    const int rc = lla_decode_ex(&p);
    if (scratch) (void)cudaFreeAsync(scratch, (cudaStream_t)stream);
    return rc;
}

int lla_decode_f32(const void* q, const void* kcache, const void* vcache, const int* lens, void* out,
                   int B, int H, int Lmax, int d, int dv, float scale, float lambda, void* stream) {
    lla_decode_params p = {};
    p.q = q; p.kcache = kcache; p.vcache = vcache; p.lens = lens; p.out = out;
    p.B = B; p.H = H; p.Lmax = Lmax; p.d = d; p.dv = dv;
    p.in_dtype = LLA_F32; p.out_dtype = LLA_F32;
    p.scale = scale; p.lambda = lambda;
    p.stream = stream;
    return lla_decode_ex(&p);
}

int lla_backward_ex(const lla_backward_params* p) {
    if (!p) return LLA_ERR_INVALID_ARG;
    if (!p->q || !p->k || !p->v || !p->out || !p->dout || !p->rho || !p->stats || !p->dq || !p->dk || !p->dv)
        return LLA_ERR_INVALID_ARG;
    if (p->B < 1 || p->H < 1 || p->n < 1 || p->d < 1) return LLA_ERR_INVALID_ARG;
    if (!(p->lambda >= 0.f) || !isfinite(p->lambda) || !isfinite(p->scale)) return LLA_ERR_INVALID_ARG;
    const uintptr_t align = (uintptr_t)p->q | (uintptr_t)p->k | (uintptr_t)p->v | (uintptr_t)p->out | (uintptr_t)p->dout |
                            (uintptr_t)p->rho | (uintptr_t)p->dq | (uintptr_t)p->dk | (uintptr_t)p->dv;
    if (align & 15u) return LLA_ERR_INVALID_ARG;
    if (p->d != 64 && p->d != 128) return LLA_ERR_UNSUPPORTED;
    if ((long long)p->B * p->H > 65535) return LLA_ERR_UNSUPPORTED;
    auto dt_ok = [](int t) { return t == LLA_BF16 || t == LLA_F32; };
    if (!dt_ok(p->out_dtype) || !dt_ok(p->dout_dtype)) return LLA_ERR_UNSUPPORTED;
    if (!p->workspace || ((uintptr_t)p->workspace & 255u) ||
        p->workspace_bytes < lla::backward_workspace_bytes(p->B, p->H, p->n, p->d))
        return LLA_ERR_WORKSPACE;
    BackwardArgs a = {};
    a.q = p->q; a.k = p->k; a.v = p->v; a.out = p->out; a.dout = p->dout;
    a.rho = p->rho; a.stats = p->stats; a.dq = p->dq; a.dk = p->dk; a.dv = p->dv;
    a.B = p->B; a.H = p->H; a.n = p->n; a.d = p->d;
    a.out_dtype = p->out_dtype; a.dout_dtype = p->dout_dtype;
    a.scale = p->scale; a.lambda = p->lambda;
    a.max_iters = p->max_iters > 0 ? p->max_iters : 64;
    a.tol = p->tol > 0.f ? p->tol : 1e-4f;
    a.head_rows = p->head_rows == 0 ? p->d + p->d / 2 : (p->head_rows < 0 ? 0 : p->head_rows);
    a.status = p->device_status;
    a.workspace = p->workspace; a.workspace_bytes = p->workspace_bytes;
    a.stream = (cudaStream_t)p->stream;
    if (p->impl != LLA_IMPL_AUTO && p->impl != LLA_IMPL_SIMT) return LLA_ERR_INVALID_ARG;
    a.cuda_core_pairs = p->impl == LLA_IMPL_SIMT;
    a.iters = p->iters;
    a.dlambda = p->dlambda;
    if (p->kv_heads < 0 || (p->kv_heads > 0 && p->H % p->kv_heads != 0)) return LLA_ERR_INVALID_ARG;
    a.kv_group = p->kv_heads > 0 ? p->H / p->kv_heads : 1;
    if (p->window < 0) return LLA_ERR_INVALID_ARG;
    // as in the forward, the window must leave the directly-solved rows whole; the CUDA-core kernels know no window
    if (p->window > 0 && (p->window < a.head_rows || a.cuda_core_pairs)) return LLA_ERR_UNSUPPORTED;
    a.window = p->window;
    if (p->cg_precondition != 0 && p->cg_precondition != 1) return LLA_ERR_INVALID_ARG;
    a.precondition = p->cg_precondition;
    // block sparsity: under the forward's conditions, and in the tensor-core kernels only
    if (p->block_mask && (a.cuda_core_pairs || a.window > 0 || p->n > 65536 || p->block_mask_stride < 0)) return LLA_ERR_UNSUPPORTED;
    a.block_mask = p->block_mask; a.block_mask_stride = p->block_mask_stride;
    // a chunk of queries against the whole key sequence: tensor-core kernels only, and not with a block mask
    if (p->q_rows < 0 || p->q_rows > p->n) return LLA_ERR_INVALID_ARG;
    a.nq = p->q_rows > 0 ? p->q_rows : p->n;
    if (a.nq != p->n && (a.cuda_core_pairs || p->block_mask)) return LLA_ERR_UNSUPPORTED;
    if (p->debug_wait_clocks < 0 || (p->debug_flags & ~LLA_DEBUG_NO_LOADS)) return LLA_ERR_INVALID_ARG;
    a.wait_clocks = p->debug_wait_clocks;
    a.no_loads = (p->debug_flags & LLA_DEBUG_NO_LOADS) ? 1 : 0;
    SideStream* side = side_stream();
    std::unique_lock<std::mutex> side_lock;
    if (side) {
        side_lock = std::unique_lock<std::mutex>(side->use);
        a.side_stream = side->stream; a.fork = side->fork; a.join = side->join;
    }
    ForwardArgs probe = {};
    probe.in_dtype = LLA_BF16; probe.d = p->d; probe.dv = p->d;
    if (!lla::forward_tensor_supported(probe)) return LLA_ERR_UNSUPPORTED;
    if (a.status) LLA_CUDA_TRY(cudaMemsetAsync(a.status, 0, sizeof(int) * LLA_STATUS_WORDS, a.stream));
    return lla::launch_backward(a);
}

size_t lla_backward_workspace_bytes(int B, int H, int n, int d) {
    if (B < 1 || H < 1 || n < 1 || d < 1) return 0;
    return lla::backward_workspace_bytes(B, H, n, d);
}

size_t lla_forward_workspace_bytes(int B, int H, int n, int d, int dv, int in_dtype, int impl) {
    if (B < 1 || H < 1 || n < 1) return 0;
    // Only the tensor-core kernel uses any: the fp16 copy of k for its later CG sweeps and, for d = 128, one
    // slot per SM id for the row vectors it keeps off chip (see lla_forward_tensor.cu).
    if (in_dtype == LLA_BF16 && (d == 64 || d == 128) && dv == d && impl != LLA_IMPL_SIMT)
        return lla::forward_tensor_workspace_bytes(B, H, n, d);
    return 0;
}

size_t lla_decode_workspace_bytes(int B, int H, int Lmax, int d, int dv, int in_dtype, int splits) {
    (void)Lmax;
    if (B < 1 || H < 1 || d < 1 || dv < 1) return 0;
    if (splits > 1) return lla::decode_workspace_bytes(B, H, d, dv, splits);
    // unsplit: optional.  The tensor-core path (bf16, d = dv = 64) uses it to run the solve as a
    // second kernel; without it the call still works (the streaming kernel solves in its epilogue).
    return (in_dtype == LLA_BF16 && d == 64 && dv == 64) ? lla::decode_record_bytes(B, H, d, dv, 1) : 0;
}

const char* lla_status_string(int status) {
    switch (status) {
        case LLA_OK: return "ok";
        case LLA_ERR_INVALID_ARG: return "invalid argument";
        case LLA_ERR_UNSUPPORTED: return "unsupported head size or dtype";
        case LLA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LLA_ERR_CUDA: return "CUDA runtime error";
        case LLA_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

int lla_version(void) { return 100; }

}  // extern "C"

// ---- host-buffer convenience entry points --------------------------------------------------
namespace {

struct DeviceScratch {   // stream-ordered allocations released on scope exit
    cudaStream_t stream;
    void* ptrs[8];
    int count = 0;
    explicit DeviceScratch(cudaStream_t s) : stream(s) {}
    void* get(size_t bytes) {
        void* p = nullptr;
        if (count >= 8 || cudaMallocAsync(&p, bytes ? bytes : 16, stream) != cudaSuccess) return nullptr;
        ptrs[count++] = p;
        return p;
    }
    ~DeviceScratch() {
        for (int i = 0; i < count; ++i) cudaFreeAsync(ptrs[i], stream);
    }
};

}  // namespace

extern "C" {

int lla_forward_host(const void* q, const void* k, const void* v, void* out, int B, int H, int n, int d,
                     int dv, int in_dtype, int out_dtype, float scale, float lambda, int causal, void* stream) {
    lla_forward_params p = {};
    p.q = q; p.k = k; p.v = v; p.out = out;   // host pointers: only checked for null / alignment here
    p.B = B; p.H = H; p.n = n; p.d = d; p.dv = dv;
    p.in_dtype = in_dtype; p.out_dtype = out_dtype;
    p.scale = scale; p.lambda = lambda; p.causal = causal;
    p.stream = stream;
    const int rc = check_forward(&p);
    if (rc != LLA_OK) return rc;
    keep_pool_memory();
    cudaStream_t st = (cudaStream_t)stream;
    const size_t esz_in = in_dtype == LLA_F32 ? 4 : 2, esz_out = out_dtype == LLA_F32 ? 4 : 2;
    const size_t nq = (size_t)B * H * n * d * esz_in, nv = (size_t)B * H * n * dv * esz_in;
    const size_t no = (size_t)B * H * n * dv * esz_out;
    DeviceScratch mem(st);
    void* dq = mem.get(nq); void* dk = mem.get(nq); void* dvv = mem.get(nv); void* dout = mem.get(no);
    if (!dq || !dk || !dvv || !dout) return LLA_ERR_CUDA;
    const int units = B * H;
    HostPipe* pipe = (units >= 2 * kHostChunks && nq + nq + nv >= (size_t)(1u << 20)) ? host_pipe() : nullptr;
    if (!pipe) {
        const size_t wsb = lla_forward_workspace_bytes(B, H, n, d, dv, in_dtype, LLA_IMPL_AUTO);
        if (wsb > 0) {
            p.workspace = mem.get(wsb);
            p.workspace_bytes = p.workspace ? wsb : 0;
        }
        LLA_CUDA_TRY(cudaMemcpyAsync(dq, q, nq, cudaMemcpyHostToDevice, st));
        LLA_CUDA_TRY(cudaMemcpyAsync(dk, k, nq, cudaMemcpyHostToDevice, st));
        LLA_CUDA_TRY(cudaMemcpyAsync(dvv, v, nv, cudaMemcpyHostToDevice, st));
        p.q = dq; p.k = dk; p.v = dvv; p.out = dout;
        const int st_rc = lla_forward_ex(&p);
        if (st_rc != LLA_OK) return st_rc;
        LLA_CUDA_TRY(cudaMemcpyAsync(out, dout, no, cudaMemcpyDeviceToHost, st));
        LLA_CUDA_TRY(cudaStreamSynchronize(st));
        return LLA_OK;
    }
    // chunked: (batch, head) units are independent and contiguous in memory; every chunk has its own scratch
    const int chunk_units = (units + kHostChunks - 1) / kHostChunks;
    const size_t wsb = lla_forward_workspace_bytes(1, chunk_units, n, d, dv, in_dtype, LLA_IMPL_AUTO);
    char* wsp = wsb > 0 ? static_cast<char*>(mem.get(wsb * kHostChunks)) : nullptr;
    std::lock_guard<std::mutex> pipe_lock(pipe->use);
    const size_t uq = (size_t)n * d * esz_in, uv = (size_t)n * dv * esz_in, uo = (size_t)n * dv * esz_out;
    int rc_chunks = LLA_OK;
    auto enqueue = [&]() -> int {
        LLA_CUDA_TRY(cudaEventRecord(pipe->ready, st));            // the buffers exist from here on
        for (int c = 0; c < kHostChunks; ++c) {
            const int u0 = (int)((long long)units * c / kHostChunks), u1 = (int)((long long)units * (c + 1) / kHostChunks);
            cudaStream_t w = pipe->stream[c];
            LLA_CUDA_TRY(cudaStreamWaitEvent(w, pipe->ready, 0));
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)dq + u0 * uq, (const char*)q + u0 * uq, (u1 - u0) * uq, cudaMemcpyHostToDevice, w));
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)dk + u0 * uq, (const char*)k + u0 * uq, (u1 - u0) * uq, cudaMemcpyHostToDevice, w));
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)dvv + u0 * uv, (const char*)v + u0 * uv, (u1 - u0) * uv, cudaMemcpyHostToDevice, w));
            lla_forward_params pc = p;
            pc.q = (char*)dq + u0 * uq; pc.k = (char*)dk + u0 * uq; pc.v = (char*)dvv + u0 * uv; pc.out = (char*)dout + u0 * uo;
            pc.B = 1; pc.H = u1 - u0;
            pc.stream = w;
            if (wsp) { pc.workspace = wsp + (size_t)c * wsb; pc.workspace_bytes = wsb; }
            const int rc_c = lla_forward_ex(&pc);
            if (rc_c != LLA_OK && rc_chunks == LLA_OK) rc_chunks = rc_c;
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)out + u0 * uo, (char*)dout + u0 * uo, (u1 - u0) * uo, cudaMemcpyDeviceToHost, w));
            LLA_CUDA_TRY(cudaEventRecord(pipe->done[c], w));
            LLA_CUDA_TRY(cudaStreamWaitEvent(st, pipe->done[c], 0));
        }
        return LLA_OK;
    };
    const int rc_q = enqueue();
    if (rc_q != LLA_OK) {
        // something could not be enqueued: the workers may still be using the buffers that go back to the pool
        // when this function returns, so wait for them here
        for (int c = 0; c < kHostChunks; ++c) (void)cudaStreamSynchronize(pipe->stream[c]);
        (void)cudaStreamSynchronize(st);
        return rc_q;
    }
    LLA_CUDA_TRY(cudaStreamSynchronize(st));
    return rc_chunks;
}

int lla_decode_host(const void* q, const void* kcache, const void* vcache, const int* lens, void* out, int B,
                    int H, int Lmax, int d, int dv, int in_dtype, int out_dtype, float scale, float lambda,
                    void* stream) {
    lla_decode_params p = {};
    p.q = q; p.kcache = kcache; p.vcache = vcache; p.lens = lens; p.out = out;
    p.B = B; p.H = H; p.Lmax = Lmax; p.d = d; p.dv = dv;
    p.in_dtype = in_dtype; p.out_dtype = out_dtype;
    p.scale = scale; p.lambda = lambda;
    p.splits = 1;
    p.stream = stream;
    const int rc = check_decode(&p);
    if (rc != LLA_OK) return rc;
    keep_pool_memory();
    cudaStream_t st = (cudaStream_t)stream;
    const size_t esz_in = in_dtype == LLA_F32 ? 4 : 2, esz_out = out_dtype == LLA_F32 ? 4 : 2;
    const size_t nq = (size_t)B * H * d * esz_in, no = (size_t)B * H * dv * esz_out;
    const size_t nk = (size_t)B * H * Lmax * d * esz_in, nv = (size_t)B * H * Lmax * dv * esz_in;
    DeviceScratch mem(st);
    void* dq = mem.get(nq); void* dk = mem.get(nk); void* dvv = mem.get(nv);
    void* dl = mem.get(sizeof(int) * (size_t)B); void* dout = mem.get(no);
    if (!dq || !dk || !dvv || !dl || !dout) return LLA_ERR_CUDA;
    const size_t ws = lla_decode_workspace_bytes(B, H, Lmax, d, dv, in_dtype, 1);
    if (ws > 0) {
        p.workspace = mem.get(ws);
        p.workspace_bytes = p.workspace ? ws : 0;
    }
    LLA_CUDA_TRY(cudaMemcpyAsync(dq, q, nq, cudaMemcpyHostToDevice, st));
    LLA_CUDA_TRY(cudaMemcpyAsync(dl, lens, sizeof(int) * (size_t)B, cudaMemcpyHostToDevice, st));
    // only the live prefix of every (sequence, head) cache crosses the bus
    for (int b = 0; b < B; ++b) {
        int L = lens[b] < 1 ? 1 : (lens[b] > Lmax ? Lmax : lens[b]);
        for (int h = 0; h < H; ++h) {
            const size_t off = ((size_t)b * H + h) * Lmax;
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)dk + off * d * esz_in, (const char*)kcache + off * d * esz_in,
                                         (size_t)L * d * esz_in, cudaMemcpyHostToDevice, st));
            LLA_CUDA_TRY(cudaMemcpyAsync((char*)dvv + off * dv * esz_in, (const char*)vcache + off * dv * esz_in,
                                         (size_t)L * dv * esz_in, cudaMemcpyHostToDevice, st));
        }
    }
    p.q = dq; p.kcache = dk; p.vcache = dvv; p.lens = (const int*)dl; p.out = dout;
    const int st_rc = lla_decode_ex(&p);
    if (st_rc != LLA_OK) return st_rc;
    LLA_CUDA_TRY(cudaMemcpyAsync(out, dout, no, cudaMemcpyDeviceToHost, st));
    LLA_CUDA_TRY(cudaStreamSynchronize(st));
    return LLA_OK;
}

}  // extern "C"
