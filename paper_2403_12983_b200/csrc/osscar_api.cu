// C ABI of libosscar: argument checks, context and workspace bookkeeping, call sequencing.
#include "osscar_internal.cuh"
#include <new>
#include <string.h>
#include <cuda_bf16.h>
#include "tc_common.cuh"

using namespace osscar;

namespace osscar { unsigned long long g_launches = 0; }

namespace {

#define CKC(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return OSSCAR_E_CUDA; } while (0)
// the same for calls that follow enqueued work: the stream is drained first, so that a failed call never returns with
// kernels still running on the caller's buffers
#define CKS(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { cudaStreamSynchronize(st); return OSSCAR_E_CUDA; } } while (0)

struct DeviceGuard {
    int prev; bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

__global__ void k_clear_status(SearchCtl* ctl) { ctl->status = OSSCAR_OK; ctl->done = 0; }
__global__ void k_set_wait_limit(SearchCtl* ctl, long long cycles) { ctl->wait_limit = cycles; }

// diag sum of H in fp64, then H += damp * mean(diag) * I
__global__ void k_diag_sum(const float* __restrict__ H, int64_t d1, double* __restrict__ out)
{
    double acc = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d1; i += (int64_t)gridDim.x * blockDim.x)
        acc += (double)H[i * d1 + i];
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) atomicAdd(out, acc);
}
__global__ void k_add_damp(float* __restrict__ H, int64_t d1, float damp, const double* __restrict__ diag_sum)
{
    const float lam = (float)((double)damp * (*diag_sum) / (double)d1);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d1; i += (int64_t)gridDim.x * blockDim.x)
        H[i * d1 + i] += lam;
}
__global__ void k_sub(const float* __restrict__ A, const float* __restrict__ B, float* __restrict__ C, int64_t n)
{
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        C[i] = A[i] - B[i];
}

// sum of squares of a row block of Y (bf16 or fp32) in two deterministic stages, added to *acc
__global__ void k_sumsq(const void* __restrict__ Y, int is_fp32, int64_t n, double* __restrict__ partial)
{
    __shared__ double red[32];
    double acc = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const double v = is_fp32 ? (double)((const float*)Y)[i] : (double)__bfloat162float(((const __nv_bfloat16*)Y)[i]);
        acc += v * v;
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) { double s = 0.0; for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i]; partial[blockIdx.x] = s; }
}
__global__ void k_add_partials(const double* __restrict__ partial, int n, double* __restrict__ acc, int reset)
{
    __shared__ double red[32];
    double a = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) a += partial[i];
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) { double s = 0.0; for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i]; *acc = reset ? s : *acc + s; }
}

}  // namespace

extern "C" {

uint64_t osscar_launch_count(void) { return g_launches; }

const char* osscar_status_string(int s)
{
    switch (s) {
        case OSSCAR_OK: return "ok";
        case OSSCAR_E_ARG: return "bad argument";
        case OSSCAR_E_SHAPE: return "inconsistent shape";
        case OSSCAR_E_NOTPD: return "H restricted to the support is not positive definite";
        case OSSCAR_E_WORKSPACE: return "workspace missing or too small";
        case OSSCAR_E_CUDA: return "CUDA call failed";
        case OSSCAR_E_TIMEOUT: return "device-side wait timed out";
        case OSSCAR_E_STATE: return "call order violated";
        default: return "unknown status";
    }
}

int osscar_create(osscar_ctx** out, int device, void* cuda_stream)
{
    if (!out) return OSSCAR_E_ARG;
    *out = nullptr;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return OSSCAR_E_CUDA;
    DeviceGuard guard(device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    osscar_ctx* ctx = new (std::nothrow) osscar_ctx();
    if (!ctx) return OSSCAR_E_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    bool ok = cudaMalloc((void**)&ctx->ctl, sizeof(SearchCtl)) == cudaSuccess
           && cudaMemset(ctx->ctl, 0, sizeof(SearchCtl)) == cudaSuccess
           && cudaMalloc((void**)&ctx->partials, sizeof(double) * kTracePartials) == cudaSuccess
           && cudaHostAlloc((void**)&ctx->ctl_host, sizeof(SearchCtl), cudaHostAllocDefault) == cudaSuccess
           && cudaHostAlloc((void**)&ctx->done_flag_host, 64, cudaHostAllocMapped) == cudaSuccess
           && cudaHostGetDevicePointer((void**)&ctx->done_flag_dev, (void*)ctx->done_flag_host, 0) == cudaSuccess
           && cudaEventCreate(&ctx->ev0) == cudaSuccess && cudaEventCreate(&ctx->ev1) == cudaSuccess;
    if (ok) {
        ctx->wait_limit = tc::kWaitLimitCycles;
        k_set_wait_limit<<<1, 1>>>(ctx->ctl, ctx->wait_limit);
        ok = cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) { osscar_destroy(ctx); return OSSCAR_E_CUDA; }
    *ctx->done_flag_host = 0;
    *out = ctx;
    return OSSCAR_OK;
}

int osscar_destroy(osscar_ctx* ctx)
{
    if (!ctx) return OSSCAR_E_ARG;
    DeviceGuard guard(ctx->device);
    if (ctx->ctl) cudaFree(ctx->ctl);
    if (ctx->partials) cudaFree(ctx->partials);
    if (ctx->ctl_host) cudaFreeHost(ctx->ctl_host);
    if (ctx->done_flag_host) cudaFreeHost((void*)ctx->done_flag_host);
    if (ctx->ev0) cudaEventDestroy(ctx->ev0);
    if (ctx->ev1) cudaEventDestroy(ctx->ev1);
    delete ctx;
    return OSSCAR_OK;
}

int osscar_set_wait_limit(osscar_ctx* ctx, uint64_t cycles)
{
    if (!ctx) return OSSCAR_E_ARG;
    if (cycles > (uint64_t)1 << 62) return OSSCAR_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    ctx->wait_limit = cycles ? (long long)cycles : tc::kWaitLimitCycles;
    k_set_wait_limit<<<1, 1, 0, ctx->stream>>>(ctx->ctl, ctx->wait_limit);
    count_launches(1);
    CKC(cudaGetLastError());
    return OSSCAR_OK;
}

int osscar_set_shard_reduce(osscar_ctx* ctx, osscar_reduce_fn fn, void* user)
{
    if (!ctx) return OSSCAR_E_ARG;
    ctx->reduce = fn;
    ctx->reduce_user = fn ? user : nullptr;
    ctx->have_state = false;
    return OSSCAR_OK;
}

int osscar_workspace_bytes(int64_t d1, int64_t m, int32_t g, int32_t k, size_t* bytes)
{
    if (!bytes) return OSSCAR_E_ARG;
    Layout L;
    const int rc = make_layout(d1, m, g, k, &L);
    if (rc != OSSCAR_OK) return rc;
    *bytes = L.bytes;
    return OSSCAR_OK;
}

int osscar_set_workspace(osscar_ctx* ctx, void* dev_ptr, size_t bytes)
{
    if (!ctx) return OSSCAR_E_ARG;
    if (dev_ptr && ((uintptr_t)dev_ptr & 255)) return OSSCAR_E_ARG;
    ctx->ws = dev_ptr;
    ctx->ws_bytes = dev_ptr ? bytes : 0;
    ctx->have_state = false;
    return OSSCAR_OK;
}

int osscar_gram(osscar_ctx* ctx, const void* X, int x_dtype, int64_t n_rows, int64_t d1,
                const float* W, int64_t m, int flags, float damp,
                float* H, float* G, double* const_term)
{
    if (!ctx || !H || (n_rows > 0 && !X)) return OSSCAR_E_ARG;
    if (x_dtype != OSSCAR_BF16 && x_dtype != OSSCAR_FP32) return OSSCAR_E_ARG;
    if (flags & ~(OSSCAR_GRAM_BEGIN | OSSCAR_GRAM_END)) return OSSCAR_E_ARG;
    if (d1 <= 0 || n_rows < 0 || !(damp >= 0.f)) return OSSCAR_E_SHAPE;
    const bool begin = flags & OSSCAR_GRAM_BEGIN, end = flags & OSSCAR_GRAM_END;
    if (end && (!W || !G || !const_term || m <= 0)) return OSSCAR_E_ARG;
    if (x_dtype == OSSCAR_BF16 && n_rows > 0 && ((d1 % 8) != 0 || ((uintptr_t)X & 15))) return OSSCAR_E_SHAPE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    cudaStream_t st = ctx->stream;
    // a device-side error of any chunk must reach the END call: the status is cleared by the BEGIN chunk only
    if (begin) { k_clear_status<<<1, 1, 0, st>>>(ctx->ctl); count_launches(1); }
    if (begin) ctx->gram_rows = 0;
    if (begin && n_rows == 0) CKS(cudaMemsetAsync(H, 0, sizeof(float) * d1 * d1, st));
    if (n_rows > 0) {
        if (x_dtype == OSSCAR_BF16) {
            // upper-triangle tiles only; the lower triangle is filled on END
            CKS(gram_tc2(st, X, n_rows, d1, nullptr, 0, 0, H, !begin, nullptr, 0, ctx->ctl));
        } else {
            // fp32 activations: three-term bf16 split on the tensor cores when a workspace is lent (its contents are
            // overwritten), else (or when it cannot hold a 64-row panel of the terms) the fp32 pipes
            cudaError_t ge = cudaErrorMemoryAllocation;
            if (ctx->ws) {
                ge = gram_tc3(st, (const float*)X, n_rows, d1, H, !begin, ctx->ws, ctx->ws_bytes, ctx->ctl);
                if (ge == cudaSuccess) ctx->have_state = false;
            }
            if (ge == cudaErrorMemoryAllocation)
                ge = sgemm(st, true, false, d1, d1, n_rows, 1.f, (const float*)X, d1, (const float*)X, d1, begin ? 0.f : 1.f, H, d1);
            CKS(ge);
        }
        ctx->gram_rows += (double)n_rows;
    }
    if (!end) { CKS(cudaGetLastError()); return OSSCAR_OK; }
    ctx->have_const = false;
    CKS(gram_mirror(st, H, d1));
    if (damp > 0.f) {
        CKS(cudaMemsetAsync(&ctx->ctl->acc[0], 0, sizeof(double), st));
        k_diag_sum<<<64, 256, 0, st>>>(H, d1, &ctx->ctl->acc[0]);
        k_add_damp<<<64, 256, 0, st>>>(H, d1, damp, &ctx->ctl->acc[0]);
        count_launches(2);
    }
    if (ctx->ws && ctx->ws_bytes >= gemm_tc_min_scratch(d1, m)) {
        // tensor-core product with the operand terms staged in the lent workspace (its contents are overwritten)
        const size_t cap = ctx->ws_bytes < ((size_t)3 << 30) ? ctx->ws_bytes : ((size_t)3 << 30);
        CKS(gemm_tc(st, d1, m, d1, 1.f, H, d1, W, m, 0.f, G, m, ctx->ws, cap, ctx->ctl));
        ctx->have_state = false;
    } else {
        CKS(sgemm(st, false, false, d1, m, d1, 1.f, H, d1, W, m, 0.f, G, m));
    }
    CKS(trace_product(st, W, m, G, m, d1, m, ctx->partials, &ctx->ctl->acc[1]));
    CKS(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CKS(cudaStreamSynchronize(st));
    if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;
    *const_term = ctx->ctl_host->acc[1];
    return OSSCAR_OK;
}

int osscar_gram_cross(osscar_ctx* ctx, const void* X, int x_dtype, const void* Y, int y_dtype,
                      int64_t n_rows, int64_t d1, int64_t m, int flags, float damp,
                      float* H, float* G, double* const_term)
{
    if (!ctx || !H || !G || (n_rows > 0 && (!X || !Y))) return OSSCAR_E_ARG;
    if ((x_dtype != OSSCAR_BF16 && x_dtype != OSSCAR_FP32) || (y_dtype != OSSCAR_BF16 && y_dtype != OSSCAR_FP32)) return OSSCAR_E_ARG;
    if (x_dtype == OSSCAR_FP32 && y_dtype != OSSCAR_FP32) return OSSCAR_E_ARG;
    if (flags & ~(OSSCAR_GRAM_BEGIN | OSSCAR_GRAM_END)) return OSSCAR_E_ARG;
    if (d1 <= 0 || m <= 0 || n_rows < 0 || !(damp >= 0.f)) return OSSCAR_E_SHAPE;
    const bool begin = flags & OSSCAR_GRAM_BEGIN, end = flags & OSSCAR_GRAM_END;
    if (end && !const_term) return OSSCAR_E_ARG;
    if (x_dtype == OSSCAR_BF16 && n_rows > 0) {
        if ((d1 % 8) != 0 || ((uintptr_t)X & 15)) return OSSCAR_E_SHAPE;
        if (y_dtype == OSSCAR_BF16 && ((m % 8) != 0 || ((uintptr_t)Y & 15))) return OSSCAR_E_SHAPE;
    }
    const size_t need = y_dtype == OSSCAR_FP32 && x_dtype == OSSCAR_BF16
                      ? 3 * (((size_t)n_rows * round_up(m, 8) * 2 + 1023) / 1024 * 1024) : 0;
    if (need > 0 && (!ctx->ws || ctx->ws_bytes < need)) return OSSCAR_E_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    cudaStream_t st = ctx->stream;
    if (begin) { k_clear_status<<<1, 1, 0, st>>>(ctx->ctl); count_launches(1); }     // sticky until END, as in osscar_gram
    if (begin && n_rows == 0) {
        CKS(cudaMemsetAsync(H, 0, sizeof(float) * d1 * d1, st));
        CKS(cudaMemsetAsync(G, 0, sizeof(float) * d1 * m, st));
        CKS(cudaMemsetAsync(&ctx->ctl->acc[2], 0, sizeof(double), st));
    }
    if (n_rows > 0) {
        if (x_dtype == OSSCAR_BF16) {
            CKS(gram_tc2(st, X, n_rows, d1, nullptr, 0, 0, H, !begin, nullptr, 0, ctx->ctl));
            CKS(gram_tc2(st, X, n_rows, d1, Y, y_dtype == OSSCAR_FP32, m, G, !begin, ctx->ws, ctx->ws_bytes, ctx->ctl));
            if (need > 0) ctx->have_state = false;
        } else {
            // H as in osscar_gram: on the tensor cores when a workspace can stage the bf16 terms, else the fp32 pipes
            cudaError_t ge = cudaErrorMemoryAllocation;
            if (ctx->ws) {
                ge = gram_tc3(st, (const float*)X, n_rows, d1, H, !begin, ctx->ws, ctx->ws_bytes, ctx->ctl);
                if (ge == cudaSuccess) ctx->have_state = false;
            }
            if (ge == cudaErrorMemoryAllocation)
                ge = sgemm(st, true, false, d1, d1, n_rows, 1.f, (const float*)X, d1, (const float*)X, d1, begin ? 0.f : 1.f, H, d1);
            CKS(ge);
            CKS(sgemm(st, true, false, d1, m, n_rows, 1.f, (const float*)X, d1, (const float*)Y, m, begin ? 0.f : 1.f, G, m));
        }
        const int nblk = kTracePartials;
        k_sumsq<<<nblk, 256, 0, st>>>(Y, y_dtype == OSSCAR_FP32, n_rows * m, ctx->partials);
        k_add_partials<<<1, 256, 0, st>>>(ctx->partials, nblk, &ctx->ctl->acc[2], begin ? 1 : 0);
        count_launches(2);
    }
    if (!end) { CKS(cudaGetLastError()); return OSSCAR_OK; }
    CKS(gram_mirror(st, H, d1));
    if (damp > 0.f) {
        CKS(cudaMemsetAsync(&ctx->ctl->acc[0], 0, sizeof(double), st));
        k_diag_sum<<<64, 256, 0, st>>>(H, d1, &ctx->ctl->acc[0]);
        k_add_damp<<<64, 256, 0, st>>>(H, d1, damp, &ctx->ctl->acc[0]);
        count_launches(2);
    }
    CKS(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CKS(cudaStreamSynchronize(st));
    if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;
    *const_term = ctx->ctl_host->acc[2];
    ctx->have_const = true;
    ctx->user_const = *const_term;
    return OSSCAR_OK;
}

int osscar_set_const_term(osscar_ctx* ctx, double const_term, int enabled)
{
    if (!ctx) return OSSCAR_E_ARG;
    ctx->have_const = enabled != 0;
    ctx->user_const = const_term;
    return OSSCAR_OK;
}

int osscar_init_support(osscar_ctx* ctx, const float* H, const float* G, const float* W,
                        int64_t d1, int64_t m, int32_t g, int32_t k, int mode,
                        int32_t* support, double* obj0)
{
    if (!ctx || !H || !G || !W || !support || !obj0) return OSSCAR_E_ARG;
    if (mode != OSSCAR_INIT_ENERGY && mode != OSSCAR_INIT_MAGNITUDE && mode != OSSCAR_INIT_USER) return OSSCAR_E_ARG;
    Layout L;
    const int rc0 = make_layout(d1, m, g, k, &L);
    if (rc0 != OSSCAR_OK) return rc0;
    if (!ctx->ws || ctx->ws_bytes < L.bytes) return OSSCAR_E_WORKSPACE;
    if (ctx->reduce && g != 1) return OSSCAR_E_ARG;             // column shards: single-row groups only
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    ctx->L = L; ctx->H = H; ctx->G = G; ctx->W = W; ctx->have_state = false;
    cudaStream_t st = ctx->stream;
    k_clear_status<<<1, 1, 0, st>>>(ctx->ctl);
    count_launches(1);
    int rc = select_support(ctx, mode, support);
    if (rc == OSSCAR_OK && mode == OSSCAR_INIT_USER) {
        // a rejected list (duplicate or out-of-range ids) ends the call here: nothing is built on it
        CKS(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
        CKS(cudaStreamSynchronize(st));
        if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;
    }
    if (rc == OSSCAR_OK) rc = build_state(ctx, false);
    if (rc == OSSCAR_OK && score_pass(ctx) != cudaSuccess) rc = OSSCAR_E_CUDA;
    if (rc != OSSCAR_OK) { cudaStreamSynchronize(st); return rc; }
    CKC(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CKC(cudaStreamSynchronize(st));
    if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;
    *obj0 = ctx->ctl_host->obj;
    ctx->have_state = true;
    return OSSCAR_OK;
}

int osscar_init_support_greedy(osscar_ctx* ctx, const float* H, const float* G, const float* W,
                               int64_t d1, int64_t m, int32_t g, int32_t k, int32_t t_hat,
                               int32_t* support, int32_t* drop_trace, double* obj0, int32_t* n_iters)
{
    if (!ctx || !H || !G || !W || !support || !obj0) return OSSCAR_E_ARG;
    Layout L;
    const int rc0 = make_layout(d1, m, g, k, &L);
    if (rc0 != OSSCAR_OK) return rc0;
    if (t_hat < 1 || (int64_t)t_hat * g > 256) return OSSCAR_E_SHAPE;
    if (ctx->reduce) return OSSCAR_E_ARG;                       // the nested phase is not sharded
    if (!ctx->ws || ctx->ws_bytes < L.bytes) return OSSCAR_E_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    ctx->L = L; ctx->H = H; ctx->G = G; ctx->W = W; ctx->have_state = false;
    cudaStream_t st = ctx->stream;
    k_clear_status<<<1, 1, 0, st>>>(ctx->ctl);
    count_launches(1);
    int iters = 0;
    int rc = greedy_support(ctx, t_hat, support, drop_trace, &iters);
    if (rc == OSSCAR_OK) rc = build_state(ctx, false);
    if (rc == OSSCAR_OK && score_pass(ctx) != cudaSuccess) rc = OSSCAR_E_CUDA;
    if (rc != OSSCAR_OK) { cudaStreamSynchronize(st); return rc; }
    CKC(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CKC(cudaStreamSynchronize(st));
    if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;
    *obj0 = ctx->ctl_host->obj;
    if (n_iters) *n_iters = iters;
    ctx->have_state = true;
    return OSSCAR_OK;
}

int osscar_local_search(osscar_ctx* ctx, const osscar_search_params* params,
                        int32_t* support_out, float* W_out, double* obj_trace, int32_t* swap_trace,
                        osscar_search_result* result)
{
    if (!ctx || !params || !support_out || !W_out || !obj_trace || !result) return OSSCAR_E_ARG;
    if (params->max_swaps < 0 || (params->max_swaps > 0 && !swap_trace)) return OSSCAR_E_ARG;
    if (params->score_mode != OSSCAR_SCORE_INDEPENDENT && params->score_mode != OSSCAR_SCORE_PAIR_EXACT) return OSSCAR_E_ARG;
    if (params->accept_mode != OSSCAR_ACCEPT_IMPROVING && params->accept_mode != OSSCAR_ACCEPT_ALWAYS) return OSSCAR_E_ARG;
    if (params->refresh_every < 0 || params->profile_samples < 0 || params->profile_samples > 8 || params->block_pairs < 0) return OSSCAR_E_ARG;
    if (params->loop_mode < OSSCAR_LOOP_AUTO || params->loop_mode > OSSCAR_LOOP_LAUNCHES || params->wait_limit_cycles > (uint64_t)1 << 62) return OSSCAR_E_ARG;
    if (!ctx->have_state) return OSSCAR_E_STATE;
    if (params->score_mode == OSSCAR_SCORE_PAIR_EXACT && ctx->L.nJ > 0 && ctx->L.pair_capacity == 0) return OSSCAR_E_SHAPE;
    if (ctx->reduce && (ctx->L.g != 1 || params->score_mode != OSSCAR_SCORE_INDEPENDENT || params->block_pairs > 1 ||
                        params->loop_mode == OSSCAR_LOOP_PERSISTENT)) return OSSCAR_E_ARG;      // what column shards support
    if (params->block_pairs > 1) {      // block exchanges: independent scores, s <= min(k, pruned groups), s g rows fit the panels
        const osscar::Layout& L = ctx->L;
        const int64_t s = params->block_pairs;
        if (params->score_mode != OSSCAR_SCORE_INDEPENDENT || s * L.g > L.block_rows_max || s > L.k || s > L.ng - L.k) return OSSCAR_E_ARG;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    memset(result, 0, sizeof(*result));
    const int rc = run_search(ctx, params, support_out, W_out, obj_trace, swap_trace, result);
    if (rc != OSSCAR_OK) ctx->have_state = false;
    return rc;
}

int osscar_objective(osscar_ctx* ctx, const float* H, const float* W, const float* Wt,
                     int64_t d1, int64_t m, double* obj)
{
    if (!ctx || !H || !W || !Wt || !obj) return OSSCAR_E_ARG;
    if (d1 <= 0 || m <= 0) return OSSCAR_E_SHAPE;
    const size_t need = sizeof(float) * 2 * (size_t)d1 * (size_t)m;
    if (!ctx->ws || ctx->ws_bytes < need) return OSSCAR_E_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    cudaStream_t st = ctx->stream;
    float* E = (float*)ctx->ws;
    float* HE = E + d1 * m;
    k_clear_status<<<1, 1, 0, st>>>(ctx->ctl);
    k_sub<<<1184, 256, 0, st>>>(W, Wt, E, d1 * m);
    count_launches(2);
    CKS(sgemm(st, false, false, d1, m, d1, 1.f, H, d1, E, m, 0.f, HE, m));
    CKS(trace_product(st, E, m, HE, m, d1, m, ctx->partials, &ctx->ctl->acc[0]));
    CKS(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CKS(cudaStreamSynchronize(st));
    ctx->have_state = false;      // the workspace start was overwritten
    if (ctx->ctl_host->status != OSSCAR_OK) return ctx->ctl_host->status;      // raised on the device during this call
    *obj = ctx->ctl_host->acc[0];
    return OSSCAR_OK;
}

int osscar_debug_get_state(osscar_ctx* ctx, int which, void* dst)
{
    if (!ctx || !dst) return OSSCAR_E_ARG;
    if (!ctx->have_state) return OSSCAR_E_STATE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return OSSCAR_E_CUDA;
    const Layout& L = ctx->L;
    char* ws = (char*)ctx->ws;
    cudaStream_t st = ctx->stream;
    const int64_t npr = L.ng - L.k;
    switch (which) {
        case 0: CKC(cudaMemcpy2DAsync(dst, sizeof(float) * L.nI, ws + L.off_Hinv, sizeof(float) * L.ldh, sizeof(float) * L.nI, L.nI, cudaMemcpyDeviceToDevice, st)); break;
        case 1: CKC(cudaMemcpy2DAsync(dst, sizeof(float) * L.m, ws + L.off_V, sizeof(float) * L.ldm, sizeof(float) * L.m, L.nI, cudaMemcpyDeviceToDevice, st)); break;
        case 2: if (L.nJ > 0) CKC(cudaMemcpy2DAsync(dst, sizeof(float) * L.m, ws + L.off_R, sizeof(float) * L.ldm, sizeof(float) * L.m, L.nJ, cudaMemcpyDeviceToDevice, st)); break;
        case 3: CKC(cudaMemcpyAsync(dst, ws + L.off_c, sizeof(double) * npr * L.g * L.g, cudaMemcpyDeviceToDevice, st)); break;
        case 4: CKC(cudaMemcpyAsync(dst, ws + L.off_perm, sizeof(int32_t) * L.ng, cudaMemcpyDeviceToDevice, st)); break;
        case 5: CKC(cudaMemcpyAsync(dst, ws + L.off_D, sizeof(double) * L.k, cudaMemcpyDeviceToDevice, st)); break;
        case 6: CKC(cudaMemcpyAsync(dst, ws + L.off_A, sizeof(double) * npr, cudaMemcpyDeviceToDevice, st)); break;
        default: return OSSCAR_E_ARG;
    }
    CKC(cudaStreamSynchronize(st));
    return OSSCAR_OK;
}

}  // extern "C"
