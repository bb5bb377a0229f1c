// Allocation-free trace reduction: sum_ij A[i][j] * B[i][j] (e.g. const = Tr(W^T G), or the objective
// identity Tr(W_J^T R_J)) with every byte of scratch taken from a fixed array that is part of the
// library image.  See osscar_trace_noalloc in osscar.h for who needs this and for its limits.
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>
#include "osscar.h"

namespace osscar { extern unsigned long long g_launches; }     // the library-wide launch counter (osscar_launch_count)

namespace {

// One partial sum per row, then one slot for the total.  This array exists once per GPU that loads the
// library and is shared by every call: two calls whose kernels overlap on the GPU would race on it.
static __device__ __align__(256) double g_noalloc_scratch[OSSCAR_NOALLOC_MAX_ROWS + 32];

constexpr int kMaxDevices = 64;
// Device address of the array, looked up on first use per device.  Callers on different host threads may arrive here
// together; every writer stores the same value, and the atomic makes that store and the later loads well defined.
std::atomic<double*> g_scratch_addr[kMaxDevices];

// true iff p is device memory of `device` (or managed memory, which every device can reach)
bool on_device(const void* p, int device)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeManaged || (at.type == cudaMemoryTypeDevice && at.device == device);
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Stage 1: block r writes partial[r] = sum_j A[r][j] * B[r][j] (every slot that stage 2 reads is written here,
// so nothing left over from an earlier call can leak into the result).
__global__ void k_noalloc_rows(const float* __restrict__ A, int64_t lda, const float* __restrict__ B, int64_t ldb,
                               int64_t cols, double* __restrict__ partial)
{
    __shared__ double red[8];
    const int64_t r = blockIdx.x;
    double acc = 0.0;
    for (int64_t c = threadIdx.x; c < cols; c += blockDim.x) acc += (double)A[r * lda + c] * (double)B[r * ldb + c];
    acc = warp_sum_d(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i];
        partial[r] = s;
    }
}
// Stage 2: one block adds the row partials in a fixed order and overwrites the total slot.
__global__ void k_noalloc_total(const double* __restrict__ partial, int64_t rows, double* __restrict__ total)
{
    __shared__ double red[32];
    double acc = 0.0;
    for (int64_t i = threadIdx.x; i < rows; i += blockDim.x) acc += partial[i];
    acc = warp_sum_d(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i];
        *total = s;
    }
}

}  // namespace

extern "C" int osscar_trace_noalloc(const float* A, int64_t lda, const float* B, int64_t ldb,
                                    int64_t rows, int64_t cols, int device, void* cuda_stream, double* out)
{
    if (!A || !B || !out) return OSSCAR_E_ARG;
    if (rows < 0 || cols < 0 || lda < cols || ldb < cols) return OSSCAR_E_SHAPE;
    if (rows > OSSCAR_NOALLOC_MAX_ROWS) return OSSCAR_E_SHAPE;          // beyond the built-in scratch
    if (device < 0 || device >= kMaxDevices) return OSSCAR_E_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return OSSCAR_E_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return OSSCAR_E_CUDA;
    int rc = OSSCAR_OK;
    // the kernels run on `device`: both matrices must live there (a wrong ordinal would aim them at foreign pointers)
    if (rows > 0 && cols > 0 && (!on_device(A, device) || !on_device(B, device))) rc = OSSCAR_E_ARG;
    // Set-up, once per device and with that device current: the array's name is only a host-side handle;
    // kernels must be given the device address that the runtime reports for it.
    double* scratch = g_scratch_addr[device].load(std::memory_order_acquire);
    if (rc == OSSCAR_OK && !scratch) {
        double* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) rc = OSSCAR_E_CUDA;
        else { g_scratch_addr[device].store(p, std::memory_order_release); scratch = p; }
    }
    if (rc == OSSCAR_OK) {
        cudaStream_t st = (cudaStream_t)cuda_stream;
        double* partial = scratch;
        double* total = partial + OSSCAR_NOALLOC_MAX_ROWS;
        if (rows > 0 && cols > 0) k_noalloc_rows<<<(unsigned)rows, 256, 0, st>>>(A, lda, B, ldb, cols, partial);
        k_noalloc_total<<<1, 1024, 0, st>>>(partial, (rows > 0 && cols > 0) ? rows : 0, total);
        osscar::g_launches += (rows > 0 && cols > 0) ? 2 : 1;
        if (cudaGetLastError() != cudaSuccess
            || cudaMemcpyAsync(out, total, sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess
            || cudaStreamSynchronize(st) != cudaSuccess)
            rc = OSSCAR_E_CUDA;
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
