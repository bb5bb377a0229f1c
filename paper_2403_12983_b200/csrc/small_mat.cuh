// Block-cooperative small dense algebra in fp64 (g x g matrices in shared or global memory) and warp sums,
// shared by the search and the greedy phase.
#pragma once
#include <float.h>

namespace osscar {
namespace smallmat {

static __device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
static __device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// Block-cooperative Cholesky inverse of the g x g SPD matrix M (ld g, overwritten by its factor).
// Lw, Out: g x g work / result.  Returns the smallest pivot (<= 0 when not positive definite).
static __device__ double chol_inverse(double* M, double* Lw, double* Out, int g)
{
    __shared__ double minpiv;
    const int t = threadIdx.x, nt = blockDim.x;
    if (t == 0) minpiv = DBL_MAX;
    __syncthreads();
    for (int j = 0; j < g; ++j) {
        if (t == 0) {
            double dd = M[j * g + j];
            if (dd < minpiv) minpiv = dd;
            if (!(dd > 0.0)) { minpiv = -1.0; dd = 1.0; }
            M[j * g + j] = sqrt(dd);
        }
        __syncthreads();
        const double djj = M[j * g + j];
        for (int i = j + 1 + t; i < g; i += nt) M[i * g + j] /= djj;
        __syncthreads();
        const int rem = g - j - 1;
        for (int idx = t; idx < rem * rem; idx += nt) {
            const int i = j + 1 + idx / rem, c = j + 1 + idx % rem;
            if (c <= i) M[i * g + c] -= M[i * g + j] * M[c * g + j];
        }
        __syncthreads();
    }
    for (int c = t; c < g; c += nt) {
        for (int i = 0; i < g; ++i) {
            double s = (i == c) ? 1.0 : 0.0;
            for (int kx = c; kx < i; ++kx) s -= M[i * g + kx] * Lw[kx * g + c];
            Lw[i * g + c] = (i < c) ? 0.0 : s / M[i * g + i];
        }
    }
    __syncthreads();
    for (int idx = t; idx < g * g; idx += nt) {
        const int i = idx / g, j = idx % g;
        double s = 0.0;
        for (int kx = (i > j ? i : j); kx < g; ++kx) s += Lw[kx * g + i] * Lw[kx * g + j];
        Out[idx] = s;
    }
    __syncthreads();
    return minpiv;
}
// C = op(A) * op(B), all g x g, block-cooperative.
static __device__ void mat_mul(const double* A, bool tA, const double* B, bool tB, double* C, int g)
{
    for (int idx = threadIdx.x; idx < g * g; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        double s = 0.0;
        for (int kx = 0; kx < g; ++kx)
            s += (tA ? A[kx * g + i] : A[i * g + kx]) * (tB ? B[j * g + kx] : B[kx * g + j]);
        C[idx] = s;
    }
    __syncthreads();
}
static __device__ double mat_trace_prod(const double* A, const double* B, int g, double* red)   // sum A .* B^T = Tr(A B)
{
    double s = 0.0;
    for (int idx = threadIdx.x; idx < g * g; idx += blockDim.x) s += A[idx] * B[(idx % g) * g + idx / g];
    s = warp_sum(s);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    double tot = 0.0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += red[i];
    __syncthreads();
    return tot;
}


}  // namespace smallmat
}  // namespace osscar
