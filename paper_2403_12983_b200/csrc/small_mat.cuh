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
// Block-cooperative inverse of the g x g SPD matrix M (ld g) by in-place Gauss-Jordan elimination without pivoting:
// g steps of one rank-1 update over all g^2 entries, so every thread of the block works in every step.
// M is overwritten (keep it in shared memory where possible); Out receives the symmetrised inverse; Lw: scratch of
// at least 2 g doubles.  Returns the smallest pivot, i.e. the smallest diagonal entry of the successive Schur
// complements = the squared diagonal of the Cholesky factor (<= 0 when M is not positive definite).
static __device__ double spd_inverse(double* M, double* Lw, double* Out, int g)
{
    __shared__ double minpiv;
    const int t = threadIdx.x, nt = blockDim.x;
    double* colj = Lw; double* rowj = Lw + g;
    __syncthreads();
    if (t == 0) minpiv = DBL_MAX;
    __syncthreads();
    for (int j = 0; j < g; ++j) {
        double d = M[j * g + j];
        const bool bad = !(d > 0.0);
        if (t == 0) { if (bad) minpiv = -1.0; else if (d < minpiv) minpiv = d; }
        if (bad) d = 1.0;
        const double pinv = 1.0 / d;
        for (int i = t; i < g; i += nt) { colj[i] = M[i * g + j]; rowj[i] = M[j * g + i] * pinv; }
        __syncthreads();
        for (int idx = t; idx < g * g; idx += nt) {
            const int i = idx / g, c = idx % g;
            double v;
            if (i == j) v = (c == j) ? pinv : rowj[c];
            else if (c == j) v = -colj[i] * pinv;
            else v = M[idx] - colj[i] * rowj[c];
            M[idx] = v;
        }
        __syncthreads();
    }
    for (int idx = t; idx < g * g; idx += nt) {          // the two triangles differ by rounding only
        const int i = idx / g, c = idx % g;
        Out[idx] = 0.5 * (M[idx] + M[c * g + i]);
    }
    __syncthreads();
    return minpiv;
}
// C = op(A) * op(B), all g x g (ld g), block-cooperative, on the fp64 tensor-core path: every warp of the block takes
// 8 x 8 tiles of C in turn and runs g / 4 steps of mma.m8n8k4 (A fragment: row lane / 4, column lane % 4; B fragment:
// row lane % 4, column lane / 4; C fragment: row lane / 4, columns 2 (lane % 4) and + 1).  Entries beyond g read as 0.
// C must not overlap A or B.  blockDim.x must be a multiple of 32.
static __device__ void mat_mul(const double* A, bool tA, const double* B, bool tB, double* C, int g)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int nt = (g + 7) >> 3;
    const int r4 = lane >> 2, c4 = lane & 3;
    for (int tile = warp; tile < nt * nt; tile += nwarps) {
        const int i0 = (tile / nt) * 8, j0 = (tile % nt) * 8;
        const int ai = i0 + r4, bj = j0 + r4;
        double d0 = 0.0, d1 = 0.0;
        for (int k0 = 0; k0 < g; k0 += 4) {
            const int kk = k0 + c4;
            const bool ka = kk < g;
            const double a = (ka && ai < g) ? (tA ? A[kk * g + ai] : A[ai * g + kk]) : 0.0;
            const double b = (ka && bj < g) ? (tB ? B[bj * g + kk] : B[kk * g + bj]) : 0.0;
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                         : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
        }
        const int ci = i0 + r4, cj = j0 + 2 * c4;
        if (ci < g) {
            if (cj < g) C[ci * g + cj] = d0;
            if (cj + 1 < g) C[ci * g + cj + 1] = d1;
        }
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
