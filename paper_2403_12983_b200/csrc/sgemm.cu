// fp32 GEMM on the CUDA cores: C = alpha * op(A) * B + beta * C, any sizes, row-major.
// Used for the fp32-accurate contractions around the search (G = H W, the block inverse of
// H_II, V, R, the Schur complements) and for the Gram matrix of fp32 activations.
#include "osscar_internal.cuh"

namespace osscar {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256;
constexpr int PADA = 4;

template <bool TA, bool TB>
__global__ void __launch_bounds__(NT)
sgemm_kernel(int64_t M, int64_t N, int64_t K, float alpha, const float* __restrict__ A, int64_t lda,
             const float* __restrict__ B, int64_t ldb, float beta, float* __restrict__ C, int64_t ldc,
             const int32_t* __restrict__ done)
{
    if (done && *done) return;
    __shared__ float As[2][BK][BM + PADA];
    __shared__ float Bs[2][BK][BN + PADA];
    const int t = threadIdx.x;
    const int tx = t & 15, ty = t >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float ra[8], rb[8];
    auto load_tiles = [&](int64_t k0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            int idx = t + i * NT;
            if (TA) {           // A stored K x M: element (kk, mm) contiguous in mm
                int kk = idx >> 7, mm = idx & 127;
                int64_t gk = k0 + kk, gm = m0 + mm;
                ra[i] = (gk < K && gm < M) ? A[gk * lda + gm] : 0.f;
            } else {            // A stored M x K: element (mm, kk) contiguous in kk
                int mm = idx >> 4, kk = idx & 15;
                int64_t gk = k0 + kk, gm = m0 + mm;
                ra[i] = (gk < K && gm < M) ? A[gm * lda + gk] : 0.f;
            }
            if (TB) {           // B stored N x K: element (nn, kk) contiguous in kk
                int nn = idx >> 4, kk = idx & 15;
                int64_t gk = k0 + kk, gn = n0 + nn;
                rb[i] = (gk < K && gn < N) ? B[gn * ldb + gk] : 0.f;
            } else {            // B stored K x N
                int kk = idx >> 7, nn = idx & 127;
                int64_t gk = k0 + kk, gn = n0 + nn;
                rb[i] = (gk < K && gn < N) ? B[gk * ldb + gn] : 0.f;
            }
        }
    };
    auto store_tiles = [&](int buf) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            int idx = t + i * NT;
            if (TA) As[buf][idx >> 7][idx & 127] = ra[i];
            else    As[buf][idx & 15][idx >> 4] = ra[i];
            if (TB) Bs[buf][idx & 15][idx >> 4] = rb[i];
            else    Bs[buf][idx >> 7][idx & 127] = rb[i];
        }
    };

    // the old tile of C is wanted only at the very end: ask for its lines now (one 128-byte line per 32 columns), so
    // that the read-modify-write of a short product (rank-64 updates of the exchange inversion) finds them in L2
    if (beta != 0.f && (tx & 7) == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int64_t gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
            if (gm >= M) continue;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t gn = n0 + h * 64 + tx * 4;
                if (gn < N) asm volatile("prefetch.global.L2 [%0];" ::"l"(C + gm * ldc + gn));
            }
        }
    }

    load_tiles(0);
    store_tiles(0);
    __syncthreads();
    int buf = 0;
    for (int64_t k0 = 0; k0 < K; k0 += BK) {
        const bool more = k0 + BK < K;
        if (more) load_tiles(k0 + BK);
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[8], b[8];
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][64 + tx * 4]);
            a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
            b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (more) {
            store_tiles(buf ^ 1);
            __syncthreads();
            buf ^= 1;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t gn = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (gn >= N) continue;
            float* p = C + gm * ldc + gn;
            const float v = alpha * acc[i][j];
            *p = (beta == 0.f) ? v : fmaf(beta, *p, v);
        }
    }
}

}  // namespace

cudaError_t sgemm(cudaStream_t st, bool transA, bool transB, int64_t M, int64_t N, int64_t K,
                  float alpha, const float* A, int64_t lda, const float* B, int64_t ldb,
                  float beta, float* C, int64_t ldc, const int32_t* done)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
    count_launches(1);
    if (transA && transB) return cudaErrorInvalidValue;
    if (transA)      sgemm_kernel<true, false><<<grid, NT, 0, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, done);
    else if (transB) sgemm_kernel<false, true><<<grid, NT, 0, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, done);
    else             sgemm_kernel<false, false><<<grid, NT, 0, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, done);
    return cudaGetLastError();
}

}  // namespace osscar
