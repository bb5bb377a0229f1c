// C = beta * C0 + alpha * A * B with fp32 operands and every product and sum in fp64 (fp64 tensor-core path, mma m8n8k4).
//
// Why it exists.  The search state is the solution of normal equations: V = (H_II)^-1 G_I (Eq. tmp5), the residual
// R = G_J - H_JI V and the Schur complements H_qq - H_qI (H_II)^-1 H_Iq (Case 2 of Proposition 1) are small differences
// of large sums, and the scores ||R_q||^2 / c_q of Eq. impact are compared between candidates that differ by 1e-4
// relative.  Products accumulated in fp32 leave errors of cond(H_II) * 2^-24 in them (measured 4e-4 in the add scores of
// an OPT-1.3B-shaped FC2 layer), enough to change the selected group.  With the residuals of one refinement step
// (I - H_II Hinv, G_I - H_II V) and the two differences themselves accumulated in fp64, the state that is then stored
// in fp32 is correct to the rounding of its entries.
//
// Tiling: block 128 x 64, k-step 16, 8 warps of 32 x 32 (4 x 4 mma tiles, 32 fp64 accumulators per lane).  Operands
// are converted to fp64 once, on their way into shared memory; fragments are 8-byte shared loads without bank conflicts
// (row strides 20 and 68 doubles).  Global loads of the next k-step are in flight while the current one is multiplied.
#include "osscar_internal.cuh"

namespace osscar {
namespace {

constexpr int DG_BM = 128, DG_BN = 64, DG_BK = 16, DG_T = 256;
constexpr int DG_AS = DG_BK + 4;      // row stride of the A tile (doubles)
constexpr int DG_BS = DG_BN + 4;      // row stride of the B tile (doubles)

__device__ __forceinline__ void dmma(double& d0, double& d1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
}

// four consecutive floats of a row, zero beyond `limit` (elements [c, c + 4) of a row whose valid length is `limit`)
__device__ __forceinline__ float4 load4_guard(const float* __restrict__ row, int64_t c, int64_t limit, bool vec)
{
    if (vec && c + 3 < limit) return *reinterpret_cast<const float4*>(row + c);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < limit) v.x = row[c];
    if (c + 1 < limit) v.y = row[c + 1];
    if (c + 2 < limit) v.z = row[c + 2];
    if (c + 3 < limit) v.w = row[c + 3];
    return v;
}

// mode 0: C = beta * C0 + alpha * A B (C0 may alias C);  mode 1: C = I + alpha * A B (C0 unused).  OutT float or double.
// tri (B square and symmetric, K = N): B is replaced by its block upper triangle U with the 64 x 64 diagonal blocks
// halved, B = U + U^T, so that x^T B x = 2 x^T U x needs only the k-range [0, n0 + 64) of every column tile: half the
// flops when only such quadratic forms of the rows of A are wanted (the Schur complements of single-row groups).
template <typename OutT>
__global__ void __launch_bounds__(DG_T, 2)
k_gemm_f64acc(int64_t M, int64_t N, int64_t K, double alpha, const float* __restrict__ A, int64_t lda,
              const float* __restrict__ B, int64_t ldb, double beta, const float* C0, int64_t ldc0,
              OutT* C, int64_t ldc, int mode, int vecA, int vecB, int tri, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    extern __shared__ double dg_smem[];
    double* As[2] = { dg_smem, dg_smem + DG_BM * DG_AS };
    double* Bs[2] = { dg_smem + 2 * DG_BM * DG_AS, dg_smem + 2 * DG_BM * DG_AS + DG_BK * DG_BS };
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp >> 1, wn = warp & 1;                   // 4 x 2 warps of 32 x 32
    const int64_t m0 = (int64_t)blockIdx.y * DG_BM, n0 = (int64_t)blockIdx.x * DG_BN;
    // loader roles: A tile 128 x 16 floats = 2 float4 per thread, B tile 16 x 64 floats = 1 float4 per thread
    const int ar = tid >> 2, ac = (tid & 3) * 4;               // rows ar and ar + 64, columns ac .. ac + 3
    const int br = tid >> 4, bc = (tid & 15) * 4;
    const int64_t arow0 = m0 + ar, arow1 = m0 + ar + 64;
    const float* Ar0 = A + (arow0 < M ? arow0 : M - 1) * lda;
    const float* Ar1 = A + (arow1 < M ? arow1 : M - 1) * lda;
    const bool a0ok = arow0 < M, a1ok = arow1 < M;

    double acc[4][4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j][0] = 0.0; acc[i][j][1] = 0.0; }

    const int64_t kend = tri && n0 + DG_BN < K ? n0 + DG_BN : K;
    const int nk = (int)((kend + DG_BK - 1) / DG_BK);
    float4 ra0, ra1, rb;
    auto fetch = [&](int kt) {
        const int64_t k0 = (int64_t)kt * DG_BK;
        ra0 = a0ok ? load4_guard(Ar0, k0 + ac, K, vecA) : make_float4(0.f, 0.f, 0.f, 0.f);
        ra1 = a1ok ? load4_guard(Ar1, k0 + ac, K, vecA) : make_float4(0.f, 0.f, 0.f, 0.f);
        const int64_t kr = k0 + br;
        rb = kr < K ? load4_guard(B + kr * ldb, n0 + bc, N, vecB) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (tri && kr >= n0) { rb.x *= 0.5f; rb.y *= 0.5f; rb.z *= 0.5f; rb.w *= 0.5f; }      // rows of the diagonal block, exact in fp32
    };
    auto stash = [&](int buf) {
        double* a = As[buf]; double* b = Bs[buf];
        a[ar * DG_AS + ac + 0] = (double)ra0.x; a[ar * DG_AS + ac + 1] = (double)ra0.y;
        a[ar * DG_AS + ac + 2] = (double)ra0.z; a[ar * DG_AS + ac + 3] = (double)ra0.w;
        a[(ar + 64) * DG_AS + ac + 0] = (double)ra1.x; a[(ar + 64) * DG_AS + ac + 1] = (double)ra1.y;
        a[(ar + 64) * DG_AS + ac + 2] = (double)ra1.z; a[(ar + 64) * DG_AS + ac + 3] = (double)ra1.w;
        b[br * DG_BS + bc + 0] = (double)rb.x; b[br * DG_BS + bc + 1] = (double)rb.y;
        b[br * DG_BS + bc + 2] = (double)rb.z; b[br * DG_BS + bc + 3] = (double)rb.w;
    };
    fetch(0);
    stash(0);
    __syncthreads();
    const int fr = lane >> 2, fk = lane & 3;                   // fragment row / column index, k index inside a k4 step
    for (int kt = 0; kt < nk; ++kt) {
        const int buf = kt & 1;
        if (kt + 1 < nk) fetch(kt + 1);
        const double* a = As[buf] + (wm * 32) * DG_AS;
        const double* b = Bs[buf] + wn * 32;
#pragma unroll
        for (int ks = 0; ks < DG_BK; ks += 4) {
            double af[4], bf[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) af[i] = a[(i * 8 + fr) * DG_AS + ks + fk];
#pragma unroll
            for (int j = 0; j < 4; ++j) bf[j] = b[(ks + fk) * DG_BS + j * 8 + fr];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) dmma(acc[i][j][0], acc[i][j][1], af[i], bf[j]);
        }
        if (kt + 1 < nk) stash(buf ^ 1);
        __syncthreads();
    }
    // lane holds C[fr][2 fk], C[fr][2 fk + 1] of every 8 x 8 tile
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = m0 + wm * 32 + i * 8 + fr;
        if (row >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t col = n0 + wn * 32 + j * 8 + 2 * fk;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (col + e >= N) continue;
                double v = alpha * acc[i][j][e];
                if (mode == 1) v += (row == col + e) ? 1.0 : 0.0;
                else if (beta != 0.0) v += beta * (double)C0[row * ldc0 + col + e];
                C[row * ldc + col + e] = (OutT)v;
            }
        }
    }
}

}  // namespace

cudaError_t gemm_f64acc(cudaStream_t st, int64_t M, int64_t N, int64_t K, double alpha, const float* A, int64_t lda,
                        const float* B, int64_t ldb, double beta, const float* C0, int64_t ldc0, float* C, int64_t ldc,
                        bool identity_plus, const int32_t* done)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    const int vecA = (((uintptr_t)A & 15) == 0 && (lda % 4) == 0) ? 1 : 0;
    const int vecB = (((uintptr_t)B & 15) == 0 && (ldb % 4) == 0) ? 1 : 0;
    dim3 grid((unsigned)((N + DG_BN - 1) / DG_BN), (unsigned)((M + DG_BM - 1) / DG_BM));
    constexpr int smem = (2 * DG_BM * DG_AS + 2 * DG_BK * DG_BS) * (int)sizeof(double);
    cudaError_t e = cudaFuncSetAttribute(k_gemm_f64acc<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    k_gemm_f64acc<float><<<grid, DG_T, smem, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc0, C, ldc, identity_plus ? 1 : 0, vecA, vecB, 0, done);
    count_launches(1);
    return cudaGetLastError();
}

// The plain product with the result kept in fp64: C (M x N doubles, row stride ldc) = A * B; with `tri` (B symmetric,
// K == N) C = A * U for the halved block upper triangle U of B (see the kernel).
cudaError_t gemm_f64out(cudaStream_t st, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                        const float* B, int64_t ldb, double* C, int64_t ldc, const int32_t* done, bool tri)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    if (tri && K != N) return cudaErrorInvalidValue;
    const int vecA = (((uintptr_t)A & 15) == 0 && (lda % 4) == 0) ? 1 : 0;
    const int vecB = (((uintptr_t)B & 15) == 0 && (ldb % 4) == 0) ? 1 : 0;
    dim3 grid((unsigned)((N + DG_BN - 1) / DG_BN), (unsigned)((M + DG_BM - 1) / DG_BM));
    constexpr int smem = (2 * DG_BM * DG_AS + 2 * DG_BK * DG_BS) * (int)sizeof(double);
    cudaError_t e = cudaFuncSetAttribute(k_gemm_f64acc<double>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    k_gemm_f64acc<double><<<grid, DG_T, smem, st>>>(M, N, K, 1.0, A, lda, B, ldb, 0.0, nullptr, 0, C, ldc, 0, vecA, vecB, tri ? 1 : 0, done);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace osscar
