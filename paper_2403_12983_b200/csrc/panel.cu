// Products of a large streamed matrix with a narrow panel, for the block exchange of the swap search:
//   Y[i][e] = sum_k A[i][k] * P[e][k]      A: M x K (row-major, streamed once), P: N x K panel.
// fp32 on the CUDA cores.  A block owns BM rows of A and up to 128 columns, so A is read once per 128 columns;
// the panel comes from L2.  Threads form a TX x TY grid (TY = N_pad / 8, TX = BM / 4): a thread owns 4 consecutive
// rows and 8 consecutive columns (32 accumulators), and reads both operands of a k-step as 16-byte shared-memory
// loads from k-major tiles.
#include "osscar_internal.cuh"

namespace osscar {
namespace {

constexpr int PD_BK = 32;

// With gridDim.z > 1 slice z of the k range (kc wide) writes its partial sums to part[z][M][N] instead of Y.
template <int TY, int BM>
__global__ void __launch_bounds__(TY * BM / 4)
k_panel_dot(int64_t M, int N, int64_t Kfull, int64_t kc, const float* __restrict__ A, int64_t lda, const float* __restrict__ P, int64_t ldp,
            float* __restrict__ Y, int64_t so_row, int64_t so_col, float* __restrict__ part, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t kbeg = (int64_t)blockIdx.z * kc;
    const int64_t K = Kfull < kbeg + kc ? Kfull : kbeg + kc;     // end of this slice
    constexpr int TX = BM / 4, NT = TX * TY, NP = TY * 8, AS = BM + 4, PS = NP + 4;
    constexpr int AL = (BM * 8 + NT - 1) / NT, PL = (NP * 8 + NT - 1) / NT;   // float4 per thread of the A tile / panel tile
    __shared__ __align__(16) float As[PD_BK][AS];
    __shared__ __align__(16) float Ps[PD_BK][PS];
    const int t = threadIdx.x, tx = t % TX, ty = t / TX;
    const int64_t m0 = (int64_t)blockIdx.x * BM;
    const int n0 = blockIdx.y * NP;

    float acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float4 ra[AL], rp[PL];
    const bool vec = (lda % 4 == 0) && (ldp % 4 == 0) && (((uintptr_t)A & 15) == 0) && (((uintptr_t)P & 15) == 0);
    auto load4 = [&](const float* src, int64_t gk) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vec && gk + 3 < K) v = *reinterpret_cast<const float4*>(src);
        else {
            if (gk < K) v.x = src[0];
            if (gk + 1 < K) v.y = src[1];
            if (gk + 2 < K) v.z = src[2];
            if (gk + 3 < K) v.w = src[3];
        }
        return v;
    };
    auto load_tiles = [&](int64_t k0) {
#pragma unroll
        for (int i = 0; i < AL; ++i) {
            const int idx = t + i * NT, row = idx >> 3, k4 = (idx & 7) * 4;
            const int64_t gm = m0 + row, gk = k0 + k4;
            ra[i] = (idx < BM * 8 && gm < M) ? load4(A + gm * lda + gk, gk) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int i = 0; i < PL; ++i) {
            const int idx = t + i * NT, n = idx >> 3, k4 = (idx & 7) * 4;
            const int64_t gk = k0 + k4;
            rp[i] = (idx < NP * 8 && n0 + n < N) ? load4(P + (int64_t)(n0 + n) * ldp + gk, gk) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto store_tiles = [&]() {
#pragma unroll
        for (int i = 0; i < AL; ++i) {
            const int idx = t + i * NT, row = idx >> 3, k4 = (idx & 7) * 4;
            if (idx >= BM * 8) continue;
            As[k4][row] = ra[i].x; As[k4 + 1][row] = ra[i].y; As[k4 + 2][row] = ra[i].z; As[k4 + 3][row] = ra[i].w;
        }
#pragma unroll
        for (int i = 0; i < PL; ++i) {
            const int idx = t + i * NT, n = idx >> 3, k4 = (idx & 7) * 4;
            if (idx >= NP * 8) continue;
            Ps[k4][n] = rp[i].x; Ps[k4 + 1][n] = rp[i].y; Ps[k4 + 2][n] = rp[i].z; Ps[k4 + 3][n] = rp[i].w;
        }
    };

    load_tiles(kbeg);
    for (int64_t k0 = kbeg; k0 < K; k0 += PD_BK) {
        store_tiles();
        __syncthreads();
        if (k0 + PD_BK < K) load_tiles(k0 + PD_BK);
#pragma unroll
        for (int kk = 0; kk < PD_BK; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][tx * 4]);
            const float4 p0 = *reinterpret_cast<const float4*>(&Ps[kk][ty * 8]);
            const float4 p1 = *reinterpret_cast<const float4*>(&Ps[kk][ty * 8 + 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc[i][0] = fmaf(a[i], p0.x, acc[i][0]); acc[i][1] = fmaf(a[i], p0.y, acc[i][1]);
                acc[i][2] = fmaf(a[i], p0.z, acc[i][2]); acc[i][3] = fmaf(a[i], p0.w, acc[i][3]);
                acc[i][4] = fmaf(a[i], p1.x, acc[i][4]); acc[i][5] = fmaf(a[i], p1.y, acc[i][5]);
                acc[i][6] = fmaf(a[i], p1.z, acc[i][6]); acc[i][7] = fmaf(a[i], p1.w, acc[i][7]);
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t gm = m0 + tx * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int gn = n0 + ty * 8 + j;
            if (gn >= N) continue;
            if (gridDim.z > 1) part[((int64_t)blockIdx.z * M + gm) * N + gn] = acc[i][j];
            else Y[gm * so_row + (int64_t)gn * so_col] = acc[i][j];
        }
    }
}

// Y = sum over the k slices, added in slice order (deterministic).
__global__ void k_panel_reduce(const float* __restrict__ part, int64_t M, int N, int splits, float* __restrict__ Y,
                               int64_t so_row, int64_t so_col, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t total = M * N;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int z = 0; z < splits; ++z) s += part[(int64_t)z * total + idx];
        Y[(idx / N) * so_row + (idx % N) * so_col] = s;
    }
}

template <int TY>
void launch_panel_dot(cudaStream_t st, dim3 grid, int64_t M, int N, int64_t K, int64_t kc, const float* A, int64_t lda,
                      const float* P, int64_t ldp, float* Y, int64_t so_row, int64_t so_col, float* part, const int32_t* done)
{
    k_panel_dot<TY, 64><<<grid, TY * 16, 0, st>>>(M, N, K, kc, A, lda, P, ldp, Y, so_row, so_col, part, done);
}

}  // namespace

cudaError_t panel_dot(cudaStream_t st, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                      const float* P, int64_t ldp, float* Y, int64_t so_row, int64_t so_col,
                      float* scratch, size_t scratch_floats, const int32_t* done)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    const int ntile = (int)((N + 127) / 128);
    const int ncol = (int)((N + ntile - 1) / ntile);                  // columns per tile
    const int TY = (ncol + 15) / 16 * 2;                              // 16-column steps: TY in {2, 4, ..., 16}
    const int64_t blocks = (M + 63) / 64 * ntile;
    // enough warps to fill the machine: split the k range when the rows alone give too few
    int64_t splits = (148 * 16 + blocks * (TY / 2) - 1) / (blocks * (TY / 2));
    if (splits > 16) splits = 16;
    if (splits > (K + 255) / 256) splits = (K + 255) / 256;
    if (splits < 1 || !scratch || (size_t)(splits * M * N) > scratch_floats) splits = 1;
    const int64_t kc = splits == 1 ? K : ((K + splits - 1) / splits + PD_BK - 1) / PD_BK * PD_BK;
    const dim3 grid((unsigned)((M + 63) / 64), (unsigned)ntile, (unsigned)splits);
    // the column tiles of one launch are TY * 8 wide; tile j starts at j * TY * 8
    switch (TY) {
    case 2:  launch_panel_dot<2>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 4:  launch_panel_dot<4>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 6:  launch_panel_dot<6>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 8:  launch_panel_dot<8>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 10: launch_panel_dot<10>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 12: launch_panel_dot<12>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    case 14: launch_panel_dot<14>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    default: launch_panel_dot<16>(st, grid, M, (int)N, K, kc, A, lda, P, ldp, Y, so_row, so_col, scratch, done); break;
    }
    count_launches(1);
    if (splits > 1) {
        k_panel_reduce<<<(unsigned)((M * N + 255) / 256 < 1184 ? (M * N + 255) / 256 : 1184), 256, 0, st>>>(scratch, M, (int)N, (int)splits, Y, so_row, so_col, done);
        count_launches(1);
    }
    return cudaGetLastError();
}

}  // namespace osscar
