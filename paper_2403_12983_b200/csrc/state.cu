// Starting support and construction of the search state for a given support:
// slot-permuted copy of H, (H_II)^-1 by an in-place blocked exchange (Gauss-Jordan) inversion,
// V = (H_II)^-1 G_I (Eq. tmp5), residual R, Schur complements c (Case 2 of Proposition 1).
#include "osscar_internal.cuh"
#include <math.h>

namespace osscar {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// Block-wide sum (blockDim.x multiple of 32, <= 1024); result valid in thread 0.
__device__ double block_sum(double v) {
    __shared__ double red[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    if (w == 0) {
        v = (lane < (int)((blockDim.x + 31) >> 5)) ? red[lane] : 0.0;
        v = warp_sum(v);
    }
    return v;
}

// e_q = Tr(W_q^T H_qq W_q) (mode 0) or ||W_q||_F^2 (mode 1); one block per group.
__global__ void k_energy(const float* __restrict__ H, const float* __restrict__ W, int64_t d1, int64_t m,
                         int g, int mode, double* __restrict__ e)
{
    const int64_t q = blockIdx.x;
    const float* Wq = W + q * g * m;
    double acc = 0.0;
    for (int64_t c = threadIdx.x; c < m; c += blockDim.x) {
        if (mode == OSSCAR_INIT_MAGNITUDE) {
            for (int a = 0; a < g; ++a) { double w = Wq[a * m + c]; acc += w * w; }
        } else {
            for (int a = 0; a < g; ++a) {
                double t = 0.0;
                const float* Hrow = H + (q * g + a) * d1 + q * g;
                for (int b = 0; b < g; ++b) t += (double)Hrow[b] * (double)Wq[b * m + c];
                acc += (double)Wq[a * m + c] * t;
            }
        }
    }
    acc = block_sum(acc);
    if (threadIdx.x == 0) e[q] = acc;
}

// kept[q] = 1 iff fewer than k groups beat q (larger energy, or equal energy and smaller id).
__global__ void k_rank_select(const double* __restrict__ e, int64_t ng, int k, int32_t* __restrict__ kept)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= ng) return;
    const double eq = e[q];
    int rank = 0;
    for (int64_t p = 0; p < ng; ++p) {
        const double ep = e[p];
        rank += (ep > eq) || (ep == eq && p < q);
    }
    kept[q] = rank < k;
}

__global__ void k_user_support(const int32_t* __restrict__ support, int k, int64_t ng,
                               int32_t* __restrict__ kept, SearchCtl* ctl)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= k) return;
    const int q = support[i];
    if (q < 0 || q >= ng) { ctl->status = OSSCAR_E_ARG; return; }
    if (atomicExch(&kept[q], 1) != 0) ctl->status = OSSCAR_E_ARG;   // duplicate id
}

// After k_user_support: a list that was rejected (id out of range, duplicate) marks fewer than k groups.  The kernels
// that follow index H and G through the slot permutation, so the marks are replaced by a valid set (the first k
// groups) and the error stays in ctl->status; nothing downstream can then leave its buffers.  One block.
__global__ void __launch_bounds__(1024) k_user_support_guard(int32_t* __restrict__ kept, int64_t ng, int k, SearchCtl* ctl)
{
    __shared__ int cnt;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    int local = 0;
    for (int64_t q = threadIdx.x; q < ng; q += blockDim.x) local += kept[q] != 0;
    if (local) atomicAdd(&cnt, local);
    __syncthreads();
    if (ctl->status == OSSCAR_OK && cnt == k) return;
    for (int64_t q = threadIdx.x; q < ng; q += blockDim.x) kept[q] = q < k;
    if (threadIdx.x == 0 && ctl->status == OSSCAR_OK) ctl->status = OSSCAR_E_ARG;
}

// Slots: kept groups in ascending id order take slots 0..k-1, pruned groups k..ng-1.
__global__ void k_build_perm(const int32_t* __restrict__ kept, int64_t ng, int k,
                             int32_t* __restrict__ perm, int32_t* __restrict__ slotof,
                             int32_t* __restrict__ support)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= ng) return;
    int before_kept = 0;
    for (int64_t p = 0; p < q; ++p) before_kept += kept[p];
    const int slot = kept[q] ? before_kept : k + (int)(q - before_kept);
    if (slot < 0 || slot >= ng || (kept[q] && slot >= k)) return;       // cannot happen with exactly k marks
    perm[slot] = (int32_t)q;
    slotof[q] = slot;
    if (kept[q]) support[slot] = (int32_t)q;
}

// Hp[i][j] = H[row(i)][row(j)], row(i) = perm[i / g] * g + i % g.
__global__ void k_gather_sym(const float* __restrict__ H, int64_t d1, int g, const int32_t* __restrict__ perm,
                             float* __restrict__ Hp, int64_t ldp)
{
    const int64_t i = blockIdx.x;
    const int64_t ri = (int64_t)perm[i / g] * g + i % g;
    for (int64_t j = (int64_t)blockIdx.y * blockDim.x + threadIdx.x; j < ldp; j += (int64_t)gridDim.y * blockDim.x) {
        float v = 0.f;
        if (j < d1) {
            const int64_t rj = (int64_t)perm[j / g] * g + j % g;
            v = H[ri * d1 + rj];
        }
        Hp[i * ldp + j] = v;
    }
}

// dst[i][0..ld) = src[row(slot0*g + i)][0..m) zero-padded, for i in [0, nrows).
__global__ void k_gather_rows(const float* __restrict__ src, int64_t m, int g, const int32_t* __restrict__ perm,
                              int64_t slot_row0, float* __restrict__ dst, int64_t ld)
{
    const int64_t i = blockIdx.x;
    const int64_t s = slot_row0 + i;
    const float* row = src + ((int64_t)perm[s / g] * g + s % g) * m;
    for (int64_t c = threadIdx.x; c < ld; c += blockDim.x) dst[i * ld + c] = c < m ? row[c] : 0.f;
}

// dst (rows x ldd, zero padded) = src[0:rows, 0:cols] (lds)
__global__ void k_copy_pad(const float* __restrict__ src, int64_t lds, int64_t rows, int64_t cols,
                           float* __restrict__ dst, int64_t ldd)
{
    const int64_t i = blockIdx.x;
    for (int64_t c = threadIdx.x; c < ldd; c += blockDim.x) dst[i * ldd + c] = c < cols ? src[i * lds + c] : 0.f;
}

// ---------------------------------------------------------------- blocked exchange inversion
constexpr int NB = 64;
constexpr double kPivotRelTol = 1e-7;

// Inverse of the nb x nb pivot block A[p0:p0+nb, p0:p0+nb] in fp64 (one block of 1024 threads): Gauss-Jordan
// elimination without pivoting with the block held in registers.  Thread (i, cb) = (t / 16, t % 16) owns the entries
// (i, cb + 16 k), k = 0..3.  In step j every thread fetches its row's entry of column j by a shuffle inside its
// half-warp, the threads of row j publish the scaled pivot row through shared memory (double-buffered: one barrier per
// step), and every entry takes its rank-1 update.  The pivots are the diagonal of the successive Schur complements
// (the squared diagonal of the Cholesky factor).  Raises OSSCAR_E_NOTPD in ctl->status when a pivot is not positive.
__global__ void __launch_bounds__(1024)
k_pivot_inverse(const float* __restrict__ A, int64_t lda, int64_t p0, int nb, float* __restrict__ Dinv,
                const float* __restrict__ Hp, int64_t ldp, SearchCtl* ctl)
{
    static_assert(NB == 64, "thread layout of the pivot inverse");
    __shared__ double rowj[2][NB];
    __shared__ double pinv_s[2];
    __shared__ double hdiag[NB];         // diagonal of the original matrix: scale of the pivot test
    __shared__ double Ls[NB][NB + 1];    // the finished inverse, for the symmetrised write
    __shared__ int bad;
    const int t = threadIdx.x, i = t >> 4, cb = t & 15, lane = t & 31;
    double Lr[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int c = cb + 16 * k;
        // symmetrise: the two triangles can differ in the last bits
        Lr[k] = (i < nb && c < nb) ? 0.5 * ((double)A[(p0 + i) * lda + p0 + c] + (double)A[(p0 + c) * lda + p0 + i]) : 0.0;
    }
    if (t == 0) bad = 0;
    if (t < nb) hdiag[t] = (double)Hp[(p0 + t) * ldp + p0 + t];
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        for (int jj = 0; jj < 16; ++jj) {
            const int j = kk * 16 + jj;
            if (j >= nb) break;
            const int buf = j & 1;
            const double x = __shfl_sync(0xffffffffu, Lr[kk], (lane & 16) | jj);     // entry (i, j) of this thread's row
            if (i == j) {
                double d = x;
                // a pivot that fp32 data cannot tell from zero counts as not positive
                if (!(d > kPivotRelTol * hdiag[j])) { if (cb == 0) bad = 1; d = 1.0; }
                const double pinv = 1.0 / d;
#pragma unroll
                for (int k = 0; k < 4; ++k) rowj[buf][cb + 16 * k] = Lr[k] * pinv;
                if (cb == 0) pinv_s[buf] = pinv;
            }
            __syncthreads();
            const double pinv = pinv_s[buf];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int c = cb + 16 * k;
                const double r = rowj[buf][c];
                double v;
                if (i == j) v = (c == j) ? pinv : r;
                else if (c == j) v = -x * pinv;
                else v = Lr[k] - x * r;
                Lr[k] = v;
            }
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) Ls[i][cb + 16 * k] = Lr[k];
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {                  // the two triangles differ by rounding only
        const int c = cb + 16 * k;
        if (i < nb && c < nb) Dinv[i * NB + c] = (float)(0.5 * (Ls[i][c] + Ls[c][i]));
    }
    if (t == 0 && bad && ctl->status == OSSCAR_OK) ctl->status = OSSCAR_E_NOTPD;       // the first error is the one reported
}

// U = A[p0:p0+nb, 0:n) (copy of the pivot rows), and zero T's pivot rows afterwards is done in k_zero_rows.
__global__ void k_copy_rows(const float* __restrict__ A, int64_t lda, int64_t p0, int nb, int64_t n,
                            float* __restrict__ U, int64_t ldu)
{
    const int i = blockIdx.y;
    if (i >= nb) return;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < n; c += (int64_t)gridDim.x * blockDim.x)
        U[i * ldu + c] = A[(p0 + i) * lda + c];
}
__global__ void k_zero_rows(float* __restrict__ T, int64_t ldt, int64_t p0, int nb, int ncols)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < nb * ncols) T[(p0 + idx / ncols) * ldt + idx % ncols] = 0.f;
}
// A[:, P] = T (rows outside P), A[P, :] = Un (columns outside P), A[P, P] = Dinv.
__global__ void k_gj_writeback(float* __restrict__ A, int64_t lda, int64_t n, int64_t p0, int nb,
                               const float* __restrict__ T, int64_t ldt, const float* __restrict__ Un, int64_t ldu,
                               const float* __restrict__ Dinv)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n * nb) return;
    {   // column panel: element (row, p0 + j)
        const int64_t row = idx / nb; const int j = (int)(idx % nb);
        if (row < p0 || row >= p0 + nb) A[row * lda + p0 + j] = T[row * ldt + j];
    }
    {   // row panel: element (p0 + i, col)
        const int i = (int)(idx / n); const int64_t col = idx % n;
        float v;
        if (col >= p0 && col < p0 + nb) v = Dinv[i * NB + (col - p0)];
        else v = Un[i * ldu + col];
        A[(p0 + i) * lda + col] = v;
    }
}

// c_t[a][b] = Hp[J_ta][J_tb] - twice * sum_s Pm[ta][s] * Hp[J_tb][s]  for pruned slot t; one block per t.
// Pm holds the rows of the pruned slots [t0, t0 + gridDim.x) in fp64 (row stride ldpm): H_JI Hinv (twice = 1), or, for
// single-row groups, H_JI U with U the halved block upper triangle of Hinv (twice = 2: h^T Hinv h = 2 h^T U h).
__global__ void k_schur(const float* __restrict__ Hp, int64_t ldp, const double* __restrict__ Pm, int64_t ldpm,
                        int64_t nI, int g, double* __restrict__ c, int64_t t0, double twice, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t t = t0 + blockIdx.x;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int pair = w; pair < g * g; pair += nw) {
        const int a = pair / g, b = pair % g;
        const double* pr = Pm + ((t - t0) * g + a) * ldpm;
        const float* hr = Hp + (nI + t * g + b) * ldp;
        double s = 0.0;
        for (int64_t x = lane; x < nI; x += 32) s = fma(pr[x], (double)hr[x], s);
        s = warp_sum(s);
        if (lane == 0) c[(t * g + a) * g + b] = (double)Hp[(nI + t * g + a) * ldp + nI + t * g + b] - twice * s;
    }
}

// Two deterministic stages: per-block partial sums, then one block adds them in a fixed order.
__global__ void k_trace_product(const float* __restrict__ A, int64_t lda, const float* __restrict__ B, int64_t ldb,
                                int64_t rows, int64_t cols, double* __restrict__ partial)
{
    double acc = 0.0;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x)
        for (int64_t c = threadIdx.x; c < cols; c += blockDim.x)
            acc += (double)A[r * lda + c] * (double)B[r * ldb + c];
    acc = block_sum(acc);
    if (threadIdx.x == 0) partial[blockIdx.x] = acc;
}
__global__ void k_sum_partials(const double* __restrict__ partial, int n, double* __restrict__ out)
{
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) acc += partial[i];
    acc = block_sum(acc);
    if (threadIdx.x == 0) *out = acc;
}

// A := sym(A + D) on the n x n leading block: the blocked inversion leaves its two triangles different in the last bits
// times cond, and the correction of that difference is the antisymmetric part of D, so both are symmetrised together.
// A thread owns the pair (r, c), (c, r) with c >= r; tiles below the diagonal have nothing to do.
__global__ void k_add_sym(float* __restrict__ A, int64_t lda, const float* __restrict__ D, int64_t ldd, int64_t n,
                          const int32_t* __restrict__ done)
{
    if (done && *done) return;
    if (blockIdx.x < blockIdx.y) return;
    const int64_t c = (int64_t)blockIdx.x * 32 + threadIdx.x;
    for (int64_t r = (int64_t)blockIdx.y * 32 + threadIdx.y; r < (int64_t)blockIdx.y * 32 + 32 && r < n; r += 8) {
        if (c >= n || c < r) continue;
        const float v = 0.5f * ((A[r * lda + c] + A[c * lda + r]) + (D[r * ldd + c] + D[c * ldd + r]));
        A[r * lda + c] = v;
        A[c * lda + r] = v;
    }
}

// acc[0], acc[1] -> sh[0], sh[1] (back = 0) or back again (back = 1)
__global__ void k_pack2(SearchCtl* ctl, double* sh, int back)
{
    if (back) { ctl->acc[0] = sh[0]; ctl->acc[1] = sh[1]; } else { sh[0] = ctl->acc[0]; sh[1] = ctl->acc[1]; }
}

__global__ void k_set_obj(SearchCtl* ctl)   // obj = const - Tr(G_I^T V), with acc[0] = const, acc[1] = trace
{
    ctl->const_term = ctl->acc[0];
    ctl->obj = ctl->acc[0] - ctl->acc[1];
}

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return OSSCAR_E_CUDA; } while (0)

}  // namespace

__global__ void k_set_double(double* dst, double v) { *dst = v; }
cudaError_t set_device_double(cudaStream_t st, double* dst, double v)
{
    k_set_double<<<1, 1, 0, st>>>(dst, v);
    count_launches(1);
    return cudaGetLastError();
}
cudaError_t gather_rows(cudaStream_t st, const float* src, int64_t m, int g, const int32_t* perm,
                        int64_t slot_row0, int64_t nrows, float* dst, int64_t ld)
{
    if (nrows > 0) { k_gather_rows<<<(unsigned)nrows, 256, 0, st>>>(src, m, g, perm, slot_row0, dst, ld); count_launches(1); }
    return cudaGetLastError();
}

cudaError_t trace_product(cudaStream_t st, const float* A, int64_t lda, const float* B, int64_t ldb,
                          int64_t rows, int64_t cols, double* partials, double* out_dev)
{
    if (rows <= 0 || cols <= 0) return cudaMemsetAsync(out_dev, 0, sizeof(double), st);
    const int grid = (int)(rows < kTracePartials ? rows : kTracePartials);
    k_trace_product<<<grid, 256, 0, st>>>(A, lda, B, ldb, rows, cols, partials);
    k_sum_partials<<<1, 256, 0, st>>>(partials, grid, out_dev);
    count_launches(2);
    return cudaGetLastError();
}

int make_layout(int64_t d1, int64_t m, int32_t g, int32_t k, Layout* L)
{
    if (d1 <= 0 || m <= 0 || g <= 0 || g > OSSCAR_MAX_GROUP || d1 % g != 0) return OSSCAR_E_SHAPE;
    const int64_t ng = d1 / g;
    if (k < 1 || k > ng) return OSSCAR_E_SHAPE;
    L->d1 = d1; L->m = m; L->ng = ng; L->g = g; L->k = k;
    L->nI = (int64_t)k * g; L->nJ = d1 - L->nI;
    L->ldp = round_up(d1, kPadF); L->ldh = round_up(L->nI, kPadF); L->ldm = round_up(m, kPadF);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
    const int64_t nI = L->nI, nJ = L->nJ, ldh = L->ldh, ldm = L->ldm;
    // `big` first: osscar_objective uses the start of the workspace as 2 * d1 * ldm floats
    int64_t big = nI * ldm;
    if (nJ * ldh > big) big = nJ * ldh;
    if (2 * d1 * ldm > big) big = 2 * d1 * ldm;
    if (2 * nI * ldh > big) big = 2 * nI * ldh;             // residual and correction of the refinement step on Hinv
    const int64_t npairs = (int64_t)k * (ng - k);
    L->pair_capacity = npairs <= kMaxPairs ? npairs : 0;
    if (L->pair_capacity > 0 && nJ * ldh + nI * round_up(nJ, kPadF) > big) big = nJ * ldh + nI * round_up(nJ, kPadF);
    {   // the nested phase keeps V of all rows plus up to 256 staged rows of Hinv (twice, and their transposes) and of V in `big`
        const int64_t gneed = d1 * ldm + 2 * 256 * L->ldp + 256 * ldm + 2 * 256 * d1;
        if (gneed > big) big = gneed;
    }
    L->off_big = take(sizeof(float) * big);
    L->off_Hp = take(sizeof(float) * d1 * L->ldp);
    L->off_Hinv = take(sizeof(float) * nI * ldh);
    L->off_Hd = take(g == 1 ? sizeof(double) * nI * ldh : 256);
    L->off_V = take(sizeof(float) * nI * ldm);
    L->off_R = take(sizeof(float) * (nJ > 0 ? nJ : 1) * ldm);
    L->off_y = take(sizeof(float) * ldh * g);
    L->off_vec_begin = L->off_y;
    L->off_b = take(sizeof(float) * ldh * g);
    L->off_u2 = take(sizeof(float) * ldh * g);
    L->off_bC = take(sizeof(float) * ldh * g);
    L->off_u2c = take(sizeof(float) * ldh * g);
    L->off_u = take(sizeof(float) * (nJ + g) * g);
    L->off_d = take(sizeof(float) * (nJ + g) * g);
    L->off_K = take(sizeof(float) * g * ldm);
    L->off_Vq = take(sizeof(float) * g * ldm);
    L->off_vec_end = off;
    L->off_vnorm = take(sizeof(float) * (nI + nJ + 1));      // row norms of V, then of R: one buffer of d1 floats (shards sum it)
    L->off_rnorm = L->off_vnorm + sizeof(float) * nI;
    L->off_shard = take(sizeof(double) * 8);
    L->off_D = take(sizeof(double) * k);
    L->off_A = take(sizeof(double) * (ng - k > 0 ? ng - k : 1));
    L->off_c = take(sizeof(double) * (ng - k > 0 ? ng - k : 1) * g * g);
    L->off_small = take(sizeof(double) * 16 * g * g + 256);
    L->off_gramV = take(sizeof(double) * k * g * g);
    L->off_gramR = take(sizeof(double) * (ng - k > 0 ? ng - k : 1) * g * g);
    L->off_perm = take(sizeof(int32_t) * ng);
    L->off_slotof = take(sizeof(int32_t) * ng);
    L->off_energy = take(sizeof(double) * ng + sizeof(int32_t) * ng);
    L->off_panel = take(sizeof(float) * (d1 * NB + 2 * NB * L->ldp + NB * NB));
    L->off_loop = take(2 * (size_t)kLoopMaxBlocks * 16 + 64);
    const size_t gg8 = sizeof(double) * g * g;
    const bool pairs_ok = L->pair_capacity > 0;
    L->off_pairCinv = take(pairs_ok ? gg8 * k : 8);
    L->off_pairKK = take(pairs_ok ? gg8 * k : 8);
    L->off_pairScratch = take(pairs_ok ? gg8 * 8 * 296 : 8);
    L->off_pairDelta = take(pairs_ok ? sizeof(double) * L->pair_capacity : 8);
    L->off_greedy = take(greedy_scratch_bytes(d1, m, g));
    {   // K panels of up to 2048 for the widest products of the state build (M <= d1, N <= max(m, n_I))
        const int64_t nmax = ldm > ldh ? ldm : ldh;
        L->tc_bytes = 3 * ((size_t)d1 * 2048 * 2 + (size_t)2048 * nmax * 2) + 16 * 1024;
        if (L->tc_bytes < gemm_tc_min_scratch(d1, nmax)) L->tc_bytes = gemm_tc_min_scratch(d1, nmax);
        L->off_tc = take(L->tc_bytes);
    }
    {   // block exchange: panels for up to min(OSSCAR_MAX_GROUP, n_I, n_J) rows on each side (a multiple of g)
        int64_t G = OSSCAR_MAX_GROUP;
        if (nI < G) G = nI;
        if (nJ < G) G = nJ;
        G = G / g * g;
        L->block_rows_max = (int32_t)G;
        const size_t n = G > 0 ? block_region_bytes(ldh, ldm, nJ, G) : 256;
        L->block_bytes = n;
        L->off_block = take(n);
    }
    L->bytes = off;
    return OSSCAR_OK;
}

int select_support(osscar_ctx* ctx, int mode, int32_t* support)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    char* ws = (char*)ctx->ws;
    double* e = (double*)(ws + L.off_energy);
    int32_t* kept = (int32_t*)(e + L.ng);
    int32_t* perm = (int32_t*)(ws + L.off_perm);
    int32_t* slotof = (int32_t*)(ws + L.off_slotof);
    const int nb = (int)((L.ng + 255) / 256);
    if (mode == OSSCAR_INIT_USER) {
        CK(cudaMemsetAsync(kept, 0, sizeof(int32_t) * L.ng, st));
        k_user_support<<<(L.k + 255) / 256, 256, 0, st>>>(support, L.k, L.ng, kept, ctx->ctl);
        k_user_support_guard<<<1, 1024, 0, st>>>(kept, L.ng, L.k, ctx->ctl);
        count_launches(1);
    } else {
        k_energy<<<(unsigned)L.ng, 128, 0, st>>>(ctx->H, ctx->W, L.d1, L.m, L.g, mode, e);
        if (ctx->reduce) { const int rr = shard_reduce(ctx, e, L.ng, OSSCAR_FP64); if (rr != OSSCAR_OK) return rr; }   // energies are sums over columns
        k_rank_select<<<nb, 256, 0, st>>>(e, L.ng, L.k, kept);
    }
    k_build_perm<<<nb, 256, 0, st>>>(kept, L.ng, L.k, perm, slotof, support);
    count_launches(mode == OSSCAR_INIT_USER ? 2 : 3);
    CK(cudaGetLastError());
    return OSSCAR_OK;
}

// In-place inverse of the n x n SPD matrix A (row stride lda) by the blocked exchange (Gauss-Jordan) scheme:
// per 64-wide pivot block an fp64 Gauss-Jordan inverse in shared memory, then one rank-64 update of the whole matrix in a GEMM.
// `ref` (row stride ldref) supplies the original diagonal, the scale of the positive-definiteness test.
// With `tensor_updates` the rank-64 updates of large matrices run on the tensor cores (three bf16 terms per operand,
// k_rank_update): their accumulation chains are 64 products long, so the truncating accumulator costs nothing that
// the correction of the inverse from an fp64 residual, which the caller then applies, does not remove.
int invert_spd_inplace(osscar_ctx* ctx, float* A, int64_t lda, int64_t n, const float* ref, int64_t ldref, const int32_t* done,
                       bool tensor_updates)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    float* T = (float*)((char*)ctx->ws + L.off_panel);
    float* U = T + L.d1 * NB;
    float* Un = U + NB * L.ldp;
    float* Dinv = Un + NB * L.ldp;
    const bool tc_updates = tensor_updates && n >= 4096 && (lda % 4) == 0 && (((uintptr_t)A & 15) == 0);
    if (tc_updates) CK(cudaMemsetAsync(U, 0, sizeof(float) * NB * lda, st));       // the pad columns of the row panel stay zero
    for (int64_t p0 = 0; p0 < n; p0 += NB) {
        const int nb = (int)(n - p0 < NB ? n - p0 : NB);
        k_pivot_inverse<<<1, 1024, 0, st>>>(A, lda, p0, nb, Dinv, ref, ldref, ctx->ctl);
        // T = A[:, P] * Dinv
        CK(sgemm(st, false, false, n, nb, nb, 1.f, A + p0, lda, Dinv, NB, 0.f, T, NB, done));
        k_zero_rows<<<(nb * nb + 255) / 256, 256, 0, st>>>(T, NB, p0, nb, nb);
        {
            dim3 grid((unsigned)((n + 255) / 256 < 32 ? (n + 255) / 256 : 32), (unsigned)nb);
            k_copy_rows<<<grid, 256, 0, st>>>(A, lda, p0, nb, n, U, lda);
        }
        CK(sgemm(st, false, false, nb, n, nb, -1.f, Dinv, NB, U, lda, 0.f, Un, lda, done));
        // the rank-64 update of the whole matrix
        if (tc_updates)
            CK(rank_update_tc(st, n, lda, nb, -1.f, T, NB, U, lda, A, lda, (char*)ctx->ws + L.off_tc, L.tc_bytes, ctx->ctl, done));
        else
            CK(sgemm(st, false, false, n, n, nb, -1.f, T, NB, U, lda, 1.f, A, lda, done));
        k_gj_writeback<<<(unsigned)((n * nb + 255) / 256), 256, 0, st>>>(A, lda, n, p0, nb, T, NB, Un, lda, Dinv);
        count_launches(4);     // pivot inverse, zero rows, copy rows, write-back (the GEMMs count themselves)
    }
    CK(cudaGetLastError());
    return OSSCAR_OK;
}

// Rebuilds every piece of the search state from H, G and the current slot permutation.
// With `guarded`, the kernels that can be skipped return at once when the loop has stopped.
int build_state(osscar_ctx* ctx, bool guarded)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    char* ws = (char*)ctx->ws;
    float* Hp = (float*)(ws + L.off_Hp);
    float* Hinv = (float*)(ws + L.off_Hinv);
    float* V = (float*)(ws + L.off_V);
    float* R = (float*)(ws + L.off_R);
    float* big = (float*)(ws + L.off_big);
    double* c = (double*)(ws + L.off_c);
    const int32_t* perm = (const int32_t*)(ws + L.off_perm);
    const int32_t* done = guarded ? &ctx->ctl->done : nullptr;
    void* tc = ws + L.off_tc;
    const int64_t nI = L.nI, nJ = L.nJ;

    {   // slot-permuted copy of H
        dim3 grid((unsigned)L.d1, (unsigned)((L.ldp + 255) / 256 < 64 ? (L.ldp + 255) / 256 : 64));
        k_gather_sym<<<grid, 256, 0, st>>>(ctx->H, L.d1, L.g, perm, Hp, L.ldp);
    }
    CK(cudaMemsetAsync(ws + L.off_vec_begin, 0, L.off_vec_end - L.off_vec_begin, st));
    k_copy_pad<<<(unsigned)nI, 256, 0, st>>>(Hp, L.ldp, nI, nI, Hinv, L.ldh);
    count_launches(2);
    CK(cudaGetLastError());
    { const int rc_inv = invert_spd_inplace(ctx, Hinv, L.ldh, nI, Hp, L.ldp, done, true); if (rc_inv != OSSCAR_OK) return rc_inv; }
    // Every product below that forms a small difference of large sums is accumulated in fp64 (gemm_f64acc): the scores
    // of Eq. impact are compared at 1e-5 relative, and fp32 accumulation leaves cond(H_II) * 2^-24 in them.
    // (1) the inverse.  Single-row groups: fp64 copy by a third-order correction from one fp64 residual, and the fp32
    //     inverse rounded from it (build_hinv64).  Groups of several rows: one Newton-Schulz step, E = I - H_II Hinv in
    //     fp64, Hinv := sym(Hinv + Hinv E) (E is tiny: any product will do)
    ctx->hd_valid = false;
    if (L.g == 1) {
        const int rc_d = build_hinv64(ctx, guarded);
        if (rc_d != OSSCAR_OK) return rc_d;
    } else {
        float* E = big;
        float* Dlt = big + nI * L.ldh;
        CK(gemm_f64acc(st, nI, nI, nI, -1.0, Hp, L.ldp, Hinv, L.ldh, 0.0, nullptr, 0, E, L.ldh, true, done));
        CK(gemm_tc(st, nI, nI, nI, 1.f, Hinv, L.ldh, E, L.ldh, 0.f, Dlt, L.ldh, tc, L.tc_bytes, ctx->ctl, done));
        k_add_sym<<<dim3((unsigned)((nI + 31) / 32), (unsigned)((nI + 31) / 32)), dim3(32, 8), 0, st>>>(Hinv, L.ldh, Dlt, L.ldh, nI, done);
        count_launches(1);
    }
    // (2) V = Hinv G_I on the tensor cores, then one refinement step with the residual G_I - H_II V in fp64
    float* GI = big;
    float* rV = big + nI * L.ldm;
    k_gather_rows<<<(unsigned)nI, 256, 0, st>>>(ctx->G, L.m, L.g, perm, 0, GI, L.ldm);
    count_launches(1);
    if (L.ldm != L.m) CK(cudaMemsetAsync(V, 0, sizeof(float) * nI * L.ldm, st));     // padding columns stay zero
    CK(gemm_tc(st, nI, L.m, nI, 1.f, Hinv, L.ldh, GI, L.ldm, 0.f, V, L.ldm, tc, L.tc_bytes, ctx->ctl, done));
    CK(gemm_f64acc(st, nI, L.m, nI, -1.0, Hp, L.ldp, V, L.ldm, 1.0, GI, L.ldm, rV, L.ldm, false, done));
    CK(gemm_tc(st, nI, L.m, nI, 1.f, Hinv, L.ldh, rV, L.ldm, 1.f, V, L.ldm, tc, L.tc_bytes, ctx->ctl, done));
    // obj = Tr(W^T G) - Tr(G_I^T V)
    if (ctx->have_const) CK(set_device_double(st, &ctx->ctl->acc[0], ctx->user_const));
    else CK(trace_product(st, ctx->W, L.m, ctx->G, L.m, L.d1, L.m, ctx->partials, &ctx->ctl->acc[0]));
    CK(trace_product(st, GI, L.ldm, V, L.ldm, nI, L.m, ctx->partials, &ctx->ctl->acc[1]));
    if (ctx->reduce) {      // both traces are sums over this shard's columns (a constant given by the caller is the layer's)
        double* sh = (double*)(ws + L.off_shard);
        k_pack2<<<1, 1, 0, st>>>(ctx->ctl, sh, 0);
        const int rr = shard_reduce(ctx, sh, 2, OSSCAR_FP64);
        if (rr != OSSCAR_OK) return rr;
        k_pack2<<<1, 1, 0, st>>>(ctx->ctl, sh, 1);
        if (ctx->have_const) CK(set_device_double(st, &ctx->ctl->acc[0], ctx->user_const));
        count_launches(2);
    }
    k_set_obj<<<1, 1, 0, st>>>(ctx->ctl);
    count_launches(1);
    if (nJ > 0) {
        // (3) R_J = G_J - Hp[J, I] V, accumulated in fp64
        k_gather_rows<<<(unsigned)nJ, 256, 0, st>>>(ctx->G, L.m, L.g, perm, nI, R, L.ldm);
        CK(gemm_f64acc(st, nJ, L.m, nI, -1.0, Hp + nI * L.ldp, L.ldp, V, L.ldm, 1.0, R, L.ldm, R, L.ldm, false, done));
        // (4) Pm = Hp[J, I] Hinv kept in fp64, in panels of whole pruned groups that fit the scratch, then the Schur
        // complements H_qq - Pm_q . H_qI as fp64 dot products
        count_launches(1);
        double* Pm = (double*)big;
        const int64_t big_floats = (int64_t)((L.off_Hp - L.off_big) / sizeof(float));
        int64_t gpp = (big_floats / 2) / (L.ldh * L.g);                 // pruned groups per panel
        if (gpp < 1) return OSSCAR_E_WORKSPACE;
        for (int64_t t0 = 0; t0 < L.ng - L.k; t0 += gpp) {
            const int64_t ngr = L.ng - L.k - t0 < gpp ? L.ng - L.k - t0 : gpp;
            const bool tri = L.g == 1;         // one quadratic form per pruned row: half of the symmetric inverse is enough
            CK(gemm_f64out(st, ngr * L.g, nI, nI, Hp + (nI + t0 * L.g) * L.ldp, L.ldp, Hinv, L.ldh, Pm, L.ldh, done, tri));
            k_schur<<<(unsigned)ngr, 256, 0, st>>>(Hp, L.ldp, Pm, L.ldh, nI, L.g, c, t0, tri ? 2.0 : 1.0, done);
            count_launches(1);
        }
    }
    CK(cudaGetLastError());
    return OSSCAR_OK;
}

}  // namespace osscar
