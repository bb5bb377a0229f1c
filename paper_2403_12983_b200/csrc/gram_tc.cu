// Lower triangle of the Gram matrix: the tensor-core pass (gemm_tc.cu, upper-triangle tiles of H = X^T X,
// Section 2 dense-layer paragraph) leaves it to this copy.
#include "osscar_internal.cuh"

namespace osscar {
namespace {

// H[i][j] = H[j][i] for i > j (the tensor-core pass fills the upper triangle).
__global__ void k_mirror(float* __restrict__ H, int64_t d1)
{
    __shared__ float tile[32][33];
    const int64_t bi = blockIdx.y, bj = blockIdx.x;      // destination block (rows bi, cols bj), bi >= bj
    if (bi < bj) return;
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (int r = ty; r < 32; r += 8) {
        const int64_t sr = bj * 32 + r, sc = bi * 32 + tx;   // source element (row in bj block, col in bi block)
        tile[r][tx] = (sr < d1 && sc < d1) ? H[sr * d1 + sc] : 0.f;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int64_t dr = bi * 32 + r, dc = bj * 32 + tx;
        if (dr < d1 && dc < d1 && dr > dc) H[dr * d1 + dc] = tile[tx][r];
    }
}

}  // namespace

cudaError_t gram_mirror(cudaStream_t st, float* H, int64_t d1)
{
    const unsigned nb = (unsigned)((d1 + 31) / 32);
    k_mirror<<<dim3(nb, nb), dim3(32, 8), 0, st>>>(H, d1);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace osscar
