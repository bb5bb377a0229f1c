// Gram matrix H (+)= Xc^T Xc of a block of bf16 activations on the 5th-generation tensor cores
// (Section 2, dense-layer paragraph: H = X^T X, accumulated over calibration rows).
//
// Xc is n x d1 row-major, so both operands of the contraction over tokens are "MN-major": a TMA box
// of 64 columns x 64 tokens lands in shared memory as 64 rows of 128 bytes with the 128-byte swizzle,
// which is the canonical MN-major SWIZZLE_128B operand layout of tcgen05.mma (8 token rows x 128 B per
// swizzle atom, atoms 1024 B apart along tokens, 64-column blocks one box apart).
// One CTA per SM, persistent over the upper-triangle output tiles of 128 x 256:
//   warp 0   : TMA producer (4-stage ring of 48 KB: A = 2 boxes, B = 4 boxes)
//   warp 1   : tcgen05.mma issuer (UMMA 128 x 256 x 16, bf16 in, fp32 accumulators in TMEM, two
//              accumulator buffers of 256 columns so the epilogue of a tile overlaps the next main loop)
//   warps 2-5: epilogue (tcgen05.ld, then H = acc or H += acc with float4 accesses)
// Every wait on an mbarrier is bounded by a cycle budget; when it runs out the CTA raises
// OSSCAR_E_TIMEOUT in *status, drains its own copies, releases TMEM and returns.
#include "osscar_internal.cuh"
#include <cuda.h>
#include <cuda_bf16.h>
#include "tc_common.cuh"

namespace osscar {
namespace {

using namespace tc;

constexpr int TILE_M = 128, TILE_N = 256, BLOCK_K = 64, UMMA_K = 16, STAGES = 4;
constexpr int BOX_COLS = 64;                                  // 128 bytes of bf16
constexpr int BOX_BYTES = BOX_COLS * BLOCK_K * 2;             // 8192
constexpr int A_BYTES = (TILE_M / BOX_COLS) * BOX_BYTES;      // 16384
constexpr int B_BYTES = (TILE_N / BOX_COLS) * BOX_BYTES;      // 32768
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;                // 49152
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int BAND = 16;                                      // tile rows per raster band

// tcgen05 instruction descriptor, kind::f16: D fp32, A/B bf16, both MN-major, M = 128, N = 256.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16)
                          | ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
    // MN-major, SWIZZLE_128B: leading byte offset = one 64-column box (8192 B), stride byte offset = one
    // 8-token swizzle atom (1024 B); descriptor version 1.
    return (uint64_t)((saddr & 0x3FFFFu) >> 4)
         | ((uint64_t)(BOX_BYTES >> 4) << 16)
         | ((uint64_t)(1024 >> 4) << 32)
         | (1ull << 46)
         | (2ull << 61);
}
// Raster order of the upper-triangle tiles: bands of BAND tile rows; inside a band column by column,
// so that concurrently running CTAs share operand columns in L2.  Tile (tm, tn) exists iff tn >= tm / 2.
__device__ __forceinline__ int band_tiles(int b, int TM, int TN) {
    int cnt = 0;
    const int r1 = min(TM, (b + 1) * BAND);
    for (int tm = b * BAND; tm < r1; ++tm) cnt += TN - tm / 2;
    return cnt;
}
__device__ void tile_coords(int id, int TM, int TN, int* tm_out, int* tn_out) {
    int b = 0;
    while (true) {
        const int cnt = band_tiles(b, TM, TN);
        if (id < cnt) break;
        id -= cnt; ++b;
    }
    const int r0 = b * BAND, r1 = min(TM, r0 + BAND);
    for (int tn = r0 / 2; tn < TN; ++tn) {
        // rows of the band that own a tile in column tn: tm / 2 <= tn
        const int last = min(r1 - 1, 2 * tn + 1);
        const int cnt = last - r0 + 1;
        if (id < cnt) { *tm_out = r0 + id; *tn_out = tn; return; }
        id -= cnt;
    }
    *tm_out = r0; *tn_out = TN - 1;   // not reached for a valid id
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
k_gram_tcgen05(const __grid_constant__ CUtensorMap tmap, int64_t n_rows, int64_t d1, float* __restrict__ H,
               int accumulate, int num_tiles, int TM, int TN, int32_t* __restrict__ status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;                      // swizzle atoms need 1024-byte alignment
    uint8_t* bar_ptr = smem_raw + (tiles_base - raw) + STAGES * STAGE_BYTES;
    const uint32_t bars = tiles_base + STAGES * STAGE_BYTES;
    // barrier map (8 bytes each): full[0..3], empty[4..7], tmem_full[8..9], tmem_empty[10..11]
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * (2 * STAGES + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 8 * (2 * STAGES + 4) + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (int)((n_rows + BLOCK_K - 1) / BLOCK_K);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int tm, tn;
                tile_coords(tile, TM, TN, &tm, &tn);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(full_bar(s), STAGE_BYTES);
                    const uint32_t a_dst = tiles_base + s * STAGE_BYTES;
                    const uint32_t b_dst = a_dst + A_BYTES;
                    const int y = kb * BLOCK_K;
#pragma unroll
                    for (int i = 0; i < TILE_M / BOX_COLS; ++i)
                        tma_load_2d(a_dst + i * BOX_BYTES, &tmap, full_bar(s), tm * TILE_M + i * BOX_COLS, y);
#pragma unroll
                    for (int i = 0; i < TILE_N / BOX_COLS; ++i)
                        tma_load_2d(b_dst + i * BOX_BYTES, &tmap, full_bar(s), tn * TILE_N + i * BOX_COLS, y);
                }
            }
            if (*abort_flag) {
                // our own copies may still be landing: wait (bounded) for the stages issued last
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1))
                        if (clock64() - t0 > kWaitLimitCycles) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0;
            int local = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local) {
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);
                if (!mbar_wait(tempty_bar(buf), (use & 1) ^ 1, abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * TILE_N);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_src = tiles_base + s * STAGE_BYTES;
                    const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
                    for (int j = 0; j < BLOCK_K / UMMA_K; ++j) {
                        const uint64_t ad = make_desc(a_src + j * (UMMA_K * 128));
                        const uint64_t bd = make_desc(b_src + j * (UMMA_K * 128));
                        umma_f16(d_tmem, ad, bd, kIdesc, (kb > 0 || j > 0) ? 1u : 0u);
                    }
                    umma_commit(empty_bar(s));          // frees the stage once these MMAs have read it
                }
                if (ok) umma_commit(tfull_bar(buf));    // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int lg = warp & 3;                        // TMEM lane group this warp may access
        int local = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local) {
            int tm, tn;
            tile_coords(tile, TM, TN, &tm, &tn);
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            if (nkb > 0) {
                if (!mbar_wait(tfull_bar(buf), use & 1, abort_flag)) { ok = false; break; }
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int64_t grow = (int64_t)tm * TILE_M + lg * 32 + lane;
            float* hrow = H + grow * d1;
#pragma unroll 1
            for (int c = 0; c < TILE_N / 32; ++c) {
                uint32_t r[32];
                if (nkb > 0) {
                    tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * TILE_N + c * 32), r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                const int64_t gcol = (int64_t)tn * TILE_N + c * 32;
                if (grow < d1) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        if (gcol + j < d1) {            // d1 is a multiple of 8: whole float4 in range
                            float4* dst = reinterpret_cast<float4*>(hrow + gcol + j);
                            float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                   __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                            if (accumulate) { const float4 o = *dst; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
                            *dst = v;
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0 && nkb > 0) mbar_arrive(tempty_bar(buf));
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) *status = OSSCAR_E_TIMEOUT;
}

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

cudaError_t gram_bf16_tcgen05(cudaStream_t st, const void* X, int64_t n_rows, int64_t d1,
                              float* H, bool accumulate, int32_t* status_dev)
{
    if (((uintptr_t)H & 15) || (d1 % 8) != 0) return cudaErrorInvalidValue;
    PFN_encodeTiled encode = get_encode();
    if (!encode) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)d1, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d1 * 2};
    const cuuint32_t box[2] = {BOX_COLS, BLOCK_K};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const int TM = (int)((d1 + TILE_M - 1) / TILE_M), TN = (int)((d1 + TILE_N - 1) / TILE_N);
    int num_tiles = 0;
    for (int tm = 0; tm < TM; ++tm) num_tiles += TN - tm / 2;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    static bool attr_set = false;
    if (!attr_set) {
        e = cudaFuncSetAttribute(k_gram_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const int grid = num_tiles < sms ? num_tiles : sms;
    count_launches(1);
    k_gram_tcgen05<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tmap, n_rows, d1, H, accumulate ? 1 : 0, num_tiles, TM, TN, status_dev);
    return cudaGetLastError();
}

}  // namespace osscar
