// fp32-accurate GEMM on the tensor cores: C = alpha * A * B + beta * C with A (M x K) and B (K x N) row-major fp32.
// Used for the dense contractions around the search: G = H W (Section 2), V = (H_II)^-1 G_I (Eq. tmp5),
// the residual R, the Schur-complement products and the rank-64 updates of the block inversion.
//
// Each fp32 operand is split into three bf16 terms (x = x1 + x2 + x3, 8 mantissa bits each); the product keeps the
// six terms down to 2^-24 relative: x1y1, x1y2, x2y1, x1y3, x2y2, x3y1.  The kernel is the persistent TMA /
// tcgen05 / TMEM pipeline of the Gram kernel with three changes: A is K-major (rows of 128 bytes, SWIZZLE_128B),
// every 64-wide k-block is visited six times (one term pair each), and the TMEM accumulator is drained into fp32
// registers every kFlush k-blocks: tcgen05.mma adds into its accumulator with truncation, so long accumulation
// chains would cost accuracy; the register sums are round-to-nearest.
//   warp 0: TMA producer     warp 1: MMA issuer     warps 2-9: accumulate (TMEM -> registers) and write C
// K is processed in panels sized to the caller's scratch (the bf16 terms of one panel of A and B live there).
//
// The same pipeline, instantiated with an MN-major A operand and a single bf16 term, is the Gram kernel
// H (+)= Xc^T Xc over the upper-triangle tiles (chains of 32 k-blocks between drains), and with B taken from a
// second matrix the cross term G (+)= Xc^T Yc (Y in bf16, or fp32 split into three terms).
#include "osscar_internal.cuh"
#include <cuda_bf16.h>
#include "tc_common.cuh"

namespace osscar {
namespace {

using namespace tc;

constexpr int TILE_M = 128, TILE_N = 256, BLOCK_K = 64, UMMA_K = 16, STAGES = 4;
constexpr int A_BYTES = TILE_M * BLOCK_K * 2;                 // 16384: one box of 128 rows x 128 bytes
constexpr int BOX_BYTES = 64 * BLOCK_K * 2;                   // 8192: 64 columns of B x 64 k-rows
constexpr int B_BYTES = (TILE_N / 64) * BOX_BYTES;            // 32768
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_LD = 33;                                    // row stride (floats) of an epilogue staging block
constexpr int EPI_BYTES = 8 * 32 * EPI_LD * 4;                // one 32 x 32 block per accumulate warp
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256 + EPI_BYTES;
constexpr int NUM_THREADS = 320;                              // 10 warps
constexpr int TMEM_COLS = 512;
constexpr int BAND = 8;                                       // tile rows per raster band (full rasters)
constexpr int TRI_BAND = 16;                                  // same for the upper-triangle raster

// Variants of the pipeline.
enum { MODE_GEMM3 = 0,      // A fp32 split, K-major; B fp32 split; six term pairs; all tiles
       MODE_GRAM = 1,       // A = B = X (bf16, MN-major); one term; upper-triangle tiles
       MODE_CROSS = 2,      // A = X (MN-major), B = Y bf16; one term; all tiles
       MODE_CROSS3 = 3,     // A = X (MN-major), B = Y fp32 split in three terms
       MODE_GRAM3 = 4 };    // A = B = X fp32 split in three terms (MN-major); six term pairs; upper-triangle tiles
template <int MODE> struct Traits {
    static constexpr bool kAMN = MODE != MODE_GEMM3;
    static constexpr bool kSixPairs = MODE == MODE_GEMM3 || MODE == MODE_GRAM3;
    static constexpr int kTerms = kSixPairs ? 6 : (MODE == MODE_CROSS3 ? 3 : 1);
    static constexpr bool kUpper = MODE == MODE_GRAM || MODE == MODE_GRAM3;
    // k-blocks per TMEM accumulation chain: short where small terms ride on large ones, 32 (128 MMAs) for plain bf16
    static constexpr int kFlush = kSixPairs ? 2 : (MODE == MODE_CROSS3 ? 4 : 32);
    static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kAMN ? 1u : 0u) << 15) | (1u << 16)
                                     | ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
};

// A tile: K-major, SWIZZLE_128B: rows of 128 bytes, 8-row swizzle atoms 1024 bytes apart (stride byte offset);
// the leading byte offset is not used by swizzled K-major layouts.
__device__ __forceinline__ uint64_t desc_a(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// B tile: MN-major, SWIZZLE_128B: 64-column boxes 8192 bytes apart (leading), 8-k-row atoms 1024 bytes apart (stride).
__device__ __forceinline__ uint64_t desc_b(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(BOX_BYTES >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

struct Maps { CUtensorMap a[3]; CUtensorMap b[3]; };

__device__ __forceinline__ void tile_full(int id, int TM, int TN, int* tm, int* tn) {
    // bands of BAND tile rows, column-major inside a band: concurrent CTAs share A rows and B columns in L2
    const int per_band = BAND * TN;
    const int b = id / per_band, r = id % per_band;
    const int rows = min(BAND, TM - b * BAND);
    *tn = r / rows; *tm = b * BAND + r % rows;
}
// Upper-triangle tiles of a symmetric result (tile (tm, tn) exists iff tn >= tm / 2), bands of TRI_BAND rows.
__device__ __forceinline__ void tile_upper(int id, int TM, int TN, int* tm_out, int* tn_out) {
    int b = 0;
    while (true) {
        int cnt = 0;
        const int r1 = min(TM, (b + 1) * TRI_BAND);
        for (int tm = b * TRI_BAND; tm < r1; ++tm) cnt += TN - tm / 2;
        if (id < cnt) break;
        id -= cnt; ++b;
    }
    const int r0 = b * TRI_BAND, r1 = min(TM, r0 + TRI_BAND);
    for (int tn = r0 / 2; tn < TN; ++tn) {
        const int last = min(r1 - 1, 2 * tn + 1);
        const int cnt = last - r0 + 1;
        if (id < cnt) { *tm_out = r0 + id; *tn_out = tn; return; }
        id -= cnt;
    }
    *tm_out = r0; *tn_out = TN - 1;
}
template <bool UPPER> __device__ __forceinline__ void tile_of(int id, int TM, int TN, int* tm, int* tn) {
    if (UPPER) tile_upper(id, TM, TN, tm, tn); else tile_full(id, TM, TN, tm, tn);
}

template <int MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
k_mma_pipe(const __grid_constant__ Maps maps, int64_t M, int64_t N, int64_t K, float alpha, float beta,
           float* __restrict__ C, int64_t ldc, int vec_ok, int num_ids, SearchCtl* __restrict__ ctl,
           const int32_t* __restrict__ done)
{
    using TR = Traits<MODE>;
    constexpr int kTerms = TR::kTerms, kFlush = TR::kFlush;
    constexpr uint32_t kIdesc = TR::kIdesc;
    if (done && *done) return;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    uint8_t* bar_ptr = smem_raw + (tiles_base - raw) + STAGES * STAGE_BYTES;
    const uint32_t bars = tiles_base + STAGES * STAGE_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);   // completion of the MMAs in flight when the issuer gives up
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * (2 * STAGES + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 8 * (2 * STAGES + 5) + 8);
    float* epi = reinterpret_cast<float*>(bar_ptr + 256);      // staging blocks of the accumulate warps
    const long long wl = ctl->wait_limit;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int TM = (int)((M + TILE_M - 1) / TILE_M), TN = (int)((N + TILE_N - 1) / TILE_N);
    const int nkb = (int)((K + BLOCK_K - 1) / BLOCK_K);
    const int nflush = (nkb + kFlush - 1) / kFlush;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 8); }
        mbar_init(drain_bar, 1);
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
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int id = blockIdx.x; id < num_ids && ok; id += gridDim.x) {
                int tm, tn;
                tile_of<TR::kUpper>(id, TM, TN, &tm, &tn);
                for (int kb = 0; kb < nkb && ok; ++kb) {
                    for (int term = 0; term < kTerms; ++term, ++it) {
                        // term pairs, small products first: (3,1) (2,2) (1,3) (2,1) (1,2) (1,1)
                        const int pa = TR::kSixPairs ? (0x001012 >> (4 * term)) & 0xF : 0;          // A term: 2,1,0,1,0,0
                        const int pb = TR::kSixPairs ? (0x010210 >> (4 * term)) & 0xF               // B term: 0,1,2,0,1,0
                                     : (MODE == MODE_CROSS3 ? 2 - term : 0);
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1;
                        if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, wl)) { ok = false; break; }
                        mbar_expect_tx(full_bar(s), STAGE_BYTES);
                        const uint32_t a_dst = tiles_base + s * STAGE_BYTES;
                        const uint32_t b_dst = a_dst + A_BYTES;
                        if (TR::kAMN) {         // A^T tile: two boxes of 64 columns x 64 k-rows
#pragma unroll
                            for (int i = 0; i < TILE_M / 64; ++i)
                                tma_load_2d(a_dst + i * BOX_BYTES, &maps.a[pa], full_bar(s), tm * TILE_M + i * 64, kb * BLOCK_K);
                        } else {
                            tma_load_2d(a_dst, &maps.a[pa], full_bar(s), kb * BLOCK_K, tm * TILE_M);
                        }
#pragma unroll
                        for (int i = 0; i < TILE_N / 64; ++i)
                            tma_load_2d(b_dst + i * BOX_BYTES, &maps.b[pb], full_bar(s), tn * TILE_N + i * 64, kb * BLOCK_K);
                    }
                }
            }
            if (*abort_flag) {                    // the copies still in flight must land before the CTA exits
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) mbar_drain(full_bar(j % STAGES), (j / STAGES) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, fl = 0;            // stage counter, flush counter (selects the TMEM buffer)
            bool ok = true;
            for (int id = blockIdx.x; id < num_ids && ok; id += gridDim.x) {
                for (int f = 0; f < nflush && ok; ++f, ++fl) {
                    const int buf = fl & 1;
                    if (!mbar_wait(tempty_bar(buf), ((fl >> 1) & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * TILE_N);
                    const int kb1 = min(nkb, (f + 1) * kFlush);
                    bool first = true;
                    for (int kb = f * kFlush; kb < kb1 && ok; ++kb) {
                        for (int term = 0; term < kTerms; ++term, ++it) {
                            const int s = it % STAGES;
                            const uint32_t ph = (it / STAGES) & 1;
                            if (!mbar_wait(full_bar(s), ph, abort_flag, wl)) { ok = false; break; }
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            const uint32_t a_src = tiles_base + s * STAGE_BYTES;
                            const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
                            for (int j = 0; j < BLOCK_K / UMMA_K; ++j) {
                                // K-major A: +32 bytes per 16 k inside the 128-byte row; MN-major: +16 k-rows of 128 bytes
                                const uint64_t ad = TR::kAMN ? desc_b(a_src + j * (UMMA_K * 128)) : desc_a(a_src + j * 32);
                                umma_f16(d_tmem, ad, desc_b(b_src + j * (UMMA_K * 128)), kIdesc, first ? 0u : 1u);
                                first = false;
                            }
                            umma_commit(empty_bar(s));
                        }
                    }
                    if (ok) umma_commit(tfull_bar(buf));
                }
            }
            if (!ok) {            // MMAs already issued keep running: they must finish before TMEM and the tiles are released
                umma_commit(drain_bar);
                mbar_drain(drain_bar, 0);
            }
        }
    } else {
        // warps 2..9: lane group = warp % 4, column half = (warp - 2) / 4
        const int lg = warp & 3, half = (warp - 2) >> 2;
        uint32_t fl = 0;
        bool ok = true;
        for (int id = blockIdx.x; id < num_ids && ok; id += gridDim.x) {
            int tm, tn;
            tile_of<TR::kUpper>(id, TM, TN, &tm, &tn);
            float acc[128];
#pragma unroll
            for (int j = 0; j < 128; ++j) acc[j] = 0.f;
            if (beta != 0.f) {      // bring this thread's part of the old C row towards L2 while the tile is computed
                const int64_t prow = (int64_t)tm * TILE_M + lg * 32 + lane;
                const int64_t pcol = (int64_t)tn * TILE_N + half * 128;
                if (prow < M) {
#pragma unroll
                    for (int j = 0; j < 128; j += 32)
                        if (pcol + j < N) asm volatile("prefetch.global.L2 [%0];" ::"l"(C + prow * ldc + pcol + j));
                }
            }
            for (int f = 0; f < nflush && ok; ++f, ++fl) {
                const int buf = fl & 1;
                if (!mbar_wait(tfull_bar(buf), (fl >> 1) & 1, abort_flag, wl)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * TILE_N + half * 128 + c * 32), r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[c * 32 + j] += __uint_as_float(r[j]);
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));
            }
            if (!ok) break;
            const int64_t grow = (int64_t)tm * TILE_M + lg * 32 + lane;
            const int64_t gcol0 = (int64_t)tn * TILE_N + half * 128;
            {
                float* crow = C + grow * ldc;
                if (vec_ok) {
                    // 32 x 32 blocks go through shared memory so that a warp touches whole 128-byte lines of C:
                    // 8 lanes per row, 4 rows per instruction, the 8 row groups of a block in flight together
                    float* stg = epi + (warp - 2) * 32 * EPI_LD;
                    const int64_t grow0 = (int64_t)tm * TILE_M + lg * 32;
                    const int rsub = lane >> 3, c4 = (lane & 7) * 4;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int64_t gc = gcol0 + c * 32 + c4;
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 32; ++j) stg[lane * EPI_LD + j] = alpha * acc[c * 32 + j];
                        __syncwarp();
                        float4 o[8];
                        if (beta != 0.f) {
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const int64_t gr = grow0 + q * 4 + rsub;
                                o[q] = (gr < M && gc < N) ? __ldcs(reinterpret_cast<const float4*>(C + gr * ldc + gc))
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const int r = q * 4 + rsub;
                            const int64_t gr = grow0 + r;
                            const float* sp = stg + r * EPI_LD + c4;
                            float4 v = make_float4(sp[0], sp[1], sp[2], sp[3]);
                            if (beta != 0.f) {
                                v.x = fmaf(beta, o[q].x, v.x); v.y = fmaf(beta, o[q].y, v.y);
                                v.z = fmaf(beta, o[q].z, v.z); v.w = fmaf(beta, o[q].w, v.w);
                            }
                            if (gr < M && gc < N) *reinterpret_cast<float4*>(C + gr * ldc + gc) = v;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 128; ++j) {
                        if (grow < M && gcol0 + j < N) {
                            float v = alpha * acc[j];
                            if (beta != 0.f) v = fmaf(beta, crow[gcol0 + j], v);
                            crow[gcol0 + j] = v;
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) ctl->status = OSSCAR_E_TIMEOUT;
}

// x = x1 + x2 + x3 with bf16 terms (round to nearest each time); dst rows are ldd wide (a multiple of 8), the tail is
// zero.  A thread converts eight consecutive elements of a row: two 16-byte loads where the source allows it (vec),
// one 16-byte store per term.
__device__ __forceinline__ void split3_one(float x, __nv_bfloat16& a, __nv_bfloat16& b, __nv_bfloat16& c)
{
    a = __float2bfloat16_rn(x);
    x -= __bfloat162float(a);
    b = __float2bfloat16_rn(x);
    x -= __bfloat162float(b);
    c = __float2bfloat16_rn(x);
}

__global__ void k_split3(const float* __restrict__ src, int64_t lds, int64_t rows, int64_t cols,
                         __nv_bfloat16* __restrict__ d1, __nv_bfloat16* __restrict__ d2, __nv_bfloat16* __restrict__ d3,
                         int64_t ldd, int vec, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t per_row = ldd / 8, total = rows * per_row;
    const bool small = total < (int64_t)0x7fffffff;          // 32-bit index arithmetic where it fits (64-bit division is slow)
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        int64_t r, j;
        if (small) { const uint32_t i32 = (uint32_t)idx, l32 = (uint32_t)per_row; r = i32 / l32; j = i32 % l32; }
        else { r = idx / per_row; j = idx % per_row; }
        const int64_t c0 = j * 8;
        const float* s = src + r * lds + c0;
        float x[8];
        if (vec && c0 + 8 <= cols) {
            const float4 lo = *reinterpret_cast<const float4*>(s), hi = *reinterpret_cast<const float4*>(s + 4);
            x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w; x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = c0 + i < cols ? s[i] : 0.f;
        }
        __align__(16) __nv_bfloat16 a[8], b[8], c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split3_one(x[i], a[i], b[i], c[i]);
        const int64_t o = r * ldd + c0;
        *reinterpret_cast<uint4*>(d1 + o) = *reinterpret_cast<const uint4*>(a);
        *reinterpret_cast<uint4*>(d2 + o) = *reinterpret_cast<const uint4*>(b);
        *reinterpret_cast<uint4*>(d3 + o) = *reinterpret_cast<const uint4*>(c);
    }
}

// Launch of k_split3: 16-byte loads when the source rows start on 16-byte boundaries.
static void launch_split3(cudaStream_t st, const float* src, int64_t lds, int64_t rows, int64_t cols,
                          __nv_bfloat16* d1, __nv_bfloat16* d2, __nv_bfloat16* d3, int64_t ldd, const int32_t* done)
{
    const int vec = (((uintptr_t)src & 15) == 0 && (lds % 4) == 0) ? 1 : 0;
    const int64_t work = rows * (ldd / 8);
    unsigned blocks = (unsigned)((work + 255) / 256 < 1184 ? (work + 255) / 256 : 1184);
    if (blocks < 1) blocks = 1;
    k_split3<<<blocks, 256, 0, st>>>(src, lds, rows, cols, d1, d2, d3, ldd, vec, done);
}

// ---------------------------------------------------------------------------------------------------------------
// Rank-K update C += alpha * U * W with a short inner dimension (K <= 128): U (M x K) and W (K x N) are panels, C is
// large and streamed once.  The generic pipeline above re-reads the operand terms for every output tile, which for
// K ~ 100 is more L2 traffic than the tile of C itself; here a CTA keeps the three bf16 terms of its 128-row band
// of U in shared memory (up to 96 KB) across a run of 128-column tiles and only the terms of W stream through a
// two-stage ring (48 KB per 64-wide k-block).  One TMEM accumulator chain per tile (at most 48 MMAs), drained by
// eight accumulate warps that do the read-modify-write of C through the shared-memory staging blocks.
constexpr int RU_TN = 128;                                   // columns per tile
constexpr int RU_W_BYTES = 3 * (RU_TN / 64) * BOX_BYTES;     // 49152: three terms of a 64 x 128 block of W
constexpr int RU_U_BYTES = 3 * 2 * A_BYTES;                  // 98304: three terms x two k-blocks of the U band
constexpr int RU_SMEM = RU_U_BYTES + 2 * RU_W_BYTES + 1024 + 256 + EPI_BYTES;
constexpr uint32_t kRuIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(RU_TN >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);

__global__ void __launch_bounds__(NUM_THREADS, 1)
k_rank_update(const __grid_constant__ Maps maps, int64_t M, int64_t N, int nkb, float alpha, float* __restrict__ C, int64_t ldc,
              int TN, int nchunk, int num_items, float* __restrict__ sq_part, SearchCtl* __restrict__ ctl,
              const int32_t* __restrict__ done)
{
    if (done && *done) return;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t u_base = base, w_base = base + RU_U_BYTES;
    uint8_t* bar_ptr = base_ptr + RU_U_BYTES + 2 * RU_W_BYTES;
    const uint32_t bars = base + RU_U_BYTES + 2 * RU_W_BYTES;
    auto w_full = [&](int s) { return bars + 8u * s; };
    auto w_empty = [&](int s) { return bars + 8u * (2 + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (4 + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (6 + b); };
    const uint32_t u_full = bars + 8u * 8, u_empty = bars + 8u * 9, drain_bar = bars + 8u * 10;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * 11);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 8 * 11 + 8);
    float* epi = reinterpret_cast<float*>(bar_ptr + 256);
    const long long wl = ctl->wait_limit;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(w_full(i), 1); mbar_init(w_empty(i), 1); mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), 8); }
        mbar_init(u_full, 1); mbar_init(u_empty, 1); mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // item = (row band, run of column tiles)
    auto item_of = [&](int id, int* tm, int* tn0, int* tn1) {
        *tm = id / nchunk;
        const int c = id % nchunk, per = (TN + nchunk - 1) / nchunk;
        *tn0 = c * per; *tn1 = min(TN, *tn0 + per);
    };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0, item = 0;          // item counts the bands this CTA has loaded
            bool ok = true;
            for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
                int tm, tn0, tn1;
                item_of(id, &tm, &tn0, &tn1);
                if (tn0 >= tn1) continue;
                if (!mbar_wait(u_empty, (item & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                ++item;
                mbar_expect_tx(u_full, (uint32_t)(3 * nkb * A_BYTES));
                for (int kb = 0; kb < nkb; ++kb)
#pragma unroll
                    for (int term = 0; term < 3; ++term)
                        tma_load_2d(u_base + (term * 2 + kb) * A_BYTES, &maps.a[term], u_full, kb * BLOCK_K, tm * TILE_M);
                for (int tn = tn0; tn < tn1 && ok; ++tn) {
                    for (int kb = 0; kb < nkb; ++kb, ++it) {
                        const int s = it & 1;
                        if (!mbar_wait(w_empty(s), ((it >> 1) & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                        mbar_expect_tx(w_full(s), RU_W_BYTES);
#pragma unroll
                        for (int term = 0; term < 3; ++term)
#pragma unroll
                            for (int i = 0; i < RU_TN / 64; ++i)
                                tma_load_2d(w_base + s * RU_W_BYTES + (term * (RU_TN / 64) + i) * BOX_BYTES, &maps.b[term], w_full(s),
                                            tn * RU_TN + i * 64, kb * BLOCK_K);
                    }
                }
            }
            if (*abort_flag) {                    // let the copies in flight land before the CTA exits
                if (item > 0) mbar_drain(u_full, (item - 1) & 1);
                for (uint32_t j = it > 2 ? it - 2 : 0; j < it; ++j) mbar_drain(w_full(j & 1), (j >> 1) & 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, tile = 0, item = 0;
            bool ok = true;
            for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
                int tm, tn0, tn1;
                item_of(id, &tm, &tn0, &tn1);
                if (tn0 >= tn1) continue;
                if (!mbar_wait(u_full, item & 1, abort_flag, wl)) { ok = false; break; }
                ++item;
                for (int tn = tn0; tn < tn1 && ok; ++tn, ++tile) {
                    const int buf = tile & 1;
                    if (!mbar_wait(tempty_bar(buf), ((tile >> 1) & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * RU_TN);
                    bool first = true;
                    for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
                        const int s = it & 1;
                        if (!mbar_wait(w_full(s), (it >> 1) & 1, abort_flag, wl)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                        for (int term = 0; term < 6; ++term) {
                            const int pa = (0x001012 >> (4 * term)) & 0xF;      // small products first
                            const int pb = (0x010210 >> (4 * term)) & 0xF;
                            const uint32_t a_src = u_base + (pa * 2 + kb) * A_BYTES;
                            const uint32_t b_src = w_base + s * RU_W_BYTES + pb * (RU_TN / 64) * BOX_BYTES;
#pragma unroll
                            for (int j = 0; j < BLOCK_K / UMMA_K; ++j) {
                                umma_f16(d_tmem, desc_a(a_src + j * 32), desc_b(b_src + j * (UMMA_K * 128)), kRuIdesc, first ? 0u : 1u);
                                first = false;
                            }
                        }
                        umma_commit(w_empty(s));
                    }
                    if (ok) umma_commit(tfull_bar(buf));
                }
                if (ok) umma_commit(u_empty);        // the band's terms may be replaced once these MMAs are done
            }
            if (!ok) {            // MMAs already issued must finish before TMEM and the operand tiles are released
                umma_commit(drain_bar);
                mbar_drain(drain_bar, 0);
            }
        }
    } else {
        const int lg = warp & 3, half = (warp - 2) >> 2;       // 32 rows x 64 columns per warp
        uint32_t tile = 0;
        bool ok = true;
        float* stg = epi + (warp - 2) * 32 * EPI_LD;
        const int rsub = lane >> 3, c4 = (lane & 7) * 4;
        for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
            int tm, tn0, tn1;
            item_of(id, &tm, &tn0, &tn1);
            for (int tn = tn0; tn < tn1 && ok; ++tn, ++tile) {
                const int buf = tile & 1;
                const int64_t grow0 = (int64_t)tm * TILE_M + lg * 32;
                const int64_t gcol0 = (int64_t)tn * RU_TN + half * 64;
                if (grow0 + lane < M) {          // bring the old values of this thread's row segment towards L2
#pragma unroll
                    for (int j = 0; j < 64; j += 32)
                        if (gcol0 + j < N) asm volatile("prefetch.global.L2 [%0];" ::"l"(C + (grow0 + lane) * ldc + gcol0 + j));
                }
                if (!mbar_wait(tfull_bar(buf), (tile >> 1) & 1, abort_flag, wl)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                float acc[64];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * RU_TN + half * 64 + c * 32), r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[c * 32 + j] = alpha * __uint_as_float(r[j]);
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));
                float sq[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) sq[q] = 0.f;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int64_t gc = gcol0 + c * 32 + c4;
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 32; ++j) stg[lane * EPI_LD + j] = acc[c * 32 + j];
                    __syncwarp();
                    float4 o[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int64_t gr = grow0 + q * 4 + rsub;
                        o[q] = (gr < M && gc < N) ? __ldcs(reinterpret_cast<const float4*>(C + gr * ldc + gc)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const int r = q * 4 + rsub;
                        const int64_t gr = grow0 + r;
                        const float* sp = stg + r * EPI_LD + c4;
                        const float4 v = make_float4(o[q].x + sp[0], o[q].y + sp[1], o[q].z + sp[2], o[q].w + sp[3]);
                        if (gr < M && gc < N) {
                            *reinterpret_cast<float4*>(C + gr * ldc + gc) = v;
                            sq[q] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                        }
                    }
                }
                if (sq_part) {           // squared norm of the new row segment (64 columns): one partial per row and segment
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        float v = sq[q];
                        v += __shfl_xor_sync(0xffffffffu, v, 1); v += __shfl_xor_sync(0xffffffffu, v, 2); v += __shfl_xor_sync(0xffffffffu, v, 4);
                        const int64_t gr = grow0 + q * 4 + rsub;
                        if ((lane & 7) == 0 && gr < M) sq_part[gr * (2 * TN) + 2 * tn + half] = v;
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(256) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) ctl->status = OSSCAR_E_TIMEOUT;
}

bool encode_2d(PFN_encodeTiled enc, CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t ld_elems,
               uint32_t box_inner, uint32_t box_outer)
{
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {ld_elems * 2};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t gemm_tc_min_scratch(int64_t M, int64_t N)
{
    // the three bf16 terms of a 64-wide panel of A and of B, each buffer 1024-byte aligned
    return (size_t)6 * (size_t)(M + round_up(N, 8)) * 64 + 8 * 1024;
}

cudaError_t gemm_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, float alpha, const float* A, int64_t lda,
                    const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                    void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    if (K <= 0 || scratch_bytes < gemm_tc_min_scratch(M, N) || ((uintptr_t)scratch & 255)) return cudaErrorInvalidValue;
    PFN_encodeTiled enc = get_encode();
    if (!enc) return cudaErrorNotSupported;
    const int64_t ldn = round_up(N, 8);                         // row stride of the B terms (16-byte multiple)
    // panel width: largest multiple of 64 whose six buffers fit
    int64_t kc = (int64_t)((scratch_bytes - 8 * 1024) / (6 * (size_t)(M + ldn))) / 64 * 64;
    if (kc > round_up(K, 64)) kc = round_up(K, 64);
    if (kc > 8192) kc = 8192;
    auto align_up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
    const size_t a_bytes = align_up((size_t)M * kc * 2), b_bytes = align_up((size_t)kc * ldn * 2);
    if (3 * (a_bytes + b_bytes) > scratch_bytes) return cudaErrorInvalidValue;
    __nv_bfloat16* ap[3]; __nv_bfloat16* bp[3];
    for (int i = 0; i < 3; ++i) {
        ap[i] = (__nv_bfloat16*)((char*)scratch + i * a_bytes);
        bp[i] = (__nv_bfloat16*)((char*)scratch + 3 * a_bytes + i * b_bytes);
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_mma_pipe<MODE_GEMM3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const int TM = (int)((M + TILE_M - 1) / TILE_M), TN = (int)((N + TILE_N - 1) / TILE_N);
    const int num_ids = TM * TN;
    const int vec_ok = (((uintptr_t)C & 15) == 0 && (ldc % 4) == 0 && (N % 4) == 0) ? 1 : 0;
    for (int64_t k0 = 0; k0 < K; k0 += kc) {
        const int64_t kw = K - k0 < kc ? K - k0 : kc;
        const int64_t kw8 = round_up(kw, 8);                    // row stride of the A terms
        launch_split3(st, A + k0, lda, M, kw, ap[0], ap[1], ap[2], kw8, done);
        launch_split3(st, B + k0 * ldb, ldb, kw, N, bp[0], bp[1], bp[2], ldn, done);
        Maps maps;
        for (int i = 0; i < 3; ++i) {
            // A terms: inner dimension k (kw valid, rows kw8 apart), box 64 x 128; B terms: inner n, box 64 x 64
            if (!encode_2d(enc, &maps.a[i], ap[i], (uint64_t)kw, (uint64_t)M, (uint64_t)kw8, BLOCK_K, TILE_M)) return cudaErrorInvalidValue;
            if (!encode_2d(enc, &maps.b[i], bp[i], (uint64_t)N, (uint64_t)kw, (uint64_t)ldn, 64, BLOCK_K)) return cudaErrorInvalidValue;
        }
        const int grid = num_ids < sms ? num_ids : sms;
        k_mma_pipe<MODE_GEMM3><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(maps, M, N, kw, alpha, k0 == 0 ? beta : 1.f, C, ldc, vec_ok,
                                                                      num_ids, ctl_dev, done);
        count_launches(3);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace osscar (reopened below)
namespace osscar {
namespace {
// norm[row] = sum of the row's partials, in segment order.
__global__ void k_rownorm_sum(const float* __restrict__ part, int64_t rows, int nseg, float* __restrict__ norm, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    float s = 0.f;
    for (int j = 0; j < nseg; ++j) s += part[r * nseg + j];
    norm[r] = s;
}
}  // namespace

// C += alpha * U * W for a short inner dimension (see k_rank_update); falls back to the generic product otherwise.
// With `row_sq` (M floats) and `sq_scratch` (M * 2 * ceil(N / 128) floats) the squared norms of the updated rows come
// out of the same pass (short-dimension path only; returns cudaErrorInvalidValue otherwise).
cudaError_t rank_update_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, float alpha, const float* U, int64_t ldu,
                           const float* W, int64_t ldw, float* C, int64_t ldc,
                           void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done,
                           float* row_sq, float* sq_scratch)
{
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    const bool fits = K <= 2 * BLOCK_K && (N % 4) == 0 && (ldc % 4) == 0 && (((uintptr_t)C & 15) == 0);
    if (!fits && row_sq) return cudaErrorInvalidValue;
    if (!fits) return gemm_tc(st, M, N, K, alpha, U, ldu, W, ldw, 1.f, C, ldc, scratch, scratch_bytes, ctl_dev, done);
    PFN_encodeTiled enc = get_encode();
    if (!enc) return cudaErrorNotSupported;
    if ((uintptr_t)scratch & 255) return cudaErrorInvalidValue;
    const int64_t k8 = round_up(K, 8), ldn = round_up(N, 8);
    auto align_up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
    const size_t u_bytes = align_up((size_t)M * k8 * 2), w_bytes = align_up((size_t)K * ldn * 2);
    if (3 * (u_bytes + w_bytes) > scratch_bytes) return cudaErrorInvalidValue;
    __nv_bfloat16* up[3]; __nv_bfloat16* wp[3];
    for (int i = 0; i < 3; ++i) {
        up[i] = (__nv_bfloat16*)((char*)scratch + i * u_bytes);
        wp[i] = (__nv_bfloat16*)((char*)scratch + 3 * u_bytes + i * w_bytes);
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_rank_update, cudaFuncAttributeMaxDynamicSharedMemorySize, RU_SMEM);
    if (e != cudaSuccess) return e;
    launch_split3(st, U, ldu, M, K, up[0], up[1], up[2], k8, done);
    launch_split3(st, W, ldw, K, N, wp[0], wp[1], wp[2], ldn, done);
    Maps maps;
    for (int i = 0; i < 3; ++i) {
        if (!encode_2d(enc, &maps.a[i], up[i], (uint64_t)K, (uint64_t)M, (uint64_t)k8, BLOCK_K, TILE_M)) return cudaErrorInvalidValue;
        if (!encode_2d(enc, &maps.b[i], wp[i], (uint64_t)N, (uint64_t)K, (uint64_t)ldn, 64, BLOCK_K)) return cudaErrorInvalidValue;
    }
    const int TM = (int)((M + TILE_M - 1) / TILE_M), TN = (int)((N + RU_TN - 1) / RU_TN);
    int nchunk = (4 * sms + TM - 1) / TM;                 // runs of column tiles per band: about four items per SM
    if (nchunk > TN) nchunk = TN;
    if (nchunk < 1) nchunk = 1;
    const int per = (TN + nchunk - 1) / nchunk;
    nchunk = (TN + per - 1) / per;                        // no empty runs
    const int num_items = TM * nchunk;
    const int nkb = (int)((K + BLOCK_K - 1) / BLOCK_K);
    k_rank_update<<<num_items < sms ? num_items : sms, NUM_THREADS, RU_SMEM, st>>>(maps, M, N, nkb, alpha, C, ldc, TN, nchunk, num_items,
                                                                                  row_sq ? sq_scratch : nullptr, ctl_dev, done);
    count_launches(3);
    if (row_sq) {
        k_rownorm_sum<<<(unsigned)((M + 255) / 256), 256, 0, st>>>(sq_scratch, M, 2 * TN, row_sq, done);
        count_launches(1);
    }
    return cudaGetLastError();
}

// H (+)= Xc^T Xc over the upper-triangle tiles (Yc == nullptr), or G (+)= Xc^T Yc over all tiles.
// Xc: n_rows x d1 bf16.  Yc: n_rows x m, bf16 (y_fp32 == 0) or fp32, which is split into three bf16 terms in
// `scratch` (3 * n_rows * round_up(m, 8) * 2 bytes, 1024-byte aligned pieces).
cudaError_t gram_tc2(cudaStream_t st, const void* X, int64_t n_rows, int64_t d1, const void* Y, int y_fp32, int64_t m,
                     float* C, bool accumulate, void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev)
{
    if (n_rows <= 0) return cudaSuccess;
    if (((uintptr_t)X & 15) || (d1 % 8) != 0) return cudaErrorInvalidValue;
    PFN_encodeTiled enc = get_encode();
    if (!enc) return cudaErrorNotSupported;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    Maps maps;
    if (!encode_2d(enc, &maps.a[0], X, (uint64_t)d1, (uint64_t)n_rows, (uint64_t)d1, 64, BLOCK_K)) return cudaErrorInvalidValue;
    maps.a[1] = maps.a[2] = maps.a[0];
    const float beta = accumulate ? 1.f : 0.f;
    const int TM = (int)((d1 + TILE_M - 1) / TILE_M);
    if (!Y) {
        for (int i = 0; i < 3; ++i) maps.b[i] = maps.a[0];
        const int TN = (int)((d1 + TILE_N - 1) / TILE_N);
        int num_ids = 0;
        for (int tm = 0; tm < TM; ++tm) num_ids += TN - tm / 2;
        const int vec_ok = (((uintptr_t)C & 15) == 0 && (d1 % 4) == 0) ? 1 : 0;
        e = cudaFuncSetAttribute(k_mma_pipe<MODE_GRAM>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        k_mma_pipe<MODE_GRAM><<<num_ids < sms ? num_ids : sms, NUM_THREADS, SMEM_BYTES, st>>>(
            maps, d1, d1, n_rows, 1.f, beta, C, d1, vec_ok, num_ids, ctl_dev, nullptr);
        count_launches(1);
        return cudaGetLastError();
    }
    const int TN = (int)((m + TILE_N - 1) / TILE_N);
    const int num_ids = TM * TN;
    const int vec_ok = (((uintptr_t)C & 15) == 0 && (m % 4) == 0) ? 1 : 0;
    if (!y_fp32) {
        if (((uintptr_t)Y & 15) || (m % 8) != 0) return cudaErrorInvalidValue;
        if (!encode_2d(enc, &maps.b[0], Y, (uint64_t)m, (uint64_t)n_rows, (uint64_t)m, 64, BLOCK_K)) return cudaErrorInvalidValue;
        maps.b[1] = maps.b[2] = maps.b[0];
        e = cudaFuncSetAttribute(k_mma_pipe<MODE_CROSS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        k_mma_pipe<MODE_CROSS><<<num_ids < sms ? num_ids : sms, NUM_THREADS, SMEM_BYTES, st>>>(
            maps, d1, m, n_rows, 1.f, beta, C, m, vec_ok, num_ids, ctl_dev, nullptr);
        count_launches(1);
        return cudaGetLastError();
    }
    const int64_t ldn = round_up(m, 8);
    const size_t piece = ((size_t)n_rows * ldn * 2 + 1023) / 1024 * 1024;
    if (!scratch || scratch_bytes < 3 * piece || ((uintptr_t)scratch & 255)) return cudaErrorInvalidValue;
    __nv_bfloat16* yp[3];
    for (int i = 0; i < 3; ++i) yp[i] = (__nv_bfloat16*)((char*)scratch + i * piece);
    launch_split3(st, (const float*)Y, m, n_rows, m, yp[0], yp[1], yp[2], ldn, nullptr);
    for (int i = 0; i < 3; ++i)
        if (!encode_2d(enc, &maps.b[i], yp[i], (uint64_t)m, (uint64_t)n_rows, (uint64_t)ldn, 64, BLOCK_K)) return cudaErrorInvalidValue;
    e = cudaFuncSetAttribute(k_mma_pipe<MODE_CROSS3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    k_mma_pipe<MODE_CROSS3><<<num_ids < sms ? num_ids : sms, NUM_THREADS, SMEM_BYTES, st>>>(
        maps, d1, m, n_rows, 1.f, beta, C, m, vec_ok, num_ids, ctl_dev, nullptr);
    count_launches(2);
    return cudaGetLastError();
}

// H (+)= Xc^T Xc for fp32 Xc (n_rows x d1, row-major) on the tensor cores: Xc is split into three bf16 terms in
// `scratch` and the six term pairs down to 2^-24 relative are accumulated over the upper-triangle tiles, in row panels
// sized to the scratch (each panel needs 6 * rows * round_up(d1, 8) bytes).  Returns cudaErrorMemoryAllocation when
// the scratch cannot hold a panel of 64 rows, so that the caller can take another path.
cudaError_t gram_tc3(cudaStream_t st, const float* X, int64_t n_rows, int64_t d1, float* C, bool accumulate,
                     void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev)
{
    if (n_rows <= 0) return cudaSuccess;
    const int64_t ldn = round_up(d1, 8);
    if (!scratch || ((uintptr_t)scratch & 255)) return cudaErrorMemoryAllocation;
    const size_t usable = scratch_bytes > 4096 ? scratch_bytes - 4096 : 0;
    int64_t panel = (int64_t)(usable / (6 * (size_t)ldn));
    if (panel >= n_rows) panel = n_rows; else panel = panel / 64 * 64;
    if (panel < 64 && panel < n_rows) return cudaErrorMemoryAllocation;
    PFN_encodeTiled enc = get_encode();
    if (!enc) return cudaErrorNotSupported;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_mma_pipe<MODE_GRAM3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    const size_t piece = ((size_t)panel * ldn * 2 + 1023) / 1024 * 1024;
    __nv_bfloat16* xp[3];
    for (int i = 0; i < 3; ++i) xp[i] = (__nv_bfloat16*)((char*)scratch + i * piece);
    const int TM = (int)((d1 + TILE_M - 1) / TILE_M), TN = (int)((d1 + TILE_N - 1) / TILE_N);
    int num_ids = 0;
    for (int tm = 0; tm < TM; ++tm) num_ids += TN - tm / 2;
    const int vec_ok = (((uintptr_t)C & 15) == 0 && (d1 % 4) == 0) ? 1 : 0;
    for (int64_t r0 = 0; r0 < n_rows; r0 += panel) {
        const int64_t rows = n_rows - r0 < panel ? n_rows - r0 : panel;
        launch_split3(st, X + r0 * d1, d1, rows, d1, xp[0], xp[1], xp[2], ldn, nullptr);
        Maps maps;
        for (int i = 0; i < 3; ++i) {
            if (!encode_2d(enc, &maps.a[i], xp[i], (uint64_t)d1, (uint64_t)rows, (uint64_t)ldn, 64, BLOCK_K)) return cudaErrorInvalidValue;
            maps.b[i] = maps.a[i];
        }
        k_mma_pipe<MODE_GRAM3><<<num_ids < sms ? num_ids : sms, NUM_THREADS, SMEM_BYTES, st>>>(
            maps, d1, d1, rows, 1.f, (accumulate || r0 > 0) ? 1.f : 0.f, C, d1, vec_ok, num_ids, ctl_dev, nullptr);
        count_launches(2);
    }
    return cudaGetLastError();
}

}  // namespace osscar
