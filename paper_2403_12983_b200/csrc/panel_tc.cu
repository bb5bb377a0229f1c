// Streamed matrix times narrow panel on the tensor cores, fp32-accurate, for the block exchange of the swap search:
//   Y[i][e] = sum_k A[i][k] * P[e][k]      A: M x K fp32 (row-major, read once from HBM), P: N x K panel, N <= 128.
// A changes or moves every iteration, so it cannot be kept as bf16 terms in memory: the split happens on the way.
//   warp 0      TMA producer: fp32 boxes of A (128 rows x 32 columns, two per 64-wide k-block) into a two-slot raw ring,
//               and the three bf16 terms of the panel's k-block (split once per call by a small kernel)
//   warps 2-5   converters: read the raw fp32 box, write x = x1 + x2 + x3 as three bf16 K-major SWIZZLE_128B tiles
//   warp 1      tcgen05.mma issuer: six term pairs per k-block (error 2^-24 relative), accumulator in TMEM
//   warps 6-9   accumulate: drain the TMEM accumulator into fp32 registers every two k-blocks (tcgen05.mma adds with
//               truncation; the register sums are round-to-nearest) and write the rows of Y
// Work items are (row tile, k slice) pairs so that short matrices still fill the machine; slices write partial sums
// that a second kernel adds in slice order.  Every mbarrier wait is bounded (status OSSCAR_E_TIMEOUT).
#include "osscar_internal.cuh"
#include <cuda_bf16.h>
#include "tc_common.cuh"

namespace osscar {
namespace {

using namespace tc;

constexpr int PT_M = 128, PT_BK = 64, PT_UK = 16, PT_NMAX = 128, PT_FLUSH = 2;
constexpr int PT_RAW_BYTES = PT_M * 32 * 4;              // one fp32 box: 128 rows x 128 bytes
constexpr int PT_AT_BYTES = PT_M * PT_BK * 2;            // one bf16 term tile of A
constexpr int PT_THREADS = 320;
constexpr int PT_TMEM_COLS = 256;                        // two accumulators of up to 128 columns

struct PanelMaps { CUtensorMap a; CUtensorMap p[3]; };

// K-major SWIZZLE_128B operand tile (rows of 128 bytes, 8-row atoms 1024 bytes apart); used for both operands.
__device__ __forceinline__ uint64_t pt_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

template <int NCH>       // NCH = padded panel width / 32
__global__ void __launch_bounds__(PT_THREADS, 1)
k_panel_tc(const __grid_constant__ PanelMaps maps, int64_t M, int N, int nkb_total, int kbs, int KS, int num_items,
           float* __restrict__ Y, int64_t so_row, int64_t so_col, float* __restrict__ part,
           SearchCtl* __restrict__ ctl, const int32_t* __restrict__ done)
{
    constexpr int NP = NCH * 32;
    constexpr int P_BYTES = NP * 128;                    // one bf16 term tile of the panel (NP rows x 64 k)
    constexpr int STAGE_BYTES = 3 * PT_AT_BYTES + 3 * P_BYTES;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NP >> 3) << 17) | ((uint32_t)(PT_M >> 4) << 24);
    if (done && *done) return;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw);
    const uint32_t raw_ring = base;                                        // 2 x 16 KB
    const uint32_t stage0 = base + 2 * PT_RAW_BYTES;                       // 2 stages of terms
    uint8_t* bar_ptr = base_ptr + 2 * PT_RAW_BYTES + 2 * STAGE_BYTES;
    const uint32_t bars = base + 2 * PT_RAW_BYTES + 2 * STAGE_BYTES;
    auto raw_full = [&](int h) { return bars + 8u * h; };
    auto raw_empty = [&](int h) { return bars + 8u * (2 + h); };
    auto p_full = [&](int s) { return bars + 8u * (4 + s); };
    auto a_ready = [&](int s) { return bars + 8u * (6 + s); };
    auto stage_free = [&](int s) { return bars + 8u * (8 + s); };
    auto tfull = [&](int b) { return bars + 8u * (10 + b); };
    auto tempty = [&](int b) { return bars + 8u * (12 + b); };
    const uint32_t drain_bar = bars + 8u * 14;           // completion of the MMAs in flight when the issuer gives up
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * 15);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 8 * 15 + 8);
    const long long wl = ctl->wait_limit;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(raw_full(i), 1); mbar_init(raw_empty(i), 4); mbar_init(p_full(i), 1); mbar_init(a_ready(i), 4);
            mbar_init(stage_free(i), 1); mbar_init(tfull(i), 1); mbar_init(tempty(i), 4);
        }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "n"(PT_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    auto item_range = [&](int id, int* tm, int* ks, int* kb0, int* kb1) {
        *tm = id / KS; *ks = id % KS;
        *kb0 = *ks * kbs;
        *kb1 = min(nkb_total, *kb0 + kbs);
    };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            uint32_t n_p[2] = {0, 0}, n_raw[2] = {0, 0};      // copy batches issued per barrier (for the drain of an abort)
            bool ok = true;
            for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
                int tm, ks, kb0, kb1;
                item_range(id, &tm, &ks, &kb0, &kb1);
                for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
                    const int s = it & 1;
                    const uint32_t ph = (it >> 1) & 1;
                    if (!mbar_wait(stage_free(s), ph ^ 1, abort_flag, wl)) { ok = false; break; }
                    mbar_expect_tx(p_full(s), 3 * P_BYTES);
                    const uint32_t p_dst = stage0 + s * STAGE_BYTES + 3 * PT_AT_BYTES;
#pragma unroll
                    for (int term = 0; term < 3; ++term)
                        tma_load_2d(p_dst + term * P_BYTES, &maps.p[term], p_full(s), kb * PT_BK, 0);
                    ++n_p[s];
                    for (int h = 0; h < 2; ++h) {
                        if (!mbar_wait(raw_empty(h), (it & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                        mbar_expect_tx(raw_full(h), PT_RAW_BYTES);
                        tma_load_2d(raw_ring + h * PT_RAW_BYTES, &maps.a, raw_full(h), kb * PT_BK + h * 32, tm * PT_M);
                        ++n_raw[h];
                    }
                }
            }
            if (*abort_flag) {                    // let the copies in flight land before the CTA exits
                for (int i = 0; i < 2; ++i) {     // the n-th batch on a barrier completes its phase n - 1
                    if (n_p[i] > 0) mbar_drain(p_full(i), (n_p[i] - 1) & 1);
                    if (n_raw[i] > 0) mbar_drain(raw_full(i), (n_raw[i] - 1) & 1);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, fl = 0;
            bool ok = true;
            for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
                int tm, ks, kb0, kb1;
                item_range(id, &tm, &ks, &kb0, &kb1);
                const int nflush = (kb1 - kb0 + PT_FLUSH - 1) / PT_FLUSH;
                for (int f = 0; f < nflush && ok; ++f, ++fl) {
                    const int buf = fl & 1;
                    if (!mbar_wait(tempty(buf), ((fl >> 1) & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * PT_NMAX);
                    const int e1 = min(kb1, kb0 + (f + 1) * PT_FLUSH);
                    bool first = true;
                    for (int kb = kb0 + f * PT_FLUSH; kb < e1 && ok; ++kb, ++it) {
                        const int s = it & 1;
                        const uint32_t ph = (it >> 1) & 1;
                        if (!mbar_wait(a_ready(s), ph, abort_flag, wl) || !mbar_wait(p_full(s), ph, abort_flag, wl)) { ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a_src = stage0 + s * STAGE_BYTES;
                        const uint32_t p_src = a_src + 3 * PT_AT_BYTES;
#pragma unroll
                        for (int term = 0; term < 6; ++term) {
                            // term pairs, small products first: (3,1) (2,2) (1,3) (2,1) (1,2) (1,1)
                            const int pa = (0x001012 >> (4 * term)) & 0xF;
                            const int pb = (0x010210 >> (4 * term)) & 0xF;
#pragma unroll
                            for (int j = 0; j < PT_BK / PT_UK; ++j) {
                                umma_f16(d_tmem, pt_desc(a_src + pa * PT_AT_BYTES + j * 32), pt_desc(p_src + pb * P_BYTES + j * 32),
                                         kIdesc, first ? 0u : 1u);
                                first = false;
                            }
                        }
                        umma_commit(stage_free(s));
                    }
                    if (ok) umma_commit(tfull(buf));
                }
            }
            if (!ok) {            // MMAs already issued must finish before TMEM and the operand tiles are released
                umma_commit(drain_bar);
                mbar_drain(drain_bar, 0);
            }
        }
    } else if (warp < 6) {
        // converters: warp cw owns rows [32 cw, 32 cw + 32) of the tile; a lane handles two adjacent k of two rows
        const int cw = warp - 2;
        const int rsub = lane >> 4, c2 = (lane & 15) * 2;
        uint32_t it = 0;
        bool ok = true;
        for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
            int tm, ks, kb0, kb1;
            item_range(id, &tm, &ks, &kb0, &kb1);
            for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
                const int s = it & 1;
                const uint32_t ph = (it >> 1) & 1;
                if (!mbar_wait(stage_free(s), ph ^ 1, abort_flag, wl)) { ok = false; break; }
                uint8_t* at = base_ptr + 2 * PT_RAW_BYTES + s * STAGE_BYTES;
                for (int h = 0; h < 2 && ok; ++h) {
                    if (!mbar_wait(raw_full(h), it & 1, abort_flag, wl)) { ok = false; break; }
                    const uint8_t* rw = base_ptr + h * PT_RAW_BYTES;
                    float2 v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int r = cw * 32 + 2 * i + rsub;
                        v[i] = *reinterpret_cast<const float2*>(rw + r * 128 + c2 * 4);
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int r = cw * 32 + 2 * i + rsub;
                        const int k = h * 32 + c2;
                        const uint32_t off = (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + (((k >> 3) ^ (r & 7)) << 4) + (k & 7) * 2);
                        float x = v[i].x, y = v[i].y;
                        const __nv_bfloat16 x1 = __float2bfloat16_rn(x), y1 = __float2bfloat16_rn(y);
                        x -= __bfloat162float(x1); y -= __bfloat162float(y1);
                        const __nv_bfloat16 x2 = __float2bfloat16_rn(x), y2 = __float2bfloat16_rn(y);
                        x -= __bfloat162float(x2); y -= __bfloat162float(y2);
                        const __nv_bfloat16 x3 = __float2bfloat16_rn(x), y3 = __float2bfloat16_rn(y);
                        *reinterpret_cast<__nv_bfloat162*>(at + off) = __halves2bfloat162(x1, y1);
                        *reinterpret_cast<__nv_bfloat162*>(at + PT_AT_BYTES + off) = __halves2bfloat162(x2, y2);
                        *reinterpret_cast<__nv_bfloat162*>(at + 2 * PT_AT_BYTES + off) = __halves2bfloat162(x3, y3);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(raw_empty(h));          // the box has been consumed
                }
                if (!ok) break;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // tiles written here are read by the MMA unit
                __syncwarp();
                if (lane == 0) mbar_arrive(a_ready(s));
            }
        }
    } else {
        // accumulate warps 6..9: TMEM lane group = warp % 4
        const int lg = warp & 3;
        uint32_t fl = 0;
        bool ok = true;
        for (int id = blockIdx.x; id < num_items && ok; id += gridDim.x) {
            int tm, ks, kb0, kb1;
            item_range(id, &tm, &ks, &kb0, &kb1);
            const int nflush = (kb1 - kb0 + PT_FLUSH - 1) / PT_FLUSH;
            float acc[NP];
#pragma unroll
            for (int j = 0; j < NP; ++j) acc[j] = 0.f;
            for (int f = 0; f < nflush && ok; ++f, ++fl) {
                const int buf = fl & 1;
                if (!mbar_wait(tfull(buf), (fl >> 1) & 1, abort_flag, wl)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * PT_NMAX + c * 32), r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[c * 32 + j] += __uint_as_float(r[j]);
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty(buf));
            }
            if (!ok) break;
            const int64_t row = (int64_t)tm * PT_M + lg * 32 + lane;
            if (row < M) {
                if (KS > 1) {
                    float* dst = part + ((int64_t)ks * M + row) * N;
#pragma unroll
                    for (int j = 0; j < NP; ++j) if (j < N) dst[j] = acc[j];
                } else {
#pragma unroll
                    for (int j = 0; j < NP; ++j) if (j < N) Y[row * so_row + (int64_t)j * so_col] = acc[j];
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(PT_TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) ctl->status = OSSCAR_E_TIMEOUT;
}

// The panel as three bf16 terms, NP rows x K8 columns each (rows >= N and columns >= K are zero).
__global__ void k_split_panel(const float* __restrict__ P, int64_t ldp, int N, int64_t K, int NP, int64_t K8,
                              __nv_bfloat16* __restrict__ t1, __nv_bfloat16* __restrict__ t2, __nv_bfloat16* __restrict__ t3,
                              const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t total = (int64_t)NP * K8;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = idx / K8, k = idx % K8;
        float x = (e < N && k < K) ? P[e * ldp + k] : 0.f;
        const __nv_bfloat16 a = __float2bfloat16_rn(x);
        x -= __bfloat162float(a);
        const __nv_bfloat16 b = __float2bfloat16_rn(x);
        x -= __bfloat162float(b);
        t1[idx] = a; t2[idx] = b; t3[idx] = __float2bfloat16_rn(x);
    }
}

__global__ void k_panel_sum(const float* __restrict__ part, int64_t M, int N, int splits, float* __restrict__ Y,
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

template <int NCH>
cudaError_t launch_panel_tc(cudaStream_t st, int grid, const PanelMaps& maps, int64_t M, int N, int nkb_total, int kbs, int KS,
                            int num_items, float* Y, int64_t so_row, int64_t so_col, float* part, SearchCtl* ctl, const int32_t* done)
{
    constexpr int smem = 2 * PT_RAW_BYTES + 2 * (3 * PT_AT_BYTES + 3 * NCH * 32 * 128) + 1024 + 256;
    cudaError_t e = cudaFuncSetAttribute(k_panel_tc<NCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    k_panel_tc<NCH><<<grid, PT_THREADS, smem, st>>>(maps, M, N, nkb_total, kbs, KS, num_items, Y, so_row, so_col, part, ctl, done);
    return cudaGetLastError();
}

}  // namespace

size_t panel_dot_tc_scratch(int64_t M, int64_t N, int64_t K)
{
    const int64_t K8 = round_up(K, 8);
    return (size_t)3 * 128 * K8 * 2 + 4096 + (size_t)16 * M * (N < 128 ? N : 128) * 4 + 2048;
}

cudaError_t panel_dot_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                         const float* P, int64_t ldp, float* Y, int64_t so_row, int64_t so_col,
                         void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    if (K <= 0 || ((uintptr_t)A & 15) || (lda % 4) != 0 || !scratch) return cudaErrorInvalidValue;
    {   // the term buffers start on a 1024-byte boundary inside the scratch
        const size_t skip = (1024 - ((uintptr_t)scratch & 1023)) & 1023;
        if (scratch_bytes < skip + panel_dot_tc_scratch(M, N, K)) return cudaErrorInvalidValue;
        scratch = (char*)scratch + skip;
    }
    PFN_encodeTiled enc = get_encode();
    if (!enc) return cudaErrorNotSupported;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int64_t K8 = round_up(K, 8);
    const int nkb_total = (int)((K + PT_BK - 1) / PT_BK);
    const int TM = (int)((M + PT_M - 1) / PT_M);
    // k slices: the fewest (at most 16, at least four k-blocks each) that keep the last wave of items at least 90 % full
    int KS = 1;
    for (int c = 1; c <= 16 && nkb_total / c >= 4; ++c) {
        const int items = TM * c, waves = (items + sms - 1) / sms;
        KS = c;
        if ((double)items / ((double)waves * sms) >= 0.9) break;
    }
    const int kbs = (nkb_total + KS - 1) / KS;
    KS = (nkb_total + kbs - 1) / kbs;
    char* sc = (char*)scratch;
    const size_t term_bytes = ((size_t)128 * K8 * 2 + 1023) / 1024 * 1024;
    float* part = (float*)(sc + 3 * term_bytes);
    for (int64_t e0 = 0; e0 < N; e0 += PT_NMAX) {
        const int n = (int)(N - e0 < PT_NMAX ? N - e0 : PT_NMAX);
        const int NCH = (n + 31) / 32, NP = NCH * 32;
        __nv_bfloat16* t[3];
        for (int i = 0; i < 3; ++i) t[i] = (__nv_bfloat16*)(sc + i * term_bytes);
        k_split_panel<<<296, 256, 0, st>>>(P + e0 * ldp, ldp, n, K, NP, K8, t[0], t[1], t[2], done);
        PanelMaps maps;
        {
            const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
            const cuuint64_t strides[1] = {(cuuint64_t)lda * 4};
            const cuuint32_t box[2] = {32, PT_M};
            const cuuint32_t estr[2] = {1, 1};
            if (enc(&maps.a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(A), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        }
        for (int i = 0; i < 3; ++i) {
            const cuuint64_t dims[2] = {(cuuint64_t)K8, (cuuint64_t)NP};
            const cuuint64_t strides[1] = {(cuuint64_t)K8 * 2};
            const cuuint32_t box[2] = {PT_BK, (cuuint32_t)NP};
            const cuuint32_t estr[2] = {1, 1};
            if (enc(&maps.p[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, t[i], dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        }
        const int num_items = TM * KS;
        const int grid = num_items < sms ? num_items : sms;
        float* Yc = Y + e0 * so_col;
        switch (NCH) {
        case 1:  e = launch_panel_tc<1>(st, grid, maps, M, n, nkb_total, kbs, KS, num_items, Yc, so_row, so_col, part, ctl_dev, done); break;
        case 2:  e = launch_panel_tc<2>(st, grid, maps, M, n, nkb_total, kbs, KS, num_items, Yc, so_row, so_col, part, ctl_dev, done); break;
        case 3:  e = launch_panel_tc<3>(st, grid, maps, M, n, nkb_total, kbs, KS, num_items, Yc, so_row, so_col, part, ctl_dev, done); break;
        default: e = launch_panel_tc<4>(st, grid, maps, M, n, nkb_total, kbs, KS, num_items, Yc, so_row, so_col, part, ctl_dev, done); break;
        }
        if (e != cudaSuccess) return e;
        count_launches(2);
        if (KS > 1) {
            const int64_t tot = M * n;
            k_panel_sum<<<(unsigned)((tot + 255) / 256 < 1184 ? (tot + 255) / 256 : 1184), 256, 0, st>>>(part, M, n, KS, Yc, so_row, so_col, done);
            count_launches(1);
        }
    }
    return cudaGetLastError();
}

}  // namespace osscar
