// Internal declarations shared by the translation units of libosscar.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "osscar.h"

namespace osscar {

constexpr int kTracePartials = 1184;   // blocks of a trace reduction; the context owns that many doubles
constexpr int64_t kMaxPairs = 1 << 20;     // PAIR_EXACT scores at most this many (kept, pruned) pairs per step
constexpr int kLoopMaxBlocks = 2048;   // most blocks the persistent swap loop is launched with (size of its candidate lists)
constexpr int kPadF = 32;   // leading dimensions of internal fp32 matrices are padded to this many floats

extern unsigned long long g_launches;      // kernels launched by the library (host-side count)
static inline void count_launches(unsigned long long n) { g_launches += n; }

static inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

// Device-side control block of the swap loop.  Lives in the context's small device allocation.
struct SearchCtl {
    int32_t done;            // set once the loop has stopped; later kernels return at once
    int32_t stop_reason;
    int32_t status;          // OSSCAR_OK or an error raised on the device
    int32_t n_swaps;
    int32_t n_refresh;
    int32_t sel_slot;        // kept slot leaving
    int32_t sel_t;           // pruned slot (0-based among pruned slots) entering
    int32_t pad0;
    double  obj;             // running objective
    double  sel_D;           // drop score of the chosen slot
    double  delta;           // exact change of obj of the chosen swap
    double  const_term;
    double  acc[4];          // scratch accumulators (traces, objective reductions)
    long long wait_limit;    // cycles a bounded device-side wait may spin before it raises OSSCAR_E_TIMEOUT
    unsigned long long bar_count;   // arrivals at the grid barrier of the persistent swap loop (monotone)
    int32_t abort;           // set by a wait that ran out: every block of the persistent loop returns
    int32_t pad1;
};

// Geometry of one layer's search state inside the caller's workspace.
struct Layout {
    int64_t d1, m, ng;       // rows of W, columns of W, number of groups
    int32_t g, k;
    int64_t nI, nJ;          // kept rows, pruned rows
    int64_t ldp;             // leading dimension of Hp (slot-permuted H)
    int64_t ldh;             // leading dimension of Hinv, and padded length of the n_I-vectors
    int64_t ldm;             // leading dimension of V, R, K, Vq
    // offsets in bytes from the workspace base
    size_t off_Hp, off_Hinv, off_V, off_R, off_big;
    size_t off_Hd;                                                     // fp64 copy of the inverse (g = 1 only, else a stub)
    size_t off_y, off_b, off_u2, off_bC, off_u2c, off_u, off_d, off_K, off_Vq;
    size_t off_vec_begin, off_vec_end;   // the staged vectors (zeroed once when the state is built)
    size_t off_vnorm, off_rnorm, off_D, off_A, off_c, off_small, off_gramV, off_gramR;
    size_t off_perm, off_slotof, off_energy, off_panel;
    size_t off_shard;                                                  // column shards: partial sums handed to the reduce hook
    size_t off_loop;                                                   // persistent swap loop: per-block candidates, phase timers
    size_t off_pairCinv, off_pairKK, off_pairScratch, off_pairDelta;   // PAIR_EXACT scoring
    size_t off_greedy;                                                 // scratch of the nested (greedy) phase
    size_t off_tc, tc_bytes;                                           // bf16 operand terms of the tensor-core GEMMs
    size_t off_block, block_bytes;                                     // panels of the block exchange (search_block.cuh)
    int32_t block_rows_max;                                            // largest s*g the block region holds
    int64_t pair_capacity;                                             // pairs the workspace can score
    size_t bytes;
};
// bytes of the block-exchange panels for G rows on each side (layout in search_block.cuh)
static inline size_t block_region_bytes(int64_t ldh, int64_t ldm, int64_t nJ, int64_t G)
{
    auto al = [](size_t b) { return (b + 255) / 256 * 256; };
    size_t n = 2 * al(sizeof(int32_t) * (size_t)G);
    n += 3 * al(sizeof(float) * (size_t)G * ldh);            // hT, yT, HrT
    n += 4 * al(sizeof(float) * 2 * (size_t)G * ldh);        // PB, PA and their transposes
    n += al(sizeof(float) * 2 * (size_t)G * ldm);            // KV
    n += 2 * al(sizeof(float) * (size_t)G * ldm);            // Vr, Rq
    n += al(sizeof(float) * (size_t)(nJ + G) * 2 * G);       // UD
    n += al(sizeof(double) * 18 * (size_t)G * G);            // small matrices
    return n;
}
int make_layout(int64_t d1, int64_t m, int32_t g, int32_t k, Layout* L);

}  // namespace osscar

struct osscar_ctx {
    int device;
    cudaStream_t stream;
    osscar::SearchCtl* ctl;          // device
    osscar::SearchCtl* ctl_host;     // pinned mirror
    double* partials;                // device, kTracePartials doubles: stage 1 of deterministic reductions
    volatile int32_t* done_flag_host; // pinned, device-mapped: copy of ctl->done pushed by the device
    int32_t* done_flag_dev;          // device alias of done_flag_host
    void* ws;
    size_t ws_bytes;
    osscar::Layout L;
    bool have_state;
    const float* H;                  // caller's matrices bound by init_support
    const float* G;
    const float* W;
    cudaEvent_t ev0, ev1;
    double gram_rows;                // rows accumulated since GRAM_BEGIN (bookkeeping only)
    bool have_const;                 // const term supplied by the caller (cross-term problems) instead of Tr(W^T G)
    double user_const;
    long long wait_limit;            // context default of SearchCtl::wait_limit
    bool hd_valid;                   // the fp64 copy of the inverse matches the state
    osscar_reduce_fn reduce;         // column shards: in-place sum over shards, enqueued by the caller's hook (or null)
    void* reduce_user;
};

namespace osscar {

// ---- sgemm.cu: C = alpha * op(A) * B + beta * C on the fp32 pipes ----------------------------
// A is M x K (lda) or, with transA, stored K x M; B is K x N (ldb) or, with transB, stored N x K.
// `done` (may be null): device flag; when non-zero the kernel returns without touching C.
cudaError_t sgemm(cudaStream_t st, bool transA, bool transB, int64_t M, int64_t N, int64_t K,
                  float alpha, const float* A, int64_t lda, const float* B, int64_t ldb,
                  float beta, float* C, int64_t ldc, const int32_t* done = nullptr);

// ---- dgemm.cu: C = beta * C0 + alpha * A * B (or I + alpha * A * B) with fp32 operands, products and sums in fp64;
// A (M x K) and B (K x N) row-major, C0 may alias C.
cudaError_t gemm_f64acc(cudaStream_t st, int64_t M, int64_t N, int64_t K, double alpha, const float* A, int64_t lda,
                        const float* B, int64_t ldb, double beta, const float* C0, int64_t ldc0, float* C, int64_t ldc,
                        bool identity_plus, const int32_t* done = nullptr);
cudaError_t gemm_f64out(cudaStream_t st, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                        const float* B, int64_t ldb, double* C, int64_t ldc, const int32_t* done = nullptr, bool tri = false);

// ---- panel_tc.cu: Y[i*so_row + e*so_col] = sum_k A[i][k] * P[e][k] on the tensor cores; A (M x K, streamed once) is split
// into bf16 terms on the way (fp32-accurate); P is an N x K panel
// A 16-byte aligned with lda % 4 == 0; scratch at least panel_dot_tc_scratch bytes.
size_t panel_dot_tc_scratch(int64_t M, int64_t N, int64_t K);
cudaError_t panel_dot_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, const float* A, int64_t lda,
                         const float* P, int64_t ldp, float* Y, int64_t so_row, int64_t so_col,
                         void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done = nullptr);

// ---- gemm_tc.cu: the same product on the tensor cores (three-term bf16 split, fp32-accurate); A and B row-major.
// `scratch` (256-byte aligned device memory, at least gemm_tc_min_scratch bytes) holds the bf16 terms of one K panel.
size_t gemm_tc_min_scratch(int64_t M, int64_t N);
cudaError_t gemm_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, float alpha, const float* A, int64_t lda,
                    const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                    void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done = nullptr);

// C += alpha * A * B for a short inner dimension (K <= 128 keeps the terms of A's row band in shared memory across a run
// of column tiles; larger K goes through gemm_tc).  Same operands and scratch as gemm_tc.  With row_sq (M floats) and
// sq_scratch (M * 2 * ceil(N / 128) floats) the squared norms of the updated rows are produced in the same pass (K <= 128 only).
cudaError_t rank_update_tc(cudaStream_t st, int64_t M, int64_t N, int64_t K, float alpha, const float* A, int64_t lda,
                           const float* B, int64_t ldb, float* C, int64_t ldc,
                           void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev, const int32_t* done = nullptr,
                           float* row_sq = nullptr, float* sq_scratch = nullptr);

// H (+)= Xc^T Xc (upper-triangle tiles; Y null) or G (+)= Xc^T Yc with the drained-accumulator pipeline of gemm_tc.cu.
cudaError_t gram_tc2(cudaStream_t st, const void* X, int64_t n_rows, int64_t d1, const void* Y, int y_fp32, int64_t m,
                     float* C, bool accumulate, void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev);
// H (+)= Xc^T Xc for fp32 Xc on the tensor cores (three-term bf16 split staged in `scratch`, row panels sized to it);
// cudaErrorMemoryAllocation when the scratch is too small for one panel.
cudaError_t gram_tc3(cudaStream_t st, const float* X, int64_t n_rows, int64_t d1, float* C, bool accumulate,
                     void* scratch, size_t scratch_bytes, SearchCtl* ctl_dev);

// ---- gram_tc.cu ---------------------------------------------------------------------------------------------
cudaError_t set_device_double(cudaStream_t st, double* dst, double v);          // *dst = v on the stream
cudaError_t gram_mirror(cudaStream_t st, float* H, int64_t d1);   // copy upper triangle to lower

// ---- state.cu: support selection and state construction --------------------------------------
int select_support(osscar_ctx* ctx, int mode, int32_t* support);
int build_state(osscar_ctx* ctx, bool guarded);
int invert_spd_inplace(osscar_ctx* ctx, float* A, int64_t lda, int64_t n, const float* ref, int64_t ldref, const int32_t* done,
                       bool tensor_updates);
cudaError_t gather_rows(cudaStream_t st, const float* src, int64_t m, int g, const int32_t* perm,
                        int64_t slot_row0, int64_t nrows, float* dst, int64_t ld);
cudaError_t trace_product(cudaStream_t st, const float* A, int64_t lda, const float* B, int64_t ldb,
                          int64_t rows, int64_t cols, double* partials, double* out_dev);   // *out = sum A.*B

// ---- greedy.cu: nested phase of Algorithm 1 down to L.k groups (leaves the slot permutation in the workspace) -----
size_t greedy_scratch_bytes(int64_t d1, int64_t m, int g);
int greedy_support(osscar_ctx* ctx, int t_hat, int32_t* support, int32_t* drop_trace, int32_t* n_iters_out);

// ---- search.cu -------------------------------------------------------------------------------
int run_search(osscar_ctx* ctx, const osscar_search_params* p, int32_t* support_out, float* W_out,
               double* obj_trace, int32_t* swap_trace, osscar_search_result* res);
cudaError_t score_pass(osscar_ctx* ctx);   // full scoring pass from the current state (fills D, A)
// fp64 copy of the inverse from the fp32 one by a Newton-Schulz step summed in fp64 (single-row groups; uses `big`)
int build_hinv64(osscar_ctx* ctx, bool guarded);
// column shards: sum `count` values of `buf` (inside the workspace) over all shards through the context's hook
int shard_reduce(osscar_ctx* ctx, void* buf, int64_t count, int dtype);

}  // namespace osscar
