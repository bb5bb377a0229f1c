/*
 * osscar.h -- C ABI of the B200 implementation of the OSSCAR per-layer solve
 * (one-shot structured pruning as a combinatorial problem, arXiv 2403.12983).
 *
 * Problem (Section 2, Eq. MIQP; Section 3.1, Eq. deff/struc).  A layer has a dense weight
 * W_hat (d1 x m) and calibration inputs X (n x d1).  The rows of W_hat are split into
 * d1/g contiguous groups of g rows (one per input neuron, per conv input channel or per
 * attention head); group q holds rows q*g .. q*g+g-1 (0-based).  Exactly k groups may stay
 * non-zero.  With H = X^T X and G = H W_hat, the reconstruction error of a kept set S is
 *     obj(S) = min_W ||X W_hat - X W||_F^2 = const - Tr(G_I^T (H_II)^-1 G_I),
 * I = rows of the kept groups, const = Tr(W_hat^T H W_hat)  (Eq. optf; obj = 2 f + const,
 * with the paper's S being the complementary, pruned set).  The library builds H and G,
 * picks a starting support and runs the swap form of Algorithm 1 (t_hat = 2, p_hat = 0) on
 * the device, moving (H_II)^-1, the optimal weights and the residual with the low-rank
 * identities of Proposition 1 instead of re-solving.
 *
 * Conventions.  All matrices are dense, row-major, leading dimension = number of columns.
 * "device" / "host" says where a pointer must live.  The caller owns every buffer; the
 * library allocates only a small control block per context.  Every call returns a status
 * (OSSCAR_OK or a negative error); nothing throws, aborts or traps.  Work is enqueued on the
 * context's stream; a call synchronises that stream once, at its end, iff it has host
 * outputs.  A failed call leaves its outputs unspecified and the context usable.
 * There is no CPU path: without a CUDA device every call fails with OSSCAR_E_CUDA.
 */
#ifndef OSSCAR_H_
#define OSSCAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct osscar_ctx osscar_ctx;

enum {
    OSSCAR_OK = 0,
    OSSCAR_E_ARG = -1,        /* null pointer, bad enum, bad flag                           */
    OSSCAR_E_SHAPE = -2,      /* sizes inconsistent (d1 % g, k out of range, g too large)   */
    OSSCAR_E_NOTPD = -3,      /* H restricted to the kept rows is not positive definite     */
    OSSCAR_E_WORKSPACE = -4,  /* workspace missing or too small                             */
    OSSCAR_E_CUDA = -5,       /* a CUDA runtime/driver call failed                          */
    OSSCAR_E_TIMEOUT = -6,    /* a bounded device-side wait ran out                         */
    OSSCAR_E_STATE = -7       /* call order violated (e.g. search before init)              */
};
enum { OSSCAR_BF16 = 0, OSSCAR_FP32 = 1 };
enum { OSSCAR_GRAM_BEGIN = 1, OSSCAR_GRAM_END = 2 };
enum { OSSCAR_INIT_ENERGY = 0, OSSCAR_INIT_MAGNITUDE = 1, OSSCAR_INIT_USER = 2 };
enum { OSSCAR_SCORE_INDEPENDENT = 0, OSSCAR_SCORE_PAIR_EXACT = 1 };
enum { OSSCAR_ACCEPT_IMPROVING = 0, OSSCAR_ACCEPT_ALWAYS = 1 };
enum { OSSCAR_STOP_MAX_SWAPS = 0, OSSCAR_STOP_NO_IMPROVEMENT = 1, OSSCAR_STOP_GUARD = 2 };
/* Swap loop of single-row groups.  PERSISTENT = one cooperative kernel that runs all steps with bounded grid-wide
 * barriers between their phases (OSSCAR_E_ARG if the device cannot launch cooperatively); LAUNCHES = five dependent
 * launches per step, enqueued ahead of the device; AUTO = PERSISTENT for states that fit the L2 cache (under 96 MB),
 * LAUNCHES for states streamed from HBM. */
enum { OSSCAR_LOOP_AUTO = 0, OSSCAR_LOOP_PERSISTENT = 1, OSSCAR_LOOP_LAUNCHES = 2 };

#define OSSCAR_MAX_GROUP 96   /* largest supported group size g */

/* Context bound to one device and one stream (a cudaStream_t passed as void*, NULL = the
 * legacy default stream).  create allocates a few KB of device and pinned host memory. */
int osscar_create(osscar_ctx** out, int device, void* cuda_stream);
int osscar_destroy(osscar_ctx* ctx);

/* Budget, in SM clock cycles, of every bounded device-side wait of kernels launched through this context (mbarrier
 * waits of the tensor-core pipelines, grid barriers of the persistent swap loop).  A wait that runs out makes its
 * kernel return early and the call that reads the device status return OSSCAR_E_TIMEOUT; the context stays usable
 * and the outputs of that call are unspecified.  0 restores the default (4e9 cycles, about two seconds).  Waits a
 * kernel makes, while giving up, for its own copies and tensor-core work in flight keep the default budget. */
int osscar_set_wait_limit(osscar_ctx* ctx, uint64_t cycles);

/*
 * Column shards (Section 2, convolutional-layer paragraph: the outputs of two filters are independent given the
 * kept set, so the columns of W_hat -- and with them G, the optimal weights and the residual -- split across devices).
 * A context that has a reduce hook holds the columns [c0, c0 + m) of one layer: it is given its own m columns of
 * W_hat and G and the whole of H.  The kept set, (H_II)^-1, the slot-permuted H and the Schur complements are then
 * replicated (every shard computes the same values), while the row norms of the weights and of the residual, the
 * cross term of the chosen pair, the group energies and the objective are sums over columns: the library leaves each
 * shard's partial sums in a buffer inside the caller's workspace and calls
 *     reduce(user, dev_buf, count, dtype, cuda_stream)        dtype: OSSCAR_FP32 or OSSCAR_FP64 (doubles)
 * from the host thread of the API call, in stream order; the hook must enqueue on `cuda_stream` an in-place sum of
 * dev_buf over all shards (ncclAllReduce, or torch.distributed.all_reduce on a view of the workspace) and return 0.
 * Two calls per swap (one double; d1 floats), none of them synchronises the host.  Every shard must make the same
 * calls in the same order.  Supported: single-row groups (g = 1), OSSCAR_SCORE_INDEPENDENT, one swap per step,
 * OSSCAR_INIT_ENERGY / MAGNITUDE / USER; anything else returns OSSCAR_E_ARG while a hook is set.  Results: support and
 * traces are identical on every shard, W_out holds the shard's columns, objectives are those of the whole layer.
 * fn = NULL removes the hook.
 */
typedef int (*osscar_reduce_fn)(void* user, void* dev_buf, int64_t count, int dtype, void* cuda_stream);
enum { OSSCAR_FP64 = 2 };
int osscar_set_shard_reduce(osscar_ctx* ctx, osscar_reduce_fn fn, void* user);

/* Scratch needed by init_support / local_search / objective for a layer of this shape.
 * The caller allocates it on the device (256-byte aligned) and lends it with set_workspace;
 * it must stay alive, and untouched by others, from init_support to the end of local_search. */
int osscar_workspace_bytes(int64_t d1, int64_t m, int32_t g, int32_t k, size_t* bytes /*host*/);
int osscar_set_workspace(osscar_ctx* ctx, void* dev_ptr, size_t bytes);

/*
 * Gram and cross term of a dense layer (Section 2, dense-layer paragraph: H = X^T X,
 * G = X^T X W_hat; conv layers pass the unfolded patch matrix, attention/FC2 layers the
 * token activations).  X is given in row blocks ("chunks" of tokens):
 *   flags & BEGIN : H := Xc^T Xc, otherwise H += Xc^T Xc   (split over calibration rows);
 *   flags & END   : H += damp * mean(diag H) * I (damp = 0: none; not in the paper),
 *                   G := H W_hat, *const_term := Tr(W_hat^T G), then one stream sync.
 *                   With a workspace set, G is formed on the tensor cores (three-term bf16 split, fp32-accurate)
 *                   and the workspace contents are overwritten; without one it runs on the fp32 pipes.
 * X: device, n_rows x d1, bf16 (tensor cores, fp32 accumulation) or fp32.  For bf16 the
 * pointer must be 16-byte aligned and d1 a multiple of 8.  fp32 X with a workspace set is split into three bf16
 * terms there (row panels of 6 * round_up(d1, 8) bytes per row, workspace contents overwritten) and accumulated on
 * the tensor cores to fp32 accuracy; without a workspace it runs on the fp32 pipes.
 * W: device d1 x m fp32 (read on END).
 * H: device d1 x d1 fp32, G: device d1 x m fp32, const_term: host (written on END).
 * n_rows may be 0 (nothing is added).
 */
int osscar_gram(osscar_ctx* ctx, const void* X, int x_dtype, int64_t n_rows, int64_t d1,
                const float* W, int64_t m, int flags, float damp,
                float* H, float* G, double* const_term);

/*
 * Gram and cross term for sequential layer-wise pruning (Appendix B.1, "Pruning strategies": the layer's target is
 * the DENSE model's output, its input the PRUNED model's activations): with X the pruned model's input block and
 * Y = X_hat W_hat the dense model's output block (n_rows x m),
 *     H (+)= Xc^T Xc,   G (+)= Xc^T Yc,   const (+)= ||Yc||_F^2,
 * so that obj(S) = min_W ||Y - X W||_F^2 = const - Tr(G_I^T (H_II)^-1 G_I).  Flags and damp as in osscar_gram (damping
 * touches H only).  X: bf16 (d1 % 8 == 0, 16-byte aligned) or fp32; Y: bf16 (m % 8 == 0) or fp32 (fp32 Y with bf16 X
 * is split into three bf16 terms in the workspace, which must hold 6 * n_rows * round_up(m, 8) bytes and is
 * overwritten); fp32 X requires fp32 Y, and with a workspace set its H runs on the tensor cores as in osscar_gram
 * (workspace contents overwritten), G on the fp32 pipes.  On END *const_term is written and remembered by the context: the following
 * init / search calls use it in place of Tr(W_hat^T G).  osscar_set_const_term sets or clears that value by hand
 * (e.g. when H and G come from elsewhere).
 */
int osscar_gram_cross(osscar_ctx* ctx, const void* X, int x_dtype, const void* Y, int y_dtype,
                      int64_t n_rows, int64_t d1, int64_t m, int flags, float damp,
                      float* H, float* G, double* const_term);
int osscar_set_const_term(osscar_ctx* ctx, double const_term, int enabled);

/*
 * Starting support and search state (Algorithm 1, line 1, for a k-group support instead of
 * the dense start).  mode ENERGY keeps the k groups with the largest Tr(W_q^T H_qq W_q),
 * MAGNITUDE the k largest ||W_q||_F^2 (the paper's MP rule, Appendix B.1), ties to the
 * smaller id; USER reads k distinct ids from `support`.  Builds (H_II)^-1, V = (H_II)^-1 G_I
 * (Eq. tmp5), the residual R = G - H[:,I] V and the Schur complements of every pruned group
 * (the C^-1 of Case 2 in the proof of Proposition 1) in the workspace.
 * H, G, W: device, as produced by osscar_gram (H symmetric).  support: device int32[k],
 * sorted ids on return.  obj0: host, obj of the starting support.  Synchronises once.
 * Errors: E_NOTPD if a pivot block of H_II fails its Cholesky factorisation.
 */
int osscar_init_support(osscar_ctx* ctx, const float* H, const float* G, const float* W,
                        int64_t d1, int64_t m, int32_t g, int32_t k, int mode,
                        int32_t* support, double* obj0);

/*
 * Starting support by the nested (greedy) phase of Algorithm 1 (t_i = p_i = t_hat; the paper's own schedule:
 * Appendix B.1 uses t_hat = 2 for channels and heads, 10 for FC neurons).  All d1/g groups start kept, with
 * H^-1 and W* = H^-1 G (Algorithm 1, line 1); each iteration prunes the t_hat kept groups whose removal raises
 * obj least (Eq. impact, evaluated by Case 1 of Proposition 1 / Lemma A.1), all chosen from the scores of the
 * current support, and moves H_II^-1 and W^(S) with the joint Case-1 downdate; the last iteration prunes only
 * what is left.  When k groups remain the search state is built as in osscar_init_support, so
 * osscar_local_search can follow (the paper's "non-nested" refinement).
 * t_hat * g <= 256, else OSSCAR_E_SHAPE.  support: device int32[k] (sorted ids on return).  drop_trace: device
 * int32[d1/g - k] or NULL, the pruned groups in pruning order (inside an iteration by increasing score).
 * obj0: host, obj of the k-group support.  n_iters: host or NULL.  Needs the workspace; synchronises once.
 */
int osscar_init_support_greedy(osscar_ctx* ctx, const float* H, const float* G, const float* W,
                               int64_t d1, int64_t m, int32_t g, int32_t k, int32_t t_hat,
                               int32_t* support, int32_t* drop_trace, double* obj0, int32_t* n_iters);

typedef struct {
    int32_t max_swaps;        /* >= 0                                                        */
    int32_t score_mode;       /* OSSCAR_SCORE_*                                              */
    int32_t accept_mode;      /* OSSCAR_ACCEPT_*                                             */
    int32_t refresh_every;    /* rebuild the state from H every this many steps (swaps, or iterations of a block exchange); 0 = never */
    double  accept_rel_tol;   /* IMPROVING: accept iff delta <= -tol * obj (1e-5 if < 0)     */
    int32_t profile_samples;  /* time each kernel of this many evenly spaced steps (0..8)    */
    int32_t block_pairs;      /* s: groups exchanged per iteration (0 or 1: one swap per step) */
    int32_t loop_mode;        /* OSSCAR_LOOP_*: how the swap loop of single-row groups is driven */
    int32_t reserved;         /* 0 */
    uint64_t wait_limit_cycles; /* budget of the bounded device-side waits of this search; 0 = the context's value */
} osscar_search_params;

#define OSSCAR_NUM_STEP_KERNELS 12   /* select, pair Grams, y pass, small algebra, staging, H pass,
                                        Hinv update, V update, R update, group scores, H row swap, H column swap */

typedef struct {
    int32_t n_swaps, stop_reason, n_refresh, status;
    double  obj_init, obj_final;     /* obj_final is recomputed from the final state         */
    float   ms_search;               /* device time of the swap loop                         */
    int32_t n_profiled;              /* steps that were timed kernel by kernel and did a swap */
    float   ms_kernel[OSSCAR_NUM_STEP_KERNELS]; /* mean device time of each kernel over those steps */
    int32_t loop_driver;             /* OSSCAR_LOOP_PERSISTENT or OSSCAR_LOOP_LAUNCHES: what drove the loop  */
} osscar_search_result;

/*
 * Swap search (Section 3.2: Eq. local with t_hat = 2, p_hat = 0; scores of Eq. impact;
 * state moved by Cases 1-3 of Proposition 1).  Each step scores every kept group (rise of
 * obj if dropped) and every pruned group (fall of obj if added), takes the cheapest drop and
 * the most valuable add (PAIR_EXACT: the pair with the best exact change among all k * (d1/g - k) pairs,
 * which must not exceed 2^20, else OSSCAR_E_SHAPE), computes the exact change of obj
 * for that pair, applies the accept rule and updates the state; the loop runs on the device
 * with no host round trip per swap.
 * support_out: device int32[k] (sorted).  W_out: device d1 x m fp32, rows of pruned groups
 * zero.  obj_trace: device double[max_swaps+1], entry 0 = starting obj.  swap_trace: device
 * int32[2*max_swaps], (group out, group in) per accepted swap.  result: host.
 * Synchronises once at the end.
 * block_pairs = s > 1 (Eq. local with t_hat = 2 s, p_hat = 0, so s_1 = s_2 = s in the rule after Eq. impact;
 * Appendix B.1 uses t_hat up to 100 for FC neurons): each iteration takes the s cheapest drops and the s most
 * valuable adds, all from the scores at the current support, and moves the state with one rank-(2 s g) update;
 * the accept rule applies to the exact change of the whole exchange.  INDEPENDENT scores only; needs
 * s <= min(k, d1/g - k) and s * g <= OSSCAR_MAX_GROUP (else OSSCAR_E_ARG).  floor(max_swaps / s) iterations at
 * most; n_swaps counts groups (s per iteration), swap_trace lists the s pairs of an iteration in order
 * (cheapest drop with best add first) and obj_trace has one entry per ITERATION after entry 0.
 */
int osscar_local_search(osscar_ctx* ctx, const osscar_search_params* params,
                        int32_t* support_out, float* W_out,
                        double* obj_trace, int32_t* swap_trace,
                        osscar_search_result* result);

/* Tr((W - Wt)^T H (W - Wt)) for any candidate Wt (Eq. obj-ver2 re-centred at W_hat); does not
 * touch the search state but uses the workspace (2*d1*m floats at its start are overwritten,
 * so call it before init_support or after local_search).  H, W, Wt: device; obj: host. */
int osscar_objective(osscar_ctx* ctx, const float* H, const float* W, const float* Wt,
                     int64_t d1, int64_t m, double* obj);

/* Test hook (not part of the contract): copy one piece of the search state to `dst` (device).
 * which: 0 Hinv (n_I x n_I), 1 V (n_I x m), 2 R of pruned slots (n_J x m), 3 c (double,
 * (d1/g-k) x g x g), 4 slot->group permutation (int32[d1/g]), 5 drop scores (double[k]),
 * 6 add scores (double[d1/g-k]).  Scores are those of the last scoring pass. */
int osscar_debug_get_state(osscar_ctx* ctx, int which, void* dst);

/*
 * Allocation-free trace reduction (the paper has no counterpart; this is a service entry point).
 * *out = sum_ij A[i][j] * B[i][j] over rows x cols, in fp64 and in a fixed summation order -- for instance
 * const = Tr(W^T G) or the identity obj = Tr(W_J^T R_J).  It is the two-stage reduction the library uses
 * internally, except that its scratch (one double per row) is a fixed array inside the library image instead
 * of memory from cudaMalloc.  It is meant for callers that must not allocate while they run: code that has
 * already handed all free device memory to its own pool, real-time loops that cannot afford the device-wide
 * synchronisation an allocation may cause, or plug-ins that are forbidden to change the memory footprint.
 * It needs no context and calls neither cudaMalloc nor cudaFree nor any allocating library routine.
 *   A, B: device fp32, row-major with leading dimensions lda, ldb >= cols.  out: host.
 *   rows <= OSSCAR_NOALLOC_MAX_ROWS, else OSSCAR_E_SHAPE (the built-in scratch is 65536 + 32 doubles,
 *   about 512 KB, resident on every GPU that loads the library until the process exits).
 *   device: ordinal that owns A and B; cuda_stream: a cudaStream_t (NULL = legacy default stream).
 *   A or B not on `device`: OSSCAR_E_ARG.
 * The first call on a device looks up the device address of the built-in array, and it may also be the moment the
 * CUDA runtime loads this library's kernels onto the device (which allocates inside the driver); make that
 * warm-up call before any stream capture begins and before the no-allocation regime starts.  All calls share the array and it keeps the previous call's contents (each call
 * overwrites every slot it later reads, so old contents never reach the result); calls whose kernels can
 * overlap on the GPU -- different streams, different threads -- race on it and must be serialised by the caller.
 * Synchronises the stream once, at its end.
 */
#define OSSCAR_NOALLOC_MAX_ROWS 65536
int osscar_trace_noalloc(const float* A, int64_t lda, const float* B, int64_t ldb,
                         int64_t rows, int64_t cols, int device, void* cuda_stream, double* out);

const char* osscar_status_string(int status);

/* Number of kernels this library has launched in this process so far (all contexts). */
uint64_t osscar_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* OSSCAR_H_ */
