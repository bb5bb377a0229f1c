// Persistent swap loop for single-row groups (g = 1, independent scores): ONE cooperative kernel runs every step of the
// search.  Included by search.cu after search_g1.cuh (same translation unit: uses its Ptrs, scalar slots and helpers).
//
// A step has four phases, separated by grid-wide barriers (all blocks are co-resident: cooperative launch):
//   P0  every block, redundantly and identically: the leaving slot r (arg-min of the per-block candidates of D), the
//       cross term V_r . R_q, the exact change of obj, the accept test; block 0 records the swap.  Then the staged
//       vectors b = Hinv[r, :], u2 = y - b y_r / C, K = V_r / C, Vq = (R_q + (y_r / C) V_r) / c1, each block a slice.
//   P1  H pass (u_l, d_l of every pruned row and of the leaving row)  ||  V' = V - b K - u2 Vq with its row norms and
//       drop scores D; every block keeps the best D among its rows.
//   P2  R' = R + u K - d Vq with row norms, Schur complements c' and add scores A (best A per block)  ||  exchange of
//       the two slots in Hp (the slot permutation itself is exchanged by block 0 in P0).
//   P3  every block: entering slot of the NEXT step (arg-max of the per-block candidates of A); then
//       Hinv' = Hinv - (b / C) b^T + (u2 / c1) u2^T fused with y_next = Hinv' Hp[q_next, 0:n_I]^T.
// Blocks walk the rows of a phase with a grid stride; a block takes PL_RB rows per pass when rows are short, so that a
// thread keeps up to PL_P 16-byte loads in flight, and the scalars a row's epilogue needs are requested together with
// the row.  Every barrier wait is bounded by ctl->wait_limit cycles: the block that runs out sets ctl->abort and
// OSSCAR_E_TIMEOUT, every other block sees the flag in its own wait, and all return.
#pragma once

constexpr int PL_T = 256;          // threads per block
constexpr int PL_P = 8;            // 16-byte loads a thread keeps in flight per pass over two or four short rows
constexpr int PL_P1 = 9;           // the same for one long row per pass: 9 x 256 x 4 floats cover n_I = 8602 in one pass
template <int RB> struct PlPieces { static constexpr int value = RB == 1 ? PL_P1 : PL_P / RB; };

struct LoopCand { double val; int32_t id; int32_t idx; };

struct LoopArgs {
    Ptrs p;
    LoopCand* candD;               // per block: cheapest drop among the rows it updated
    LoopCand* candA;               // per block: most valuable add among the rows it updated
    unsigned long long* prof;      // [0..3] nanoseconds spent in P0..P3 (block 0), [4] steps counted
    double* obj_trace;
    int32_t* swap_trace;
    double tol;
    int accept_mode;
    int max_steps;                 // steps this launch may run
    int max_swaps;                 // the loop ends when ctl->n_swaps reaches this
};

struct StepScal {                  // scalars of a step, identical in every block
    int64_t r0, t;                 // leaving kept slot, entering pruned slot
    float Cinv, c1inv, Q1, M2;     // 1/C, 1/c1, y_r / C, y_r / (C c1)
    double Cinv_d, c1inv_d, hdiag; // the same in double, H diagonal entry of the leaving row
    float dr;                      // d of the leaving row (valid after P1)
};

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* ptr) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ int ld_volatile_s32(const int32_t* ptr) {
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Grid-wide barrier over `nblocks` co-resident blocks on the monotone counter ctl->bar_count (zeroed by the host
// before the launch); `epoch` is the count this block expects after the barrier.  Returns false when the wait ran out
// or another block gave up.
__device__ __forceinline__ bool grid_barrier(SearchCtl* ctl, unsigned long long& epoch, unsigned nblocks, long long limit, int* s_flag)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        epoch += nblocks;
        __threadfence();
        atomicAdd(&ctl->bar_count, 1ULL);
        const long long t0 = clock64();
        int bad = 0;
        while (ld_acquire_u64(&ctl->bar_count) < epoch) {
            if (ld_volatile_s32(&ctl->abort)) { bad = 1; break; }
            if (clock64() - t0 > limit) {
                atomicExch(&ctl->abort, 1);
                ctl->status = OSSCAR_E_TIMEOUT;
                bad = 1;
                break;
            }
        }
        __threadfence();
        *s_flag = bad;
    }
    __syncthreads();
    return *s_flag == 0;
}

// lexicographic "better" for minimisation with ties to the smaller group id
__device__ __forceinline__ bool cand_less(double v, int id, double bv, int bid) { return v < bv || (v == bv && id < bid); }

// Arg-min over the per-block candidates (negate: arg-max); every thread of warp 0 takes part, result in lane 0.
__device__ __forceinline__ void reduce_cands(const LoopCand* cand, unsigned nblocks, bool negate, double* val, int* idx)
{
    const int lane = threadIdx.x & 31;
    double best = INFINITY; int bid = INT_MAX, bidx = -1;
    for (unsigned i = lane; i < nblocks; i += 32) {
        const LoopCand c = cand[i];
        const double v = negate ? -c.val : c.val;
        if (c.idx >= 0 && cand_less(v, c.id, best, bid)) { best = v; bid = c.id; bidx = c.idx; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oid = __shfl_xor_sync(0xffffffffu, bid, o), oidx = __shfl_xor_sync(0xffffffffu, bidx, o);
        if (cand_less(ov, oid, best, bid)) { best = ov; bid = oid; bidx = oidx; }
    }
    *val = negate ? -best : best;
    *idx = bidx;
}

// Sums of RB values over the block (PL_T threads); result r in every thread's out[r].
template <int RB>
__device__ __forceinline__ void block_sums(float (&v)[RB], float* red /*[RB * 8]*/)
{
#pragma unroll
    for (int r = 0; r < RB; ++r) v[r] = warp_sum(v[r]);
    __syncthreads();                       // the previous use of `red` is over
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int r = 0; r < RB; ++r) red[r * 8 + (threadIdx.x >> 5)] = v[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < PL_T / 32; ++i) t += red[r * 8 + i];
        v[r] = t;
    }
}

template <int RB>
__device__ __forceinline__ void block_sums_d(double (&v)[RB], double* red /*[RB * 8]*/)
{
#pragma unroll
    for (int r = 0; r < RB; ++r) v[r] = warp_sum(v[r]);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int r = 0; r < RB; ++r) red[r * 8 + (threadIdx.x >> 5)] = v[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        double t = 0.0;
#pragma unroll
        for (int i = 0; i < PL_T / 32; ++i) t += red[r * 8 + i];
        v[r] = t;
    }
}

// P1 / P2 row updates.  kind 0: V'[s] = V[s] - b[s] K - u2[s] Vq (row r0 := Vq), D'[s];
// kind 1: R'[l] = R[l] + u[l] K - d[l] Vq (row t := K - d_r Vq), c'[l], A'[l].  RB rows per pass, grid stride.
template <int RB>
__device__ __noinline__ void pl_update_rows(const Ptrs& p, const int kind, const StepScal& sc, unsigned nblocks,
                                               float* red, LoopCand* s_best /*[4]*/)
{
    constexpr int PP = PlPieces<RB>::value;
    float* M = kind == 0 ? p.V : p.R;
    const int64_t nrows = kind == 0 ? p.nI : p.nJ;
    const int64_t special = kind == 0 ? sc.r0 : sc.t;
    const int64_t n4 = p.ldm / 4;
    const float4* K4 = reinterpret_cast<const float4*>(p.K);
    const float4* Q4 = reinterpret_cast<const float4*>(p.Vq);
    const int tid = threadIdx.x;
    for (int64_t rows0 = (int64_t)blockIdx.x * RB; rows0 < nrows; rows0 += (int64_t)nblocks * RB) {
        float4* row[RB];
        int64_t srow[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            srow[r] = rows0 + r < nrows ? rows0 + r : nrows - 1;
            row[r] = reinterpret_cast<float4*>(M + srow[r] * p.ldm);
        }
        float nrm[RB], ck[RB], cq[RB];
        bool sp[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) nrm[r] = 0.f;
        // epilogue scalars of row `tid` (tid < RB), requested now so that their latency hides behind the row itself
        double e0 = 0.0, e1 = 0.0, e2 = 0.0;
        for (int64_t base = tid; base < n4; base += (int64_t)PL_T * PP) {
            float4 v[RB][PP];
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int j = 0; j < PP; ++j) {
                    const int64_t c = base + PL_T * j;
                    v[r][j] = c < n4 ? row[r][c] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            if (base == tid) {
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const int64_t s = srow[r];
                    sp[r] = s == special;
                    if (kind == 0) { ck[r] = -p.b[s]; cq[r] = -p.u2[s]; }
                    else { ck[r] = p.u[s]; cq[r] = -p.d[s]; }
                    if (sp[r]) { ck[r] = kind == 0 ? 0.f : 1.f; cq[r] = kind == 0 ? 1.f : -sc.dr; }
                }
                if (tid < RB && rows0 + tid < nrows) {
                    const int64_t s = rows0 + tid;
                    if (kind == 0) { e0 = p.Hd[s * p.ldh + s]; e1 = (double)p.b[s]; e2 = (double)p.u2[s]; }
                    else { e0 = p.c[s]; e1 = (double)p.Hp[(p.nI + s) * p.ldp + p.nI + s]; }
                }
            }
#pragma unroll
            for (int j = 0; j < PP; ++j) {
                const int64_t c = base + PL_T * j;
                if (c < n4) {
                    const float4 kk = __ldg(K4 + c), qq = __ldg(Q4 + c);
#pragma unroll
                    for (int r = 0; r < RB; ++r) {
                        if (sp[r]) v[r][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        fma4(v[r][j], ck[r], kk);
                        fma4(v[r][j], cq[r], qq);
                        if (rows0 + r < nrows) row[r][c] = v[r][j];
                        nrm[r] += dot4(v[r][j], v[r][j]);
                    }
                }
            }
        }
        block_sums<RB>(nrm, red);
        if (tid < RB && rows0 + tid < nrows) {
            const int64_t s = rows0 + tid;
            float nr = nrm[0];
#pragma unroll
            for (int r = 1; r < RB; ++r) nr = tid == r ? nrm[r] : nr;
            double score; bool have;
            if (kind == 0) {
                p.vnorm[s] = nr;
                const double hd = s == special ? sc.c1inv_d : e0 - e1 * e1 * sc.Cinv_d + e2 * e2 * sc.c1inv_d;
                score = hd > 0.0 ? (double)nr / hd : INFINITY;
                p.D[s] = score;
                have = isfinite(score);
            } else {
                p.rnorm[s] = nr;
                double cc, hd;
                if (s == special) { cc = sc.Cinv_d - (double)sc.dr * (double)sc.dr * sc.c1inv_d; hd = sc.hdiag; }
                else { const double uu = p.u[s], dd = p.d[s]; cc = e0 + uu * uu * sc.Cinv_d - dd * dd * sc.c1inv_d; hd = e1; }
                p.c[s] = cc;
                score = cc > kAddPivotTol * hd ? (double)nr / cc : -INFINITY;
                p.A[s] = score;
                have = isfinite(score);
                score = -score;                       // candidates are kept as minima
            }
            if (have) {
                const int id = p.perm[kind == 0 ? s : p.k + s];
                LoopCand& b = s_best[tid];
                if (b.idx < 0 || cand_less(score, id, b.val, b.id)) { b.val = score; b.id = id; b.idx = (int)s; }
            }
        }
    }
}

// P1, second half: u_l = Hp[l, 0:n_I] . b, d_l = Hp[l, q] - Hp[l, 0:n_I] . u2 for the pruned rows (items 0 .. n_J - 1) and
// the leaving row (item n_J), RB rows per pass.
template <int RB>
__device__ __noinline__ void pl_hpass(const Ptrs& p, const StepScal& sc, unsigned nblocks, float* red)
{
    constexpr int PP = PlPieces<RB>::value;
    const float4* bv = reinterpret_cast<const float4*>(p.b);
    const float4* uv = reinterpret_cast<const float4*>(p.u2);
    const int64_t n4 = p.ldh / 4;
    const int64_t nitems = p.nJ + 1;
    const int64_t qcol = p.nI + sc.t;
    const int tid = threadIdx.x;
    // start in the middle of the grid so that the blocks that got one V row more get one H row less
    for (int64_t l0 = (int64_t)((blockIdx.x + nblocks / 2) % nblocks) * RB; l0 < nitems; l0 += (int64_t)nblocks * RB) {
        const float4* row[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            const int64_t l = l0 + r < nitems ? l0 + r : nitems - 1;
            row[r] = reinterpret_cast<const float4*>(p.Hp + (l < p.nJ ? p.nI + l : sc.r0) * p.ldp);
        }
        float acc[2 * RB];
#pragma unroll
        for (int r = 0; r < 2 * RB; ++r) acc[r] = 0.f;
        for (int64_t base = tid; base < n4; base += (int64_t)PL_T * PP) {
            float4 x[RB][PP];
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int j = 0; j < PP; ++j) {
                    const int64_t c = base + PL_T * j;
                    x[r][j] = c < n4 ? row[r][c] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int j = 0; j < PP; ++j) {
                const int64_t c = base + PL_T * j;
                if (c < n4) {
                    const float4 bb = __ldg(bv + c), uu = __ldg(uv + c);
#pragma unroll
                    for (int r = 0; r < RB; ++r) { acc[r] += dot4(x[r][j], bb); acc[RB + r] += dot4(x[r][j], uu); }
                }
            }
        }
        block_sums<2 * RB>(acc, red);
        if (tid < RB && l0 + tid < nitems) {
            float su = acc[0], sd = acc[RB];
#pragma unroll
            for (int r = 1; r < RB; ++r) { su = tid == r ? acc[r] : su; sd = tid == r ? acc[RB + r] : sd; }
            const int64_t l = l0 + tid;
            const float* rowf = p.Hp + (l < p.nJ ? p.nI + l : sc.r0) * p.ldp;
            p.u[l] = su;
            p.d[l] = rowf[qcol] - sd;
        }
    }
}

// P3: rows of the inverse, kept in fp64 (row and column r0 replaced), and y_next = Hinv' h; RB rows per pass.
// The inverse is the one piece of the state that fp32 cannot carry: y = Hinv h cancels the common component of the
// rows of H to a few parts in 10^4, so an entry rounded to 2^-24 shows up in y, then in u2, and from there in every
// matrix (measured: the scores drift 3e-7 per swap with an fp32 inverse, 5e-9 with this one).  A piece is a double2.
template <int RB>
__device__ __noinline__ void pl_update_hinv(const Ptrs& p, const StepScal& sc, int64_t t_next, unsigned nblocks, float* red)
{
    constexpr int PP = PlPieces<RB>::value;
    const float2* b2 = reinterpret_cast<const float2*>(p.b);
    const float2* u2v = reinterpret_cast<const float2*>(p.u2);
    const float2* h2 = reinterpret_cast<const float2*>(p.Hp + (p.nI + t_next) * p.ldp);
    const int64_t n2 = p.ldh / 2;
    const int tid = threadIdx.x;
    for (int64_t s0 = (int64_t)blockIdx.x * RB; s0 < p.nI; s0 += (int64_t)nblocks * RB) {
        double2* row[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) row[r] = reinterpret_cast<double2*>(p.Hd + (s0 + r < p.nI ? s0 + r : p.nI - 1) * p.ldh);
        bool srow[RB];
        double nb[RB], us[RB], corner[RB], yacc[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) { yacc[r] = 0.0; srow[r] = false; nb[r] = 0.0; us[r] = 0.0; corner[r] = 0.0; }
        for (int64_t base = tid; base < n2; base += (int64_t)PL_T * PP) {
            double2 h[RB][PP];
#pragma unroll
            for (int r = 0; r < RB; ++r)
#pragma unroll
                for (int j = 0; j < PP; ++j) {
                    const int64_t c = base + PL_T * j;
                    h[r][j] = c < n2 ? row[r][c] : make_double2(0.0, 0.0);
                }
            if (base == tid) {
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const int64_t s = s0 + r < p.nI ? s0 + r : p.nI - 1;
                    srow[r] = s == sc.r0;
                    // row r0 becomes -u2 / c1: 0 * old - 0 * b + (-1 / c1) * u2
                    nb[r] = srow[r] ? 0.0 : -(double)p.b[s] * sc.Cinv_d;
                    us[r] = srow[r] ? -sc.c1inv_d : (double)p.u2[s] * sc.c1inv_d;
                    corner[r] = srow[r] ? sc.c1inv_d : -us[r];       // value of column r0 in this row
                }
            }
#pragma unroll
            for (int j = 0; j < PP; ++j) {
                const int64_t c = base + PL_T * j;
                if (c < n2) {
                    const float2 bb = __ldg(b2 + c), uu = __ldg(u2v + c), hh = __ldg(h2 + c);
                    const int64_t rc = sc.r0 - c * 2;                // position of column r0 inside this piece, if any
#pragma unroll
                    for (int r = 0; r < RB; ++r) {
                        double2 v = srow[r] ? make_double2(0.0, 0.0) : h[r][j];
                        v.x = fma(us[r], (double)uu.x, fma(nb[r], (double)bb.x, v.x));
                        v.y = fma(us[r], (double)uu.y, fma(nb[r], (double)bb.y, v.y));
                        v.x = rc == 0 ? corner[r] : v.x;
                        v.y = rc == 1 ? corner[r] : v.y;
                        if (s0 + r < p.nI) row[r][c] = v;
                        yacc[r] = fma(v.x, (double)hh.x, fma(v.y, (double)hh.y, yacc[r]));
                    }
                }
            }
        }
        block_sums_d<RB>(yacc, reinterpret_cast<double*>(red));
        if (tid < RB && s0 + tid < p.nI) {
            double t = yacc[0];
#pragma unroll
            for (int r = 1; r < RB; ++r) t = tid == r ? yacc[r] : t;
            p.y[s0 + tid] = (float)t;
        }
    }
}

// rows per pass for rows of n4 float4: as many as keep about PL_P loads per thread in flight
__host__ __device__ inline int pl_rows_per_pass(int64_t n4) { return n4 * 4 <= (int64_t)PL_T * PL_P ? 4 : (n4 * 2 <= (int64_t)PL_T * PL_P ? 2 : 1); }
constexpr int PL_MAX_BLOCKS = kLoopMaxBlocks;

__device__ __forceinline__ void merge_best(LoopCand* s_best, LoopCand* out)
{
    LoopCand b = s_best[0];
#pragma unroll
    for (int r = 1; r < 4; ++r) {
        const LoopCand c = s_best[r];
        if (c.idx >= 0 && (b.idx < 0 || cand_less(c.val, c.id, b.val, b.id))) b = c;
    }
    *out = b;
}

__global__ void __launch_bounds__(PL_T, 3) k_swap_loop_g1(LoopArgs a)
{
    // the phase routines are separate functions (their streaming loops get registers of their own); they read the
    // pointers and sizes from this shared copy
    __shared__ Ptrs s_p;
    if (threadIdx.x == 0) s_p = a.p;
    __syncthreads();
    const Ptrs& p = s_p;
    SearchCtl* ctl = a.p.ctl;
    __shared__ __align__(16) float red[8 * 8];
    __shared__ LoopCand s_best[4];
    __shared__ StepScal s_sc;
    __shared__ int s_flag, s_stop, s_idx;
    __shared__ double s_val;
    const int tid = threadIdx.x;
    const unsigned nblocks = gridDim.x;
    if (ctl->done) return;                              // uniform: nothing writes `done` before every block has read it
    const long long limit = ctl->wait_limit;
    unsigned long long epoch = 0;
    double obj = ctl->obj;
    int n_swaps = ctl->n_swaps;
    const int rbm = pl_rows_per_pass(p.ldm / 4), rbh = pl_rows_per_pass(p.ldh / 4), rbd = pl_rows_per_pass(p.ldh / 2);

    // candidates from the score vectors that the host-side bootstrap left (D, A of the current state)
    if (tid < 4) s_best[tid].idx = -1;
    __syncthreads();
    if (tid == 0) {
        LoopCand bd; bd.idx = -1; bd.val = 0.0; bd.id = 0;
        for (int64_t s = blockIdx.x; s < p.nI; s += nblocks) {
            const double v = p.D[s]; const int id = p.perm[s];
            if (isfinite(v) && (bd.idx < 0 || cand_less(v, id, bd.val, bd.id))) { bd.val = v; bd.id = id; bd.idx = (int)s; }
        }
        a.candD[blockIdx.x] = bd;
        LoopCand ba; ba.idx = -1; ba.val = 0.0; ba.id = 0;
        for (int64_t s = blockIdx.x; s < p.nJ; s += nblocks) {
            const double v = -p.A[s]; const int id = p.perm[p.k + s];
            if (isfinite(v) && (ba.idx < 0 || cand_less(v, id, ba.val, ba.id))) { ba.val = v; ba.id = id; ba.idx = (int)s; }
        }
        a.candA[blockIdx.x] = ba;
    }
    if (!grid_barrier(ctl, epoch, nblocks, limit, &s_flag)) return;
    int64_t t_cur;
    {
        if (tid < 32) {
            double v; int idx;
            reduce_cands(a.candA, nblocks, false, &v, &idx);
            if (tid == 0) s_idx = idx;
        }
        __syncthreads();
        t_cur = s_idx;
        __syncthreads();
    }
    if (t_cur < 0) {                                    // no eligible group to add
        if (blockIdx.x == 0 && tid == 0) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
        return;
    }
    unsigned long long tp = 0;
    const bool timer = blockIdx.x == 0 && tid == 0;
    if (timer) tp = global_timer_ns();
#define PL_LAP(phase) do { if (timer) { const unsigned long long now_ = global_timer_ns(); a.prof[phase] += now_ - tp; tp = now_; } } while (0)

    for (int step = 0; step < a.max_steps && n_swaps < a.max_swaps; ++step) {
        // ---------------------------------------------------------------- P0
        if (tid < 32) {
            double v; int idx;
            reduce_cands(a.candD, nblocks, false, &v, &idx);
            if (tid == 0) { s_idx = idx; s_val = v; }
        }
        __syncthreads();
        const int slot = s_idx;
        if (slot < 0) {
            if (blockIdx.x == 0 && tid == 0) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
            return;
        }
        const int64_t r0 = slot, t = t_cur;
        {
            const float4* vr = reinterpret_cast<const float4*>(p.V + r0 * p.ldm);
            const float4* rq = reinterpret_cast<const float4*>(p.R + t * p.ldm);
            float gx[1] = {0.f};
            for (int64_t c = tid; c < p.ldm / 4; c += PL_T) gx[0] += dot4(vr[c], rq[c]);
            block_sums<1>(gx, red);
            if (tid == 0) {
                const double GX = (double)gx[0];
                const double C = p.Hd[r0 * p.ldh + r0], P = p.y[r0], cq = p.c[t];
                const double GV = p.vnorm[r0], GR = p.rnorm[t];
                const double Cinv = 1.0 / C;
                const double Ds = GV * Cinv;
                const double RR1 = GR + 2.0 * P * Cinv * GX + P * P * Cinv * Cinv * GV;
                const double c1 = cq + P * P * Cinv;
                const double c1inv = 1.0 / c1;
                const double delta = Ds - c1inv * RR1;
                int stop = 0, reason = 0;
                if (!(C > 0.0) || !(c1 > 0.0) || !isfinite(delta)) { stop = 1; reason = OSSCAR_STOP_GUARD; }
                else if (a.accept_mode == OSSCAR_ACCEPT_IMPROVING && !(delta <= -a.tol * obj)) { stop = 1; reason = OSSCAR_STOP_NO_IMPROVEMENT; }
                s_stop = stop;
                s_val = delta;
                s_sc.r0 = r0; s_sc.t = t;
                s_sc.Cinv_d = Cinv; s_sc.c1inv_d = c1inv;
                s_sc.Cinv = (float)Cinv; s_sc.c1inv = (float)c1inv;
                s_sc.Q1 = (float)(Cinv * P); s_sc.M2 = (float)(c1inv * P * Cinv);
                s_sc.hdiag = p.Hp[r0 * p.ldp + r0];
                s_sc.dr = 0.f;
                if (blockIdx.x == 0) {
                    ctl->delta = delta; ctl->sel_D = Ds; ctl->sel_slot = slot; ctl->sel_t = (int)t;
                    if (stop) { ctl->done = 1; ctl->stop_reason = reason; *p.done_host = 1; }
                    else {
                        a.swap_trace[2 * n_swaps] = p.perm[slot];
                        a.swap_trace[2 * n_swaps + 1] = p.perm[p.k + t];
                        a.obj_trace[n_swaps + 1] = obj + delta;
                        ctl->obj = obj + delta;
                        ctl->n_swaps = n_swaps + 1;
                        p.small[S_CINV] = Cinv; p.small[S_C1INV] = c1inv;
                        // the two groups trade slots now: the ids that P1 and P2 attach to the scores of rows r0 and t are
                        // then those of the new occupants (no block reads the permutation during P0)
                        const int tt = p.k + (int)t;
                        const int gi = p.perm[slot], gj = p.perm[tt];
                        p.perm[slot] = gj; p.perm[tt] = gi;
                        p.slotof[gj] = slot; p.slotof[gi] = tt;
                    }
                }
            }
            __syncthreads();
        }
        if (s_stop) return;
        obj += s_val;
        ++n_swaps;
        StepScal sc = s_sc;
        {   // staged vectors, a slice per block
            const int64_t gidx = (int64_t)blockIdx.x * PL_T + tid, gstride = (int64_t)nblocks * PL_T;
            const double2* hrow2 = reinterpret_cast<const double2*>(p.Hd + r0 * p.ldh);
            const float4* y4 = reinterpret_cast<const float4*>(p.y);
            float4* b4 = reinterpret_cast<float4*>(p.b);
            float4* u4 = reinterpret_cast<float4*>(p.u2);
            for (int64_t c = gidx; c < p.ldh / 4; c += gstride) {
                const double2 h0 = hrow2[2 * c], h1 = hrow2[2 * c + 1];
                const float4 bs = make_float4((float)h0.x, (float)h0.y, (float)h1.x, (float)h1.y), yy = y4[c];
                float4 uu = make_float4(fmaf(-bs.x, sc.Q1, yy.x), fmaf(-bs.y, sc.Q1, yy.y), fmaf(-bs.z, sc.Q1, yy.z), fmaf(-bs.w, sc.Q1, yy.w));
                const int64_t rc = r0 - c * 4;
                uu.x = rc == 0 ? 0.f : uu.x; uu.y = rc == 1 ? 0.f : uu.y; uu.z = rc == 2 ? 0.f : uu.z; uu.w = rc == 3 ? 0.f : uu.w;
                b4[c] = bs;
                u4[c] = uu;
            }
            const float4* v4 = reinterpret_cast<const float4*>(p.V + r0 * p.ldm);
            const float4* r4 = reinterpret_cast<const float4*>(p.R + t * p.ldm);
            float4* k4 = reinterpret_cast<float4*>(p.K);
            float4* q4 = reinterpret_cast<float4*>(p.Vq);
            for (int64_t c = gidx; c < p.ldm / 4; c += gstride) {
                const float4 v = v4[c], r = r4[c];
                k4[c] = make_float4(sc.Cinv * v.x, sc.Cinv * v.y, sc.Cinv * v.z, sc.Cinv * v.w);
                q4[c] = make_float4(fmaf(sc.c1inv, r.x, sc.M2 * v.x), fmaf(sc.c1inv, r.y, sc.M2 * v.y),
                                    fmaf(sc.c1inv, r.z, sc.M2 * v.z), fmaf(sc.c1inv, r.w, sc.M2 * v.w));
            }
        }
        if (tid < 4) s_best[tid].idx = -1;
        PL_LAP(0);
        if (!grid_barrier(ctl, epoch, nblocks, limit, &s_flag)) return;

        // ---------------------------------------------------------------- P1
        if (rbm == 4) pl_update_rows<4>(p, 0, sc, nblocks, red, s_best);
        else if (rbm == 2) pl_update_rows<2>(p, 0, sc, nblocks, red, s_best);
        else pl_update_rows<1>(p, 0, sc, nblocks, red, s_best);
        if (rbh == 4) pl_hpass<4>(p, sc, nblocks, red);
        else if (rbh == 2) pl_hpass<2>(p, sc, nblocks, red);
        else pl_hpass<1>(p, sc, nblocks, red);
        __syncthreads();
        if (tid == 0) merge_best(s_best, &a.candD[blockIdx.x]);
        __syncthreads();
        if (tid < 4) s_best[tid].idx = -1;
        PL_LAP(1);
        if (!grid_barrier(ctl, epoch, nblocks, limit, &s_flag)) return;

        // ---------------------------------------------------------------- P2
        sc.dr = p.d[p.nJ];
        {   // exchange of the two slots in Hp: the strided column part first, its latency hides behind the row updates
            hswap_g1_at(p, sc.r0, p.nI + sc.t, (int64_t)blockIdx.x * PL_T + tid, (int64_t)nblocks * PL_T);
        }
        if (rbm == 4) pl_update_rows<4>(p, 1, sc, nblocks, red, s_best);
        else if (rbm == 2) pl_update_rows<2>(p, 1, sc, nblocks, red, s_best);
        else pl_update_rows<1>(p, 1, sc, nblocks, red, s_best);
        __syncthreads();
        if (tid == 0) merge_best(s_best, &a.candA[blockIdx.x]);
        PL_LAP(2);
        if (!grid_barrier(ctl, epoch, nblocks, limit, &s_flag)) return;

        // ---------------------------------------------------------------- P3
        if (tid < 32) {
            double v; int idx;
            reduce_cands(a.candA, nblocks, false, &v, &idx);
            if (tid == 0) s_idx = idx;
        }
        __syncthreads();
        const int64_t t_next = s_idx >= 0 ? s_idx : 0;
        const bool no_add = s_idx < 0;
        if (rbd == 4) pl_update_hinv<4>(p, sc, t_next, nblocks, red);
        else if (rbd == 2) pl_update_hinv<2>(p, sc, t_next, nblocks, red);
        else pl_update_hinv<1>(p, sc, t_next, nblocks, red);
        t_cur = t_next;
        if (timer) a.prof[4] += 1;
        PL_LAP(3);
        if (no_add) {                                   // the state is complete; nothing can enter at the next step
            if (blockIdx.x == 0 && tid == 0) { ctl->sel_t = -1; ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
            return;
        }
        if (!grid_barrier(ctl, epoch, nblocks, limit, &s_flag)) return;
    }
    if (blockIdx.x == 0 && tid == 0) ctl->sel_t = (int)t_cur;
#undef PL_LAP
}
