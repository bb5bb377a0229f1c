// Device-resident swap search: scoring (Eq. impact), selection, exact swap change and the
// rank-2g update of (H_II)^-1, V, R and the Schur complements (Proposition 1, Cases 1-3),
// on a slot-permuted layout in which kept rows occupy slots [0, n_I) and pruned rows the rest.
//
// Notation inside one step.  r = rows of the leaving slot, q = rows of the entering pruned slot,
//   C = Hinv[r,r], b = Hinv[:,r], h = Hp[q, 0:n_I]^T, y = Hinv h, P = y[r,:]^T (= H_qI Hinv_Ir),
//   K = C^-1 V_r, R1 = R_q + P K, c1 = c_q + P C^-1 P^T, Vq = c1^-1 R1 (new rows of V),
//   u2 = y - b C^-1 y_r on kept rows (0 on r), u = Hp[:,I] b, d = Hp[:,q] - Hp[:,I] u2.
//   Hinv' = Hinv - b C^-1 b^T + u2 c1^-1 u2^T (rows/cols r: -u2 c1^-1, block rr: c1^-1)
//   V'    = V - b K - u2 Vq (rows r: Vq)        R' = R + u K - d Vq        obj' = obj + delta
//   c_l'  = c_l + u_l C^-1 u_l^T - d_l c1^-1 d_l^T,   delta = Tr(C^-1 V_r V_r^T) - Tr(c1^-1 R1 R1^T).
#include "osscar_internal.cuh"
#include <math.h>
#include <float.h>
#include <limits.h>
#include "small_mat.cuh"

namespace osscar {
namespace {

using namespace smallmat;

constexpr double kAddPivotTol = 1e-6;   // pruned group ineligible if min pivot of c <= tol * max diag(H_qq)

__device__ float block_sum_f(float v, float* red) {      // result in every thread
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float s = 0.f;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i];
    return s;
}

__device__ __forceinline__ float dot4f(const float4& a, const float4& b) {
    return a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
}

struct Ptrs {
    float *Hp, *Hinv, *V, *R, *y, *b, *u2, *bC, *u2c, *u, *d, *K, *Vq, *vnorm, *rnorm;
    double *D, *A, *c, *small, *gramV, *gramR;
    double *shard;                                           // column shards: partial sums handed to the reduce hook
    double *Hd;                                              // fp64 copy of the inverse (single-row groups, independent scores)
    double *pairCinv, *pairKK, *pairScratch, *pairDelta;     // PAIR_EXACT scoring
    int32_t *perm, *slotof;
    SearchCtl* ctl;
    int32_t* done_host;
    int64_t nI, nJ, ldp, ldh, ldm, m, ng;
    int g, k;
};
// layout of the `small` region (doubles, each g*g): indices of the matrices
enum { S_CINV = 0, S_C1INV, S_Q1, S_Q1C, S_M2, S_GV, S_GX, S_GR, S_C, S_P, S_T1, S_T2, S_T3, S_C1, S_L, S_LI };

// Programmatic dependent launch: the kernels of a swap step are launched so that the next one may start while the
// current one is still running.  A kernel of single-row groups first requests the rows it streams (written by kernels
// that finished long ago), the kernels of wider groups begin with the wait; a kernel waits here for the kernel before
// it to complete before it reads anything that kernel wrote (staged vectors, scalars, the control block), and only then
// lets its own successor start: a successor's early part can thus overlap only the late part of its immediate
// predecessor, and its blocks are already resident when the predecessor drains.  Without the launch attribute both
// instructions do nothing.  What the predecessor wrote is read with ordinary loads only: the read-only (non-coherent)
// path may still hold a line from the step before, since no kernel boundary separates the two any more.
__device__ __forceinline__ void pdl_wait_then_release() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------ row norms / group Grams
// norm[i] = ||M[i, 0:ld)||^2 (pads are zero); one block per row.
__global__ void k_row_norms(const float* __restrict__ M, int64_t ld, float* __restrict__ norm, const SearchCtl* ctl)
{
    if (ctl->done) return;
    __shared__ float red[32];
    const float4* row = reinterpret_cast<const float4*>(M + (int64_t)blockIdx.x * ld);
    float acc = 0.f;
    for (int64_t c = threadIdx.x; c < ld / 4; c += blockDim.x) {
        const float4 v = row[c];
        acc += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    acc = block_sum_f(acc, red);
    if (threadIdx.x == 0) norm[blockIdx.x] = acc;
}

// gram[grp][a][b] = M[grp*g+a,:] . M[grp*g+b,:] for the kept groups (rows of V -> gramV) and the pruned groups (rows of
// R -> gramR) in one launch.  Grid (ng, ceil(g / GG_AT)): blocks [0, k) take kept slots, the rest pruned slots; a block
// owns GG_AT rows a of its group, its warps loop over the rows b >= the first of them, and each streamed piece of row b
// meets the GG_AT rows a (cache resident) at once; the lower triangle is written as the mirror image.
constexpr int GG_AT = 4;
__global__ void __launch_bounds__(256) k_group_gram(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g;
    const bool kept = (int)blockIdx.x < p.k;
    const int64_t grp = kept ? blockIdx.x : blockIdx.x - p.k;
    const float* M = (kept ? p.V : p.R) + grp * g * p.ldm;
    double* gram = (kept ? p.gramV : p.gramR) + grp * g * g;
    const int64_t n4 = p.ldm / 4;
    const int a0 = blockIdx.y * GG_AT;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const float4* ra[GG_AT];
#pragma unroll
    for (int i = 0; i < GG_AT; ++i) ra[i] = reinterpret_cast<const float4*>(M + (int64_t)(a0 + i < g ? a0 + i : a0) * p.ldm);
    for (int b = a0 + w; b < g; b += nw) {
        const float4* rb = reinterpret_cast<const float4*>(M + (int64_t)b * p.ldm);
        float s[GG_AT];
#pragma unroll
        for (int i = 0; i < GG_AT; ++i) s[i] = 0.f;
        for (int64_t c = lane; c < n4; c += 32) {
            const float4 z = rb[c];
#pragma unroll
            for (int i = 0; i < GG_AT; ++i) s[i] += dot4f(ra[i][c], z);
        }
#pragma unroll
        for (int i = 0; i < GG_AT; ++i) {
            const float t = warp_sum(s[i]);
            const int a = a0 + i;
            if (lane == 0 && a <= b) { gram[a * g + b] = (double)t; gram[b * g + a] = (double)t; }
        }
    }
}

// Scores of groups of more than one row: score = Tr(M^-1 Gram); one block per group.
// Blocks [0, k): kept slots (M = Hinv_rr, Gram of V rows) -> D; the rest: pruned slots (M = c, Gram of R rows) -> A.
__global__ void __launch_bounds__(1024) k_scores_general(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    extern __shared__ double smd[];
    const int g = p.g;
    double* M = smd; double* Lw = smd + g * g; double* Out = Lw + g * g;
    __shared__ double red[32];
    const int kind = (int)blockIdx.x < p.k ? 0 : 1;
    const int64_t grp = kind == 0 ? blockIdx.x : blockIdx.x - p.k;
    double scale = 0.0;
    for (int idx = threadIdx.x; idx < g * g; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        if (kind == 0) {
            M[idx] = 0.5 * ((double)p.Hinv[(grp * g + i) * p.ldh + grp * g + j] + (double)p.Hinv[(grp * g + j) * p.ldh + grp * g + i]);
        } else {
            M[idx] = 0.5 * (p.c[grp * g * g + idx] + p.c[grp * g * g + j * g + i]);
        }
    }
    if (kind == 1) {
        for (int i = 0; i < g; ++i) {
            const double hd = p.Hp[(p.nI + grp * g + i) * p.ldp + p.nI + grp * g + i];
            if (hd > scale) scale = hd;
        }
    }
    __syncthreads();
    const double piv = spd_inverse(M, Lw, Out, g);
    const double* gram = (kind == 0 ? p.gramV : p.gramR) + grp * g * g;
    const double tr = mat_trace_prod(Out, gram, g, red);
    if (threadIdx.x == 0) {
        if (kind == 0) p.D[grp] = (piv > 0.0) ? tr : INFINITY;
        else p.A[grp] = (piv > kAddPivotTol * scale) ? tr : -INFINITY;
    }
}

// ------------------------------------------------------------------ selection
// Cheapest drop (min D, ties -> smaller group id) and most valuable add (max A, ties -> smaller id).
__global__ void __launch_bounds__(1024) k_select(Ptrs p)
{
    pdl_wait_then_release();
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ double sv[32]; __shared__ int sid[32]; __shared__ int sidx[32];
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int npr = (int)(p.ng - p.k);
    for (int pass = 0; pass < 2; ++pass) {
        const int n = pass == 0 ? p.k : npr;
        double best = INFINITY; int bid = INT_MAX; int bidx = -1;
        for (int i = t; i < n; i += blockDim.x) {
            double v;
            if (pass == 0) {
                if (p.g == 1) {
                    const double hd = p.Hinv[(int64_t)i * p.ldh + i];
                    v = hd > 0.0 ? (double)p.vnorm[i] / hd : INFINITY;
                    p.D[i] = v;
                } else v = p.D[i];
            } else {
                if (p.g == 1) {
                    const double cc = p.c[i];
                    const double hd = p.Hp[(p.nI + i) * p.ldp + p.nI + i];
                    v = cc > kAddPivotTol * hd ? (double)p.rnorm[i] / cc : -INFINITY;
                    p.A[i] = v;
                } else v = p.A[i];
                v = -v;
            }
            const int id = p.perm[pass == 0 ? i : p.k + i];
            if (v < best || (v == best && id < bid)) { best = v; bid = id; bidx = i; }
        }
        for (int o = 16; o > 0; o >>= 1) {
            const double ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oid = __shfl_xor_sync(0xffffffffu, bid, o);
            const int oidx = __shfl_xor_sync(0xffffffffu, bidx, o);
            if (ov < best || (ov == best && oid < bid)) { best = ov; bid = oid; bidx = oidx; }
        }
        __syncthreads();
        if (lane == 0) { sv[w] = best; sid[w] = bid; sidx[w] = bidx; }
        __syncthreads();
        if (t == 0) {
            for (int i = 1; i < (int)(blockDim.x >> 5); ++i)
                if (sv[i] < best || (sv[i] == best && sid[i] < bid)) { best = sv[i]; bid = sid[i]; bidx = sidx[i]; }
            const bool ok = bidx >= 0 && isfinite(best);
            if (pass == 0) { ctl->sel_slot = bidx; ctl->sel_D = best; }
            else ctl->sel_t = bidx;
            if (!ok) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ y = Hinv h  (one warp per row, grid.y = e)
__global__ void __launch_bounds__(256) k_ypass(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int e = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int64_t s = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= p.nI) return;
    const float4* hrow = reinterpret_cast<const float4*>(p.Hp + (p.nI + (int64_t)p.ctl->sel_t * p.g + e) * p.ldp);
    const float4* arow = reinterpret_cast<const float4*>(p.Hinv + s * p.ldh);
    float a0 = 0.f, a1 = 0.f;
    const int64_t n4 = p.ldh / 4;
    int64_t c = lane;
    for (; c + 32 < n4; c += 64) {
        const float4 x0 = arow[c], x1 = arow[c + 32];
        const float4 h0 = *(hrow + c), h1 = *(hrow + c + 32);
        a0 += x0.x * h0.x + x0.y * h0.y + x0.z * h0.z + x0.w * h0.w;
        a1 += x1.x * h1.x + x1.y * h1.y + x1.z * h1.z + x1.w * h1.w;
    }
    for (; c < n4; c += 32) {
        const float4 x0 = arow[c]; const float4 h0 = *(hrow + c);
        a0 += x0.x * h0.x + x0.y * h0.y + x0.z * h0.z + x0.w * h0.w;
    }
    a0 = warp_sum(a0 + a1);
    if (lane == 0) p.y[(int64_t)e * p.ldh + s] = a0;
}

// Grams of the chosen rows: GV = V_r V_r^T, GX = V_r R_q^T, GR = R_q R_q^T; one warp per entry.
__global__ void __launch_bounds__(256) k_pairgram(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= 3LL * g * g) return;
    const int which = (int)(wid / (g * g)), a = (int)((wid / g) % g), b = (int)(wid % g);
    const int lane = threadIdx.x & 31;
    const float* Vr = p.V + (int64_t)p.ctl->sel_slot * g * p.ldm;
    const float* Rq = p.R + (int64_t)p.ctl->sel_t * g * p.ldm;
    const float4* x = reinterpret_cast<const float4*>((which == 2 ? Rq : Vr) + (int64_t)a * p.ldm);
    const float4* z = reinterpret_cast<const float4*>((which == 0 ? Vr : Rq) + (int64_t)b * p.ldm);
    float s = 0.f;
    for (int64_t c = lane; c < p.ldm / 4; c += 32) {
        const float4 xa = x[c], zb = z[c];
        s += xa.x * zb.x + xa.y * zb.y + xa.z * zb.z + xa.w * zb.w;
    }
    s = warp_sum(s);
    if (lane == 0) p.small[(S_GV + which) * g * g + a * g + b] = (double)s;
}

// One block: the g x g algebra of the step, the exact change of obj and the accept decision.
__global__ void __launch_bounds__(1024)
k_small(Ptrs p, int accept_mode, double accept_tol, int max_swaps, double* __restrict__ obj_trace, int32_t* __restrict__ swap_trace)
{
    pdl_wait_then_release();
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ double red[32];
    extern __shared__ double smd[];             // g^2 + 2 g doubles: the matrix being inverted and the pivot row/column
    const int g = p.g, gg = g * g;
    double* Ms = smd; double* Lws = smd + gg;
    double* S = p.small;
    double *Cinv = S + S_CINV * gg, *c1inv = S + S_C1INV * gg, *Q1 = S + S_Q1 * gg, *Q1c = S + S_Q1C * gg, *M2 = S + S_M2 * gg;
    double *GV = S + S_GV * gg, *GX = S + S_GX * gg, *GR = S + S_GR * gg, *P = S + S_P * gg;
    double *T1 = S + S_T1 * gg, *T2 = S + S_T2 * gg, *T3 = S + S_T3 * gg, *Lw = S + S_L * gg;
    const int64_t r0 = (int64_t)ctl->sel_slot * g;
    const int64_t tq = ctl->sel_t;
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        Ms[idx] = 0.5 * ((double)p.Hinv[(r0 + i) * p.ldh + r0 + j] + (double)p.Hinv[(r0 + j) * p.ldh + r0 + i]);
        P[idx] = (double)p.y[(int64_t)i * p.ldh + r0 + j];           // P[a][b] = y_a[r_b]
    }
    __syncthreads();
    const double pivC = spd_inverse(Ms, Lws, Cinv, g);
    const double Ds = mat_trace_prod(Cinv, GV, g, red);               // Tr(C^-1 V_r V_r^T)
    // R1 R1^T = GR + P (Cinv GX) + (P Cinv GX)^T + P Cinv GV Cinv P^T
    mat_mul(Cinv, false, GX, false, T1, g);                           // K R_q^T
    mat_mul(P, false, T1, false, T2, g);                              // P K R_q^T
    mat_mul(P, false, Cinv, false, T1, g);                            // P Cinv
    mat_mul(T1, false, GV, false, T3, g);                             // P Cinv GV
    mat_mul(T3, false, T1, true, Lw, g);                              // P Cinv GV Cinv P^T  (Lw reused as scratch)
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        T3[idx] = GR[idx] + T2[idx] + T2[j * g + i] + Lw[idx];
    }
    __syncthreads();
    mat_mul(T1, false, P, true, T2, g);                               // P Cinv P^T
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        const double cq = 0.5 * (p.c[tq * gg + idx] + p.c[tq * gg + j * g + i]);
        Ms[idx] = cq + 0.5 * (T2[idx] + T2[j * g + i]);
    }
    __syncthreads();
    const double pivc1 = spd_inverse(Ms, Lws, c1inv, g);
    const double gain = mat_trace_prod(c1inv, T3, g, red);
    const double delta = Ds - gain;
    mat_mul(Cinv, false, P, true, Q1, g);                             // Q1 = Cinv y_r = Cinv P^T
    mat_mul(Q1, false, c1inv, false, Q1c, g);                         // Q1 c1inv
    mat_mul(c1inv, false, T1, false, M2, g);                          // c1inv P Cinv
    if (threadIdx.x == 0) {
        const double obj = ctl->obj;
        bool stop = false; int reason = 0;
        if (!(pivC > 0.0) || !(pivc1 > 0.0) || !isfinite(delta)) { stop = true; reason = OSSCAR_STOP_GUARD; }
        else if (accept_mode == OSSCAR_ACCEPT_IMPROVING && !(delta <= -accept_tol * obj)) { stop = true; reason = OSSCAR_STOP_NO_IMPROVEMENT; }
        ctl->delta = delta;
        if (stop) { ctl->done = 1; ctl->stop_reason = reason; *p.done_host = 1; }
        else {
            const int n = ctl->n_swaps;
            swap_trace[2 * n] = p.perm[ctl->sel_slot];
            swap_trace[2 * n + 1] = p.perm[p.k + tq];
            obj_trace[n + 1] = obj + delta;
            ctl->obj = obj + delta;
            ctl->n_swaps = n + 1;
        }
    }
}

// Staged vectors of the step.  Part A (threads over kept rows s): b, bC = b C^-1, u2, u2c = u2 c1^-1.
// Part B (threads over columns): K = C^-1 V_r, Vq = c1^-1 R_q + (c1^-1 P C^-1) V_r.
__global__ void __launch_bounds__(256) k_prep(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g, gg = g * g;
    const double* S = p.small;
    const double *Cinv = S + S_CINV * gg, *c1inv = S + S_C1INV * gg, *Q1 = S + S_Q1 * gg, *Q1c = S + S_Q1C * gg, *M2 = S + S_M2 * gg;
    const int64_t r0 = (int64_t)p.ctl->sel_slot * g;
    const int64_t q0 = (int64_t)p.ctl->sel_t * g;
    const int64_t nA = p.nI * g, nB = p.ldm * g;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < nA + nB; idx += (int64_t)gridDim.x * blockDim.x) {
        if (idx < nA) {
            const int e = (int)(idx / p.nI); const int64_t s = idx % p.nI;
            double bc = 0.0, bq = 0.0, bqc = 0.0, yc = 0.0;
            for (int f = 0; f < g; ++f) {
                const double bf = (double)p.Hinv[(r0 + f) * p.ldh + s];
                bc += bf * Cinv[f * g + e];
                bq += bf * Q1[f * g + e];
                bqc += bf * Q1c[f * g + e];
                yc += (double)p.y[(int64_t)f * p.ldh + s] * c1inv[f * g + e];
            }
            const bool in_r = s >= r0 && s < r0 + g;
            p.b[(int64_t)e * p.ldh + s] = p.Hinv[(r0 + e) * p.ldh + s];
            p.bC[(int64_t)e * p.ldh + s] = (float)bc;
            p.u2[(int64_t)e * p.ldh + s] = in_r ? 0.f : (float)((double)p.y[(int64_t)e * p.ldh + s] - bq);
            p.u2c[(int64_t)e * p.ldh + s] = in_r ? 0.f : (float)(yc - bqc);
        } else {
            const int64_t j = idx - nA;
            const int e = (int)(j / p.ldm); const int64_t c = j % p.ldm;
            double kk = 0.0, vq = 0.0;
            for (int f = 0; f < g; ++f) {
                const double vr = (double)p.V[(r0 + f) * p.ldm + c];
                const double rq = (double)p.R[(q0 + f) * p.ldm + c];
                kk += Cinv[e * g + f] * vr;
                vq += c1inv[e * g + f] * rq + M2[e * g + f] * vr;
            }
            p.K[(int64_t)e * p.ldm + c] = (float)kk;
            p.Vq[(int64_t)e * p.ldm + c] = (float)vq;
        }
    }
}

// u_l = Hp[l, 0:n_I] b,  d_l = Hp[l, q] - Hp[l, 0:n_I] u2   for the pruned rows and the g leaving rows.
// One warp handles RPW consecutive rows for one e (grid.y = e).
template <int RPW>
__global__ void __launch_bounds__(256) k_hpass(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int e = blockIdx.y, g = p.g;
    const int lane = threadIdx.x & 31;
    const int64_t nrows = p.nJ + g;
    const int64_t l0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RPW;
    if (l0 >= nrows) return;
    const int64_t r0 = (int64_t)p.ctl->sel_slot * g;
    const int64_t qcol = p.nI + (int64_t)p.ctl->sel_t * g + e;
    const float4* rows[RPW];
#pragma unroll
    for (int i = 0; i < RPW; ++i) {
        int64_t l = l0 + i; if (l >= nrows) l = nrows - 1;
        const int64_t hrow = l < p.nJ ? p.nI + l : r0 + (l - p.nJ);
        rows[i] = reinterpret_cast<const float4*>(p.Hp + hrow * p.ldp);
    }
    const float4* bv = reinterpret_cast<const float4*>(p.b + (int64_t)e * p.ldh);
    const float4* uv = reinterpret_cast<const float4*>(p.u2 + (int64_t)e * p.ldh);
    float au[RPW], ad[RPW];
#pragma unroll
    for (int i = 0; i < RPW; ++i) { au[i] = 0.f; ad[i] = 0.f; }
    for (int64_t c = lane; c < p.ldh / 4; c += 32) {
        const float4 bb = *(bv + c), uu = *(uv + c);
#pragma unroll
        for (int i = 0; i < RPW; ++i) {
            const float4 x = rows[i][c];
            au[i] += x.x * bb.x + x.y * bb.y + x.z * bb.z + x.w * bb.w;
            ad[i] += x.x * uu.x + x.y * uu.y + x.z * uu.z + x.w * uu.w;
        }
    }
#pragma unroll
    for (int i = 0; i < RPW; ++i) {
        const float su = warp_sum(au[i]), sd = warp_sum(ad[i]);
        const int64_t l = l0 + i;
        if (lane == 0 && l < nrows) {
            p.u[l * g + e] = su;
            p.d[l * g + e] = reinterpret_cast<const float*>(rows[i])[qcol] - sd;
        }
    }
}

// Single-row groups outside the fused five-launch step (exhaustive pair scoring with g = 1):
// Hinv' = Hinv - bC b^T + u2c u2^T; row/column r takes -u2c, the corner 1/c1.
// Block: 256 threads x float4 = 1024 columns, RT rows.
constexpr int HI_RT = 8;
__global__ void __launch_bounds__(256) k_update_hinv(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int64_t c4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;     // float4 column index
    if (c4 * 4 >= p.ldh) return;
    const int64_t col = c4 * 4;
    const int64_t r0 = p.ctl->sel_slot;
    const int64_t row0 = (int64_t)blockIdx.y * HI_RT;
    const double* c1inv = p.small + S_C1INV;
    const float4 bb = reinterpret_cast<const float4*>(p.b)[c4];
    const float4 uu = reinterpret_cast<const float4*>(p.u2)[c4];
    const float4 uc = reinterpret_cast<const float4*>(p.u2c)[c4];
#pragma unroll
    for (int i = 0; i < HI_RT; ++i) {
        const int64_t s = row0 + i;
        if (s >= p.nI) break;
        float4* ptr = reinterpret_cast<float4*>(p.Hinv + s * p.ldh) + c4;
        float4 h = *ptr;
        if (s == r0) {
            h.x = -uc.x; h.y = -uc.y; h.z = -uc.z; h.w = -uc.w;
        } else {
            const float nb = -p.bC[s], us = p.u2c[s];
            h.x = fmaf(us, uu.x, fmaf(nb, bb.x, h.x));
            h.y = fmaf(us, uu.y, fmaf(nb, bb.y, h.y));
            h.z = fmaf(us, uu.z, fmaf(nb, bb.z, h.z));
            h.w = fmaf(us, uu.w, fmaf(nb, bb.w, h.w));
        }
        float* hf = reinterpret_cast<float*>(&h);
        if (r0 >= col && r0 < col + 4) hf[r0 - col] = (s == r0) ? (float)c1inv[0] : -p.u2c[s];
        *ptr = h;
    }
}

// Single-row groups outside the fused five-launch step: row updates of V (kind 0) and R (kind 1) with the squared
// row norm of the result (the next scores).
//   V'[s] = V[s] - b[s] K - u2[s] Vq   (row r: Vq)        R'[l] = R[l] + u[l] K - d[l] Vq   (row q: K - d[nJ] Vq)
// The R pass also moves c.  One block per UP_ROWS rows.
constexpr int UP_ROWS = 4;
__global__ void __launch_bounds__(256) k_update_rows(Ptrs p, int kind)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    __shared__ float red[32];
    float* M = kind == 0 ? p.V : p.R;
    const int64_t nrows = kind == 0 ? p.nI : p.nJ;
    const int64_t special0 = kind == 0 ? (int64_t)p.ctl->sel_slot : (int64_t)p.ctl->sel_t;
    const int64_t n4 = p.ldm / 4;
    const int64_t row0 = (int64_t)blockIdx.x * UP_ROWS;
    const float4* K4 = reinterpret_cast<const float4*>(p.K);
    const float4* Q4 = reinterpret_cast<const float4*>(p.Vq);
    for (int i = 0; i < UP_ROWS; ++i) {
        const int64_t s = row0 + i;
        if (s >= nrows) break;
        const bool special = s == special0;
        float ck, cq;
        if (special) { ck = kind == 0 ? 0.f : 1.f; cq = kind == 0 ? 1.f : -p.d[p.nJ]; }
        else { ck = kind == 0 ? -p.b[s] : p.u[s]; cq = kind == 0 ? -p.u2[s] : -p.d[s]; }
        float4* row = reinterpret_cast<float4*>(M + s * p.ldm);
        float nrm = 0.f;
        for (int64_t c = threadIdx.x; c < n4; c += blockDim.x) {
            float4 v = special ? make_float4(0.f, 0.f, 0.f, 0.f) : row[c];
            const float4 kk = K4[c], q = Q4[c];
            v.x = fmaf(cq, q.x, fmaf(ck, kk.x, v.x));
            v.y = fmaf(cq, q.y, fmaf(ck, kk.y, v.y));
            v.z = fmaf(cq, q.z, fmaf(ck, kk.z, v.z));
            v.w = fmaf(cq, q.w, fmaf(ck, kk.w, v.w));
            row[c] = v;
            nrm += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        nrm = block_sum_f(nrm, red);
        if (threadIdx.x == 0) {
            if (kind == 0) p.vnorm[s] = nrm;
            else {
                p.rnorm[s] = nrm;
                const double Cinv = p.small[S_CINV], c1inv = p.small[S_C1INV];
                if (special) { const double dd = p.d[p.nJ]; p.c[s] = Cinv - dd * dd * c1inv; }
                else { const double uu = p.u[s], dd = p.d[s]; p.c[s] += uu * uu * Cinv - dd * dd * c1inv; }
            }
        }
    }
}

// Groups of more than one row: y = Hinv h and the H pass as warp tiles of TP_R rows x TP_E right-hand sides, so that a
// streamed piece of a matrix row meets TP_E vectors and a piece of a vector TP_R rows (the per-(row, vector) kernels
// above re-read every row g times from L2).  Blocks of TP_W warps; grid (row tiles, ceil(g / TP_E)); TP_R is chosen per
// launch so that small layers still fill the machine.
constexpr int TP_E = 4, TP_W = 4;

// y[e][s] = Hinv[s, :] . Hp[q_e, 0:n_I]
template <int TP_R>
__global__ void __launch_bounds__(32 * TP_W) k_ypass_g(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g, e0 = blockIdx.y * TP_E;
    const int lane = threadIdx.x & 31;
    const int64_t s0 = ((int64_t)blockIdx.x * TP_W + (threadIdx.x >> 5)) * TP_R;
    if (s0 >= p.nI) return;
    const float4 *arow[TP_R], *hrow[TP_E];
#pragma unroll
    for (int i = 0; i < TP_R; ++i) arow[i] = reinterpret_cast<const float4*>(p.Hinv + (s0 + i < p.nI ? s0 + i : p.nI - 1) * p.ldh);
#pragma unroll
    for (int j = 0; j < TP_E; ++j)
        hrow[j] = reinterpret_cast<const float4*>(p.Hp + (p.nI + (int64_t)p.ctl->sel_t * g + (e0 + j < g ? e0 + j : g - 1)) * p.ldp);
    float acc[TP_R][TP_E];
#pragma unroll
    for (int i = 0; i < TP_R; ++i)
#pragma unroll
        for (int j = 0; j < TP_E; ++j) acc[i][j] = 0.f;
    for (int64_t c = lane; c < p.ldh / 4; c += 32) {
        float4 x[TP_R], h[TP_E];
#pragma unroll
        for (int i = 0; i < TP_R; ++i) x[i] = arow[i][c];
#pragma unroll
        for (int j = 0; j < TP_E; ++j) h[j] = *(hrow[j] + c);
#pragma unroll
        for (int i = 0; i < TP_R; ++i)
#pragma unroll
            for (int j = 0; j < TP_E; ++j) acc[i][j] += dot4f(x[i], h[j]);
    }
#pragma unroll
    for (int i = 0; i < TP_R; ++i)
#pragma unroll
        for (int j = 0; j < TP_E; ++j) {
            const float t = warp_sum(acc[i][j]);
            if (lane == 0 && s0 + i < p.nI && e0 + j < g) p.y[(int64_t)(e0 + j) * p.ldh + s0 + i] = t;
        }
}

// u_l = Hp[l, 0:n_I] b,  d_l = Hp[l, q] - Hp[l, 0:n_I] u2   for the pruned rows and the g leaving rows.
template <int TP_R>
__global__ void __launch_bounds__(32 * TP_W) k_hpass_g(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g, e0 = blockIdx.y * TP_E;
    const int lane = threadIdx.x & 31;
    const int64_t nrows = p.nJ + g;
    const int64_t l0 = ((int64_t)blockIdx.x * TP_W + (threadIdx.x >> 5)) * TP_R;
    if (l0 >= nrows) return;
    const int64_t r0 = (int64_t)p.ctl->sel_slot * g;
    const int64_t qcol0 = p.nI + (int64_t)p.ctl->sel_t * g;
    const float4 *rows[TP_R], *bv[TP_E], *uv[TP_E];
#pragma unroll
    for (int i = 0; i < TP_R; ++i) {
        const int64_t l = l0 + i < nrows ? l0 + i : nrows - 1;
        rows[i] = reinterpret_cast<const float4*>(p.Hp + (l < p.nJ ? p.nI + l : r0 + (l - p.nJ)) * p.ldp);
    }
#pragma unroll
    for (int j = 0; j < TP_E; ++j) {
        const int64_t e = e0 + j < g ? e0 + j : g - 1;
        bv[j] = reinterpret_cast<const float4*>(p.b + e * p.ldh);
        uv[j] = reinterpret_cast<const float4*>(p.u2 + e * p.ldh);
    }
    float au[TP_R][TP_E], ad[TP_R][TP_E];
#pragma unroll
    for (int i = 0; i < TP_R; ++i)
#pragma unroll
        for (int j = 0; j < TP_E; ++j) { au[i][j] = 0.f; ad[i][j] = 0.f; }
    for (int64_t c = lane; c < p.ldh / 4; c += 32) {
        float4 x[TP_R];
#pragma unroll
        for (int i = 0; i < TP_R; ++i) x[i] = rows[i][c];
#pragma unroll
        for (int j = 0; j < TP_E; ++j) {
            const float4 bb = *(bv[j] + c), uu = *(uv[j] + c);
#pragma unroll
            for (int i = 0; i < TP_R; ++i) { au[i][j] += dot4f(x[i], bb); ad[i][j] += dot4f(x[i], uu); }
        }
    }
#pragma unroll
    for (int i = 0; i < TP_R; ++i)
#pragma unroll
        for (int j = 0; j < TP_E; ++j) {
            const float su = warp_sum(au[i][j]), sd = warp_sum(ad[i][j]);
            const int64_t l = l0 + i;
            if (lane == 0 && l < nrows && e0 + j < g) {
                p.u[l * g + e0 + j] = su;
                p.d[l * g + e0 + j] = reinterpret_cast<const float*>(rows[i])[qcol0 + e0 + j] - sd;
            }
        }
}

// Groups of more than one row: the rank-2g updates as register tiles.  A block owns TG_RT rows x (TG_T float4) columns;
// the 2 g coefficients of its rows sit in shared memory, every streamed piece of the g-row panels (b, u2 / K, Vq) is
// used by all TG_RT rows, and the rows and columns that the formulas replace are patched before the store.
constexpr int TG_RT = 8;
constexpr int TG_T = 128;

// Hinv' = Hinv - bC b^T + u2c u2^T; rows/columns of r take -u2c, the rr block c1^-1.  Grid (column tiles, row tiles),
// dynamic shared memory 2 g TG_RT floats.
__device__ __forceinline__ void update_hinv_g_tile(const Ptrs& p, float* smf, unsigned bx, unsigned by)
{
    const int g = p.g;
    float* nbs = smf;                       // [e][i] = -bC[e][row0 + i]
    float* ucs = smf + g * TG_RT;           // [e][i] = u2c[e][row0 + i]
    const int64_t row0 = (int64_t)by * TG_RT;
    const int64_t r0 = (int64_t)p.ctl->sel_slot * g;
    for (int idx = threadIdx.x; idx < g * TG_RT; idx += TG_T) {
        const int e = idx / TG_RT; const int64_t s = row0 + idx % TG_RT;
        const bool ok = s < p.nI;
        nbs[idx] = ok ? -p.bC[(int64_t)e * p.ldh + s] : 0.f;
        ucs[idx] = ok ? p.u2c[(int64_t)e * p.ldh + s] : 0.f;
    }
    __syncthreads();
    const int64_t n4 = p.ldh / 4;
    const int64_t c4 = (int64_t)bx * TG_T + threadIdx.x;
    if (c4 >= n4) return;
    float4 h[TG_RT];
#pragma unroll
    for (int i = 0; i < TG_RT; ++i)
        h[i] = row0 + i < p.nI ? reinterpret_cast<const float4*>(p.Hinv + (row0 + i) * p.ldh)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
    const float4* b4 = reinterpret_cast<const float4*>(p.b) + c4;
    const float4* u4 = reinterpret_cast<const float4*>(p.u2) + c4;
    for (int e = 0; e < g; ++e) {
        const float4 bb = *(b4 + (int64_t)e * n4), uu = *(u4 + (int64_t)e * n4);
#pragma unroll
        for (int i = 0; i < TG_RT; ++i) {
            const float nb = nbs[e * TG_RT + i], us = ucs[e * TG_RT + i];
            h[i].x = fmaf(us, uu.x, fmaf(nb, bb.x, h[i].x)); h[i].y = fmaf(us, uu.y, fmaf(nb, bb.y, h[i].y));
            h[i].z = fmaf(us, uu.z, fmaf(nb, bb.z, h[i].z)); h[i].w = fmaf(us, uu.w, fmaf(nb, bb.w, h[i].w));
        }
    }
    const int64_t col = c4 * 4;
    const bool col_hit = col + 4 > r0 && col < r0 + g;
    const double* c1inv = p.small + S_C1INV * g * g;
#pragma unroll
    for (int i = 0; i < TG_RT; ++i) {
        const int64_t s = row0 + i;
        if (s >= p.nI) break;
        const bool srow = s >= r0 && s < r0 + g;
        if (srow || col_hit) {
            float* hf = reinterpret_cast<float*>(&h[i]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t sc = col + j;
                const bool scol = sc >= r0 && sc < r0 + g;
                if (srow && scol) hf[j] = (float)c1inv[(s - r0) * g + (sc - r0)];
                else if (srow) hf[j] = -p.u2c[(s - r0) * p.ldh + sc];
                else if (scol) hf[j] = -p.u2c[(sc - r0) * p.ldh + s];
            }
        }
        reinterpret_cast<float4*>(p.Hinv + s * p.ldh)[c4] = h[i];
    }
}

// V'[s] = V[s] - sum_e b[e][s] K[e] - sum_e u2[e][s] Vq[e] (rows of r: Vq) for kind 0,
// R'[l] = R[l] + sum_e u[l][e] K[e] - sum_e d[l][e] Vq[e] (rows of q: K[e] - sum_f d[nJ+e][f] Vq[f]) for kind 1.
// The replaced rows are the same sum started from zero with their own coefficients.
__device__ __forceinline__ void update_rows_g_tile(const Ptrs& p, float* smf, int kind, unsigned bx, unsigned by)
{
    const int g = p.g;
    float* cks = smf;                       // coefficient of K[e] for row i
    float* cqs = smf + g * TG_RT;           // coefficient of Vq[e]
    float* M = kind == 0 ? p.V : p.R;
    const int64_t nrows = kind == 0 ? p.nI : p.nJ;
    const int64_t special0 = (kind == 0 ? (int64_t)p.ctl->sel_slot : (int64_t)p.ctl->sel_t) * g;
    const int64_t row0 = (int64_t)by * TG_RT;
    for (int idx = threadIdx.x; idx < g * TG_RT; idx += TG_T) {
        const int e = idx / TG_RT; const int64_t s = row0 + idx % TG_RT;
        float ck = 0.f, cq = 0.f;
        if (s < nrows) {
            if (s >= special0 && s < special0 + g) {
                const int ee = (int)(s - special0);
                if (kind == 0) cq = e == ee ? 1.f : 0.f;
                else { ck = e == ee ? 1.f : 0.f; cq = -p.d[(p.nJ + ee) * g + e]; }
            } else if (kind == 0) { ck = -p.b[(int64_t)e * p.ldh + s]; cq = -p.u2[(int64_t)e * p.ldh + s]; }
            else { ck = p.u[s * g + e]; cq = -p.d[s * g + e]; }
        }
        cks[idx] = ck; cqs[idx] = cq;
    }
    __syncthreads();
    const int64_t n4 = p.ldm / 4;
    const int64_t c4 = (int64_t)bx * TG_T + threadIdx.x;
    if (c4 >= n4) return;
    float4 v[TG_RT];
#pragma unroll
    for (int i = 0; i < TG_RT; ++i) {
        const int64_t s = row0 + i;
        const bool keep = s < nrows && !(s >= special0 && s < special0 + g);
        v[i] = keep ? reinterpret_cast<const float4*>(M + s * p.ldm)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const float4* K4 = reinterpret_cast<const float4*>(p.K) + c4;
    const float4* Q4 = reinterpret_cast<const float4*>(p.Vq) + c4;
    for (int e = 0; e < g; ++e) {
        const float4 kk = *(K4 + (int64_t)e * n4), q = *(Q4 + (int64_t)e * n4);
#pragma unroll
        for (int i = 0; i < TG_RT; ++i) {
            const float ck = cks[e * TG_RT + i], cq = cqs[e * TG_RT + i];
            v[i].x = fmaf(cq, q.x, fmaf(ck, kk.x, v[i].x)); v[i].y = fmaf(cq, q.y, fmaf(ck, kk.y, v[i].y));
            v[i].z = fmaf(cq, q.z, fmaf(ck, kk.z, v[i].z)); v[i].w = fmaf(cq, q.w, fmaf(ck, kk.w, v[i].w));
        }
    }
#pragma unroll
    for (int i = 0; i < TG_RT; ++i)
        if (row0 + i < nrows) reinterpret_cast<float4*>(M + (row0 + i) * p.ldm)[c4] = v[i];
}

__global__ void __launch_bounds__(TG_T) k_update_hinv_g(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    extern __shared__ float smf[];
    update_hinv_g_tile(p, smf, blockIdx.x, blockIdx.y);
}

__global__ void __launch_bounds__(TG_T) k_update_rows_g(Ptrs p, int kind)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    extern __shared__ float smf[];
    update_rows_g_tile(p, smf, kind, blockIdx.x, blockIdx.y);
}

// The three updates of a step in one launch (they depend on the same staged vectors and on nothing of each other):
// blocks [0, nh) are the tiles of Hinv, the next nv those of V, the rest those of R; hx and mx are the column tiles of a
// row tile of Hinv and of V / R.
__global__ void __launch_bounds__(TG_T) k_update_all_g(Ptrs p, unsigned nh, unsigned nv, unsigned hx, unsigned mx)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    extern __shared__ float smf[];
    unsigned b = blockIdx.x;
    if (b < nh) { update_hinv_g_tile(p, smf, b % hx, b / hx); return; }
    b -= nh;
    if (b < nv) { update_rows_g_tile(p, smf, 0, b % mx, b / mx); return; }
    b -= nv;
    update_rows_g_tile(p, smf, 1, b % mx, b / mx);
}

// C += sign * A * B^T (all g x g, ld g) on the fp64 tensor-core path; each entry of C is owned by one lane.
__device__ void mat_mul_nt_acc(const double* A, const double* B, double* C, int g, double sign)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int nt = (g + 7) >> 3, r4 = lane >> 2, c4 = lane & 3;
    for (int tile = warp; tile < nt * nt; tile += nwarps) {
        const int i0 = (tile / nt) * 8, j0 = (tile % nt) * 8;
        const int ai = i0 + r4, bj = j0 + r4;
        double d0 = 0.0, d1 = 0.0;
        for (int k0 = 0; k0 < g; k0 += 4) {
            const int kk = k0 + c4;
            const double a = (kk < g && ai < g) ? A[ai * g + kk] : 0.0;
            const double b = (kk < g && bj < g) ? B[bj * g + kk] : 0.0;
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                         : "+d"(d0), "+d"(d1) : "d"(a), "d"(b));
        }
        const int ci = i0 + r4, cj = j0 + 2 * c4;
        if (ci < g) {
            if (cj < g) C[ci * g + cj] += sign * d0;
            if (cj + 1 < g) C[ci * g + cj + 1] += sign * d1;
        }
    }
    __syncthreads();
}

// c_l' = c_l + u_l C^-1 u_l^T - d_l c1^-1 d_l^T for every pruned slot (g > 1); the entering slot receives
// the leaving group: c' = C^-1 - d_r c1^-1 d_r^T.  One block per pruned slot; u_l (then d_l) and its product
// with C^-1 (c1^-1) sit in shared memory (2 g^2 doubles), the four g x g products run on the fp64 tensor-core path.
__global__ void __launch_bounds__(1024) k_update_c(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    extern __shared__ double smc[];
    const int g = p.g, gg = g * g;
    double* X = smc; double* T = smc + gg;
    const int64_t t = blockIdx.x;
    const bool special = t == p.ctl->sel_t;
    const double* Cinv = p.small + S_CINV * gg;
    const double* c1inv = p.small + S_C1INV * gg;
    const float* ul = p.u + (special ? p.nJ : t * g) * g;     // g x g, row a = row of the group
    const float* dl = p.d + (special ? p.nJ : t * g) * g;
    double* c = p.c + t * gg;
    if (special) {
        for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) c[idx] = Cinv[idx];
    } else {
        for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) X[idx] = (double)ul[idx];
        __syncthreads();
        mat_mul(X, false, Cinv, false, T, g);                 // u_l C^-1
        mat_mul_nt_acc(T, X, c, g, 1.0);
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) X[idx] = (double)dl[idx];
    __syncthreads();
    mat_mul(X, false, c1inv, false, T, g);                    // d_l c1^-1
    mat_mul_nt_acc(T, X, c, g, -1.0);
}

// Exchange the rows (phase 0) or columns (phase 1) of Hp that belong to the leaving and entering groups;
// phase 1 also exchanges the two groups in the slot permutation.
__global__ void __launch_bounds__(256) k_hswap(Ptrs p, int phase)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int g = p.g;
    const int64_t a0 = (int64_t)p.ctl->sel_slot * g, b0 = p.nI + (int64_t)p.ctl->sel_t * g;
    const int64_t n = p.ldp * g;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (int64_t)gridDim.x * blockDim.x) {
        const int e = (int)(idx / p.ldp); const int64_t x = idx % p.ldp;
        float *pa, *pb;
        if (phase == 0) { pa = p.Hp + (a0 + e) * p.ldp + x; pb = p.Hp + (b0 + e) * p.ldp + x; }
        else {
            if (x >= p.nI + p.nJ) continue;
            pa = p.Hp + x * p.ldp + a0 + e; pb = p.Hp + x * p.ldp + b0 + e;
        }
        const float va = *pa, vb = *pb;
        *pa = vb; *pb = va;
    }
    if (phase == 1 && blockIdx.x == 0 && threadIdx.x == 0) {
        const int s = p.ctl->sel_slot, t = p.k + p.ctl->sel_t;
        const int gi = p.perm[s], gj = p.perm[t];
        p.perm[s] = gj; p.perm[t] = gi;
        p.slotof[gj] = s; p.slotof[gi] = t;
    }
}

// ------------------------------------------------------------------ finalize
__global__ void k_scatter_rows(Ptrs p, float* __restrict__ W_out)
{
    const int64_t s = blockIdx.x;
    const int64_t row = (int64_t)p.perm[s / p.g] * p.g + s % p.g;
    for (int64_t c = threadIdx.x; c < p.m; c += blockDim.x) W_out[row * p.m + c] = p.V[s * p.ldm + c];
}
__global__ void k_sorted_support(Ptrs p, int32_t* __restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.k) return;
    const int id = p.perm[i];
    int rank = 0;
    for (int j = 0; j < p.k; ++j) rank += p.perm[j] < id;
    out[rank] = id;
}
__global__ void k_begin(SearchCtl* ctl, double* obj_trace, int32_t* done_host)
{
    ctl->done = 0; ctl->stop_reason = OSSCAR_STOP_MAX_SWAPS; ctl->n_swaps = 0; ctl->n_refresh = 0;
    obj_trace[0] = ctl->obj;
    ctl->acc[2] = ctl->obj;
    *done_host = 0;
}
__global__ void k_count_refresh(SearchCtl* ctl) { if (!ctl->done) ctl->n_refresh += 1; }
__global__ void k_search_wait_limit(SearchCtl* ctl, long long cycles) { ctl->wait_limit = cycles; }
__global__ void k_shard_scalar(SearchCtl* ctl, double* sh, int back) { if (back) ctl->acc[1] = sh[0]; else sh[0] = ctl->acc[1]; }
__global__ void k_final_obj(SearchCtl* ctl) { ctl->acc[3] = ctl->const_term - ctl->acc[1]; }

// ------------------------------------------------------------------ exhaustive pair scoring (PAIR_EXACT)
// For every kept slot s and pruned slot t the exact change of obj of swapping them (Case 3 = Case 1 then Case 2):
//   delta(s,t) = D_s - Tr(c1^-1 R1 R1^T),  P = Pm[t-rows, s-cols] with Pm = Hp[J,I] Hinv,  T1 = P C_s^-1,
//   c1 = c_t + T1 P^T,  R1 R1^T = GR_t + T1 GX + (T1 GX)^T + P (C_s^-1 GV_s C_s^-1) P^T,  GX = V_s R_t^T.
constexpr int kPairBlocks = 296;
constexpr int kPairTemps = 8;

// Per kept slot: C_s^-1, KK_s = C_s^-1 GV_s C_s^-1 and D_s (block per slot; dynamic smem 3 g^2 doubles).
__global__ void __launch_bounds__(1024) k_pair_slots(Ptrs p)
{
    if (p.ctl->done) return;
    extern __shared__ double smd[];
    __shared__ double red[32];
    const int g = p.g, gg = g * g;
    double* M = smd; double* Lw = smd + gg; double* T = Lw + gg;
    const int64_t s = blockIdx.x;
    double* Cinv = p.pairCinv + s * gg;
    double* KK = p.pairKK + s * gg;
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        M[idx] = 0.5 * ((double)p.Hinv[(s * g + i) * p.ldh + s * g + j] + (double)p.Hinv[(s * g + j) * p.ldh + s * g + i]);
    }
    __syncthreads();
    const double piv = spd_inverse(M, Lw, Cinv, g);
    const double* GV = p.gramV + s * gg;
    mat_mul(Cinv, false, GV, false, T, g);
    mat_mul(T, false, Cinv, false, KK, g);
    const double tr = mat_trace_prod(Cinv, GV, g, red);
    if (threadIdx.x == 0) p.D[s] = piv > 0.0 ? tr : INFINITY;
}

__global__ void __launch_bounds__(1024)
k_pair_delta(Ptrs p, const float* __restrict__ Pm, int64_t ldpm, const float* __restrict__ XG, int64_t ldxg, int64_t npairs)
{
    if (p.ctl->done) return;
    __shared__ double red[32];
    extern __shared__ double smd[];             // g^2 + 2 g doubles: c1 while it is inverted
    const int g = p.g, gg = g * g;
    double* Ms = smd; double* Lws = smd + gg;
    const int64_t npr = p.ng - p.k;
    double* S = p.pairScratch + (int64_t)blockIdx.x * kPairTemps * gg;
    double *P = S, *GX = S + gg, *T1 = S + 2 * gg, *RR = S + 4 * gg, *TMP = S + 5 * gg, *OUT = S + 7 * gg;
    for (int64_t pair = blockIdx.x; pair < npairs; pair += gridDim.x) {
        const int64_t s = pair / npr, t = pair % npr;
        const double Ds = p.D[s], At = p.A[t];
        if (!isfinite(Ds) || !isfinite(At)) {            // a side that cannot move
            if (threadIdx.x == 0) p.pairDelta[pair] = INFINITY;
            continue;
        }
        const double* Cinv = p.pairCinv + s * gg;
        const double* KK = p.pairKK + s * gg;
        for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
            const int a = idx / g, b = idx % g;
            P[idx] = (double)Pm[(t * g + a) * ldpm + s * g + b];
            GX[idx] = (double)XG[(s * g + a) * ldxg + t * g + b];
        }
        __syncthreads();
        mat_mul(P, false, Cinv, false, T1, g);                   // P C^-1
        mat_mul(T1, false, P, true, TMP, g);                     // P C^-1 P^T
        for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
            const int i = idx / g, j = idx % g;
            Ms[idx] = 0.5 * (p.c[t * gg + idx] + p.c[t * gg + j * g + i]) + 0.5 * (TMP[idx] + TMP[j * g + i]);
        }
        __syncthreads();
        mat_mul(T1, false, GX, false, TMP, g);                   // P C^-1 V_s R_t^T
        mat_mul(P, false, KK, false, OUT, g);                    // P KK
        mat_mul(OUT, false, P, true, RR, g);                     // P KK P^T
        for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
            const int i = idx / g, j = idx % g;
            RR[idx] += p.gramR[t * gg + idx] + TMP[idx] + TMP[j * g + i];
        }
        __syncthreads();
        const double piv = spd_inverse(Ms, Lws, OUT, g);
        const double gain = mat_trace_prod(OUT, RR, g, red);
        if (threadIdx.x == 0) p.pairDelta[pair] = piv > 0.0 ? Ds - gain : INFINITY;
        __syncthreads();
    }
}

// Best pair: smallest delta, ties to the smaller leaving id, then the smaller entering id.
__global__ void __launch_bounds__(1024) k_pair_select(Ptrs p, int64_t npairs)
{
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ double sv[32]; __shared__ int so[32], si[32]; __shared__ long long sx[32];
    const int64_t npr = p.ng - p.k;
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    double best = INFINITY; int bo = INT_MAX, bi = INT_MAX; long long bx = -1;
    auto better = [](double v, int o, int i, double bv, int bo2, int bi2) {
        return v < bv || (v == bv && (o < bo2 || (o == bo2 && i < bi2)));
    };
    for (int64_t pair = t; pair < npairs; pair += blockDim.x) {
        const double v = p.pairDelta[pair];
        const int o = p.perm[pair / npr], i = p.perm[p.k + pair % npr];
        if (better(v, o, i, best, bo, bi)) { best = v; bo = o; bi = i; bx = pair; }
    }
    for (int off = 16; off > 0; off >>= 1) {
        const double ov = __shfl_xor_sync(0xffffffffu, best, off);
        const int oo = __shfl_xor_sync(0xffffffffu, bo, off), oi = __shfl_xor_sync(0xffffffffu, bi, off);
        const long long ox = __shfl_xor_sync(0xffffffffu, bx, off);
        if (better(ov, oo, oi, best, bo, bi)) { best = ov; bo = oo; bi = oi; bx = ox; }
    }
    if (lane == 0) { sv[w] = best; so[w] = bo; si[w] = bi; sx[w] = bx; }
    __syncthreads();
    if (t == 0) {
        for (int j = 1; j < (int)(blockDim.x >> 5); ++j)
            if (better(sv[j], so[j], si[j], best, bo, bi)) { best = sv[j]; bo = so[j]; bi = si[j]; bx = sx[j]; }
        if (bx < 0 || !isfinite(best)) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
        else { ctl->sel_slot = (int)(bx / npr); ctl->sel_t = (int)(bx % npr); ctl->sel_D = p.D[bx / npr]; }
    }
}

// Launch, with `dependent` set, as a programmatic dependent of the kernel before it on the stream (see
// pdl_wait_then_release).  Only a launch that directly follows another kernel launch of the step may be one: behind an
// event record, a copy or a reduction by the caller's hook the launch is an ordinary, fully ordered one.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_smem(bool dependent, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = dependent ? 1 : 0;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(bool dependent, void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args)
{
    return launch_pdl_smem(dependent, kernel, grid, block, 0, st, args...);
}

#include "search_g1.cuh"

Ptrs make_ptrs(osscar_ctx* ctx)
{
    const Layout& L = ctx->L;
    char* ws = (char*)ctx->ws;
    Ptrs p;
    p.Hp = (float*)(ws + L.off_Hp); p.Hinv = (float*)(ws + L.off_Hinv); p.V = (float*)(ws + L.off_V);
    p.R = (float*)(ws + L.off_R);
    p.y = (float*)(ws + L.off_y); p.b = (float*)(ws + L.off_b); p.u2 = (float*)(ws + L.off_u2);
    p.bC = (float*)(ws + L.off_bC); p.u2c = (float*)(ws + L.off_u2c);
    p.u = (float*)(ws + L.off_u); p.d = (float*)(ws + L.off_d);
    p.K = (float*)(ws + L.off_K); p.Vq = (float*)(ws + L.off_Vq);
    p.vnorm = (float*)(ws + L.off_vnorm); p.rnorm = (float*)(ws + L.off_rnorm);
    p.D = (double*)(ws + L.off_D); p.A = (double*)(ws + L.off_A); p.c = (double*)(ws + L.off_c);
    p.small = (double*)(ws + L.off_small); p.gramV = (double*)(ws + L.off_gramV); p.gramR = (double*)(ws + L.off_gramR);
    p.Hd = (double*)(ws + L.off_Hd); p.shard = (double*)(ws + L.off_shard);
    p.perm = (int32_t*)(ws + L.off_perm); p.slotof = (int32_t*)(ws + L.off_slotof);
    p.pairCinv = (double*)(ws + L.off_pairCinv); p.pairKK = (double*)(ws + L.off_pairKK);
    p.pairScratch = (double*)(ws + L.off_pairScratch); p.pairDelta = (double*)(ws + L.off_pairDelta);
    p.ctl = ctx->ctl; p.done_host = ctx->done_flag_dev;
    p.nI = L.nI; p.nJ = L.nJ; p.ldp = L.ldp; p.ldh = L.ldh; p.ldm = L.ldm; p.m = L.m; p.ng = L.ng;
    p.g = L.g; p.k = L.k;
    return p;
}

// Threads of the one-block-per-matrix kernels of the g x g algebra: a thread per entry up to the block limit.
static unsigned small_threads(int g) { return g * g >= 1024 ? 1024u : 256u; }

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return OSSCAR_E_CUDA; } while (0)

// Everything the selection needs from a freshly built or freshly updated state.
cudaError_t enqueue_scores(osscar_ctx* ctx, const Ptrs& p, bool norms, bool general = false, bool chain = false, bool dependent = false)
{
    cudaStream_t st = ctx->stream;
    if (p.g == 1 && !general) {
        if (norms) {
            k_row_norms<<<(unsigned)p.nI, 256, 0, st>>>(p.V, p.ldm, p.vnorm, p.ctl);
            count_launches(p.nJ > 0 ? 2 : 1);
            if (p.nJ > 0) k_row_norms<<<(unsigned)p.nJ, 256, 0, st>>>(p.R, p.ldm, p.rnorm, p.ctl);
        }
    } else {
        const size_t smem = 3 * (size_t)p.g * p.g * sizeof(double);
        cudaError_t e = cudaFuncSetAttribute(k_scores_general, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        // kept and pruned groups together; inside a swap step (chain) the two are programmatic dependents
        launch_pdl(chain && dependent, k_group_gram, dim3((unsigned)p.ng, (unsigned)((p.g + GG_AT - 1) / GG_AT)), dim3(256), st, p);
        launch_pdl_smem(chain, k_scores_general, dim3((unsigned)p.ng), dim3(small_threads(p.g)), smem, st, p);
        count_launches(2);
    }
    return cudaGetLastError();
}

#include "search_block.cuh"
#include "search_loop_g1.cuh"

// Blocks of the persistent loop: every block the device can hold at once (cooperative launch), but no more than the
// longest phase has passes to hand out.  0 when the device cannot launch cooperatively.
int persistent_grid(const Layout& L)
{
    int dev = 0, coop = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_swap_loop_g1, PL_T, 0) != cudaSuccess || per_sm < 1) return 0;
    int64_t grid = (int64_t)sms * per_sm;
    const int rbm = pl_rows_per_pass(L.ldm / 4), rbh = pl_rows_per_pass(L.ldh / 4);
    int64_t passes = (L.nI + rbm - 1) / rbm;
    if ((L.nJ + rbm - 1) / rbm > passes) passes = (L.nJ + rbm - 1) / rbm;
    if ((L.nJ + rbh) / rbh > passes) passes = (L.nJ + rbh) / rbh;
    if (grid > passes) grid = passes;
    if (grid > PL_MAX_BLOCKS) grid = PL_MAX_BLOCKS;
    return (int)(grid < 1 ? 1 : grid);
}

}  // namespace

int build_hinv64(osscar_ctx* ctx, bool guarded)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    char* ws = (char*)ctx->ws;
    float* Hp = (float*)(ws + L.off_Hp);
    float* Hinv = (float*)(ws + L.off_Hinv);
    double* Hd = (double*)(ws + L.off_Hd);
    float* E = (float*)(ws + L.off_big);
    float* T = E + L.nI * L.ldh;
    const int32_t* done = guarded ? &ctx->ctl->done : nullptr;
    void* tc = ws + L.off_tc;
    // X0 = the fp32 inverse at hand (raw from the blocked inversion, or carried by an fp32 driver).  With E = I - H_II X0,
    // H_II^-1 = X0 (I + E + E^2 + ...): E is formed once with fp64 sums, the series is cut after E^2 (its products are
    // corrections of corrections: the tensor-core split product is ample), and the sum X0 + X0 (E + E^2) is taken in fp64.
    // The error left is E^3 (below 1e-9 for any start within 1e-3), against E^2 for a single Newton-Schulz step.
    if (gemm_f64acc(st, L.nI, L.nI, L.nI, -1.0, Hp, L.ldp, Hinv, L.ldh, 0.0, nullptr, 0, E, L.ldh, true, done) != cudaSuccess) return OSSCAR_E_CUDA;
    if (cudaMemcpyAsync(T, E, sizeof(float) * L.nI * L.ldh, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return OSSCAR_E_CUDA;
    if (gemm_tc(st, L.nI, L.nI, L.nI, 1.f, E, L.ldh, E, L.ldh, 1.f, T, L.ldh, tc, L.tc_bytes, ctx->ctl, done) != cudaSuccess) return OSSCAR_E_CUDA;
    if (gemm_tc(st, L.nI, L.nI, L.nI, 1.f, Hinv, L.ldh, T, L.ldh, 0.f, E, L.ldh, tc, L.tc_bytes, ctx->ctl, done) != cudaSuccess) return OSSCAR_E_CUDA;
    k_hinv_to_d<<<(unsigned)L.nI, 256, 0, st>>>(Hinv, E, Hd, L.ldh, L.nI, done);
    k_hinv_from_d<<<(unsigned)L.nI, 256, 0, st>>>(Hd, Hinv, L.ldh, done);
    count_launches(2);
    if (cudaGetLastError() != cudaSuccess) return OSSCAR_E_CUDA;
    ctx->hd_valid = true;
    return OSSCAR_OK;
}

int shard_reduce(osscar_ctx* ctx, void* buf, int64_t count, int dtype)
{
    if (!ctx->reduce) return OSSCAR_OK;
    if (cudaGetLastError() != cudaSuccess) return OSSCAR_E_CUDA;
    return ctx->reduce(ctx->reduce_user, buf, count, dtype, (void*)ctx->stream) == 0 ? OSSCAR_OK : OSSCAR_E_CUDA;
}

cudaError_t score_pass(osscar_ctx* ctx)
{
    Ptrs p = make_ptrs(ctx);
    cudaError_t e = enqueue_scores(ctx, p, true);
    if (e != cudaSuccess) return e;
    if (ctx->reduce && shard_reduce(ctx, p.vnorm, ctx->L.d1, OSSCAR_FP32) != OSSCAR_OK) return cudaErrorUnknown;   // row norms are sums over columns
    k_select<<<1, 1024, 0, ctx->stream>>>(p);      // also leaves the score vectors D and A readable
    count_launches(1);
    return cudaGetLastError();
}

int run_search(osscar_ctx* ctx, const osscar_search_params* prm, int32_t* support_out, float* W_out,
               double* obj_trace, int32_t* swap_trace, osscar_search_result* res)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    Ptrs p = make_ptrs(ctx);
    const int g = L.g;
    const double tol = prm->accept_rel_tol < 0 ? 1e-5 : prm->accept_rel_tol;
    int max_swaps = (L.nJ > 0) ? prm->max_swaps : 0;

    k_begin<<<1, 1, 0, st>>>(ctx->ctl, obj_trace, ctx->done_flag_dev);
    count_launches(1);
    const bool own_limit = prm->wait_limit_cycles != 0;       // this search's budget for bounded waits; restored at the end
    if (own_limit) { k_search_wait_limit<<<1, 1, 0, st>>>(ctx->ctl, (long long)prm->wait_limit_cycles); count_launches(1); }
    CK(cudaGetLastError());
    CK(cudaEventRecord(ctx->ev0, st));
    const bool pair = prm->score_mode == OSSCAR_SCORE_PAIR_EXACT;
    const bool sharded = ctx->reduce != nullptr;          // column shards: sums over shards go through the caller's hook
    const int bs = prm->block_pairs > 1 ? prm->block_pairs : 1;     // groups exchanged per iteration
    const bool block = bs > 1;
    if (block) {
        if (pair || (int64_t)bs * g > L.block_rows_max || bs > L.k || bs > L.ng - L.k) return OSSCAR_E_ARG;
        if (block_bytes_for(L, bs * g) > L.block_bytes) return OSSCAR_E_WORKSPACE;
        if (panel_dot_tc_scratch(L.nJ > L.nI ? L.nJ : L.nI, 2 * bs * g, L.nI) + 1024 > L.tc_bytes) return OSSCAR_E_WORKSPACE;
    }
    BlockPtrs bp = make_block_ptrs(ctx, bs);
    const bool fast = g == 1 && !pair && !block;  // fused step for single-row groups
    // one cooperative kernel for the whole loop, unless asked otherwise or the device cannot hold such a grid
    // AUTO: the cooperative loop for states that stay in L2 (its barriers cost less than five launches per step: 2-8 x
    // the swaps per second measured on the small layers); the launch chain for states streamed from HBM, where four
    // resident blocks per SM of one-row kernels keep more loads in flight than the loop's blocks do (measured 0.81
    // against 0.71 of copy bandwidth on the OPT-30B-shaped FC2 layer)
    const double state_bytes = 8.0 * L.nI * L.ldh + 4.0 * (L.nI + L.nJ) * L.ldm + 4.0 * L.nJ * L.ldh;
    const bool want_persistent = sharded ? false : prm->loop_mode == OSSCAR_LOOP_PERSISTENT || (prm->loop_mode == OSSCAR_LOOP_AUTO && state_bytes <= 96.0e6);
    const int pgrid = (fast && want_persistent && L.nJ > 0) ? persistent_grid(L) : 0;
    if (prm->loop_mode == OSSCAR_LOOP_PERSISTENT && pgrid == 0) return OSSCAR_E_ARG;
    const bool persistent = pgrid > 0;
    if (block) max_swaps /= bs;                   // from here on: iterations
    const int64_t npairs = (int64_t)L.k * (L.ng - L.k);
    if (sharded && !(g == 1 && !pair && !block)) return OSSCAR_E_ARG;
    if (max_swaps > 0) CK(enqueue_scores(ctx, p, true, pair));
    if (max_swaps > 0 && sharded && shard_reduce(ctx, p.vnorm, L.d1, OSSCAR_FP32) != OSSCAR_OK) return OSSCAR_E_CUDA;
    const size_t inv_smem = ((size_t)g * g + 2 * (size_t)g) * sizeof(double);      // matrix under inversion + pivot row/column
    if (inv_smem > 48 * 1024) {
        CK(cudaFuncSetAttribute(k_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)inv_smem));
        CK(cudaFuncSetAttribute(k_pair_delta, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)inv_smem));
    }
    auto pair_scores = [&]() -> cudaError_t {      // PAIR_EXACT: exact change of obj of every (kept, pruned) pair
        float* Pm = (float*)((char*)ctx->ws + L.off_big);
        const int64_t ldj = round_up(L.nJ, kPadF);
        float* XG = Pm + L.nJ * L.ldh;
        cudaError_t e = sgemm(st, false, false, L.nJ, L.nI, L.nI, 1.f, p.Hp + L.nI * L.ldp, L.ldp, p.Hinv, L.ldh, 0.f, Pm, L.ldh,
                              &ctx->ctl->done);
        if (e != cudaSuccess) return e;
        e = sgemm(st, false, true, L.nI, L.nJ, L.m, 1.f, p.V, L.ldm, p.R, L.ldm, 0.f, XG, ldj, &ctx->ctl->done);
        if (e != cudaSuccess) return e;
        const size_t smem = 3 * (size_t)g * g * sizeof(double);
        e = cudaFuncSetAttribute(k_pair_slots, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_pair_slots<<<(unsigned)L.k, small_threads(g), smem, st>>>(p);
        k_pair_delta<<<(unsigned)(npairs < kPairBlocks ? npairs : kPairBlocks), small_threads(g), inv_smem, st>>>(p, Pm, L.ldh, XG, ldj, npairs);
        k_pair_select<<<1, 1024, 0, st>>>(p, npairs);
        count_launches(3);
        return cudaGetLastError();
    };
    auto bootstrap_g1 = [&]() -> cudaError_t {       // score vectors, first entering group and its y from the current state
        k_scores_g1<<<(unsigned)((L.d1 + 255) / 256), 256, 0, st>>>(p);
        k_select_in_g1<<<1, 1024, 0, st>>>(p);
        k_ypass_d<<<dim3((unsigned)((L.nI + 7) / 8), 1), 256, 0, st>>>(p);
        count_launches(3);
        return cudaGetLastError();
    };
    if (g == 1 && !fast) ctx->hd_valid = false;          // these drivers move the fp32 inverse only
    if (max_swaps > 0 && fast) {
        if (!ctx->hd_valid) { const int rcd = build_hinv64(ctx, false); if (rcd != OSSCAR_OK) return rcd; }
        CK(bootstrap_g1());
    }

    if (block) {
        CK(cudaMemsetAsync((char*)ctx->ws + L.off_block, 0, block_bytes_for(L, bs * g), st));
        const size_t smem = 2 * (size_t)g * bs * g * sizeof(double);
        if (smem > 48 * 1024) CK(cudaFuncSetAttribute(k_blk_update_c, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        const size_t smem2 = 2 * (size_t)bs * g * bs * g * sizeof(double);
        if (smem2 > 48 * 1024) CK(cudaFuncSetAttribute(k_blk_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
        if (smem2 / 2 > 48 * 1024) CK(cudaFuncSetAttribute(k_blk_update_c_g1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem2 / 2)));
    }
    if (g > 1) CK(cudaFuncSetAttribute(k_update_c, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * (size_t)g * g * sizeof(double))));

    // Steps per host batch.  The host stays at most two batches ahead of the device, so a loop that stops has up to
    // three batches of launches behind it that return at once (about 2 us each): short batches for states whose step is
    // short, where those launches would be a visible part of the solve.
    const int batch = block ? 4 : 8;
    cudaEvent_t evb[2];
    CK(cudaEventCreateWithFlags(&evb[0], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&evb[1], cudaEventDisableTiming));
    // optional kernel-by-kernel timing of a few evenly spaced steps
    constexpr int NK = OSSCAR_NUM_STEP_KERNELS;
    const int nprof = max_swaps > 0 ? (prm->profile_samples < max_swaps ? prm->profile_samples : max_swaps) : 0;
    cudaEvent_t evp[8][NK + 1];
    int prof_it[8];
    for (int i = 0; i < nprof; ++i) {
        prof_it[i] = (2 << i) - 1 < max_swaps ? (2 << i) - 1 : max_swaps - nprof + i;   // steps 1, 3, 7, 15, ...
        for (int j = 0; j <= NK; ++j) CK(cudaEventCreate(&evp[i][j]));
    }
    int rc = OSSCAR_OK;
    const unsigned yblocks = (unsigned)((L.nI + 7) / 8);
    constexpr int RPW = 4;
    const unsigned hblocks = (unsigned)((L.nJ + g + 8 * RPW - 1) / (8 * RPW));
    const unsigned gtiles = (unsigned)((g + TP_E - 1) / TP_E);
    auto tile_blocks = [](int64_t rows, int R) { return (unsigned)((rows + TP_W * R - 1) / (TP_W * R)); };
    auto tile_rows = [&](int64_t rows) {           // rows per warp: as many as still leave about 4096 warps in flight
        for (int R = 4; R > 1; R >>= 1) if ((rows + R - 1) / R * gtiles >= 4096) return R;
        return 1;
    };
    const unsigned prep_blocks = (unsigned)(((L.nI + L.ldm) * g + 255) / 256);
    // threads per block of the three streaming kernels of the single-row step, by the length of the rows they stream
    const unsigned t_l1 = (unsigned)g1_threads(L.ldm > L.ldh ? L.ldm / 4 : L.ldh / 4), t_l2 = (unsigned)g1_threads(L.ldm / 4),
                   t_l4 = (unsigned)g1_threads(L.ldh / 2);
    bool after_kernel = false;      // the last operation put on the stream was a kernel of the step
    auto dep = [&]() { const bool d = after_kernel; after_kernel = true; return d; };
    auto launch_l1 = [&](unsigned nbV, unsigned nbH) {
        const bool dp = dep();
        if (t_l1 == 64) launch_pdl(dp, k_l1_g1<64>, dim3(nbV + nbH), dim3(64), st, p, nbV);
        else if (t_l1 == 128) launch_pdl(dp, k_l1_g1<128>, dim3(nbV + nbH), dim3(128), st, p, nbV);
        else launch_pdl(dp, k_l1_g1<256>, dim3(nbV + nbH), dim3(256), st, p, nbV);
    };
    auto launch_l2 = [&](unsigned nbR) {       // the same number of threads exchange the two slots whatever the block size
        const bool dp = dep();
        if (t_l2 == 64) launch_pdl(dp, k_l2_g1<64>, dim3(nbR + 128), dim3(64), st, p, nbR);
        else if (t_l2 == 128) launch_pdl(dp, k_l2_g1<128>, dim3(nbR + 64), dim3(128), st, p, nbR);
        else launch_pdl(dp, k_l2_g1<256>, dim3(nbR + 32), dim3(256), st, p, nbR);
    };
    auto launch_l4 = [&]() {
        const unsigned nb = (unsigned)((L.nI + G1_RB4 - 1) / G1_RB4);
        const bool dp = dep();
        if (t_l4 == 64) launch_pdl(dp, k_l4_g1<G1_RB4, 64>, dim3(nb), dim3(64), st, p);
        else if (t_l4 == 128) launch_pdl(dp, k_l4_g1<G1_RB4, 128>, dim3(nb), dim3(128), st, p);
        else launch_pdl(dp, k_l4_g1<G1_RB4, 256>, dim3(nb), dim3(256), st, p);
    };
    int next_prof = 0;
    int nmarks = 0;                 // events recorded per profiled step (depends on the step variant)
    unsigned long long* loop_prof = (unsigned long long*)((char*)ctx->ws + L.off_loop + 2 * (size_t)kLoopMaxBlocks * 16);
    if (persistent && max_swaps > 0) {
        // chunks of steps between rebuilds of the state (one chunk when the state is only ever updated); a stopped loop
        // makes the remaining launches return at once, so no host round trip is needed in between
        LoopArgs la;
        la.p = p;
        la.candD = (LoopCand*)((char*)ctx->ws + L.off_loop);
        la.candA = la.candD + kLoopMaxBlocks;
        la.prof = loop_prof;
        la.obj_trace = obj_trace; la.swap_trace = swap_trace;
        la.tol = tol; la.accept_mode = prm->accept_mode; la.max_swaps = max_swaps;
        if (cudaMemsetAsync(loop_prof, 0, 8 * sizeof(unsigned long long), st) != cudaSuccess) rc = OSSCAR_E_CUDA;
        const int chunk = prm->refresh_every > 0 ? prm->refresh_every : max_swaps;
        for (int it0 = 0; it0 < max_swaps && rc == OSSCAR_OK; it0 += chunk) {
            if (it0 > 0) {
                rc = build_state(ctx, true);
                if (rc != OSSCAR_OK) break;
                k_count_refresh<<<1, 1, 0, st>>>(ctx->ctl);
                count_launches(1);
                if (enqueue_scores(ctx, p, true, false) != cudaSuccess || bootstrap_g1() != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            }
            la.max_steps = max_swaps - it0 < chunk ? max_swaps - it0 : chunk;
            if (cudaMemsetAsync(&ctx->ctl->bar_count, 0, sizeof(unsigned long long) + sizeof(int32_t), st) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            void* kargs[] = { (void*)&la };
            if (cudaLaunchCooperativeKernel((const void*)k_swap_loop_g1, dim3((unsigned)pgrid), dim3(PL_T), kargs, 0, st) != cudaSuccess) {
                rc = OSSCAR_E_CUDA; break;
            }
            count_launches(1);
        }
    }
    for (int it = 0; it < (persistent ? 0 : max_swaps) && rc == OSSCAR_OK; ++it) {
        if (it % batch == 0) {
            const int bi = it / batch;
            if (bi >= 2) {      // stay at most two batches ahead of the device, and stop feeding a finished loop
                if (cudaEventSynchronize(evb[bi & 1]) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
                // the loop's state at the end of batch bi - 2, copied in stream order: unlike the live flag, every shard
                // of a column-sharded layer reads the same value here, so all of them stop feeding at the same step
                if (ctx->done_flag_host[1 + (bi & 1)]) break;
            }
        }
        if (prm->refresh_every > 0 && it > 0 && it % prm->refresh_every == 0) {
            rc = build_state(ctx, true);
            if (rc != OSSCAR_OK) break;
            k_count_refresh<<<1, 1, 0, st>>>(ctx->ctl);
            count_launches(1);
            if (enqueue_scores(ctx, p, true, pair) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            if (sharded && shard_reduce(ctx, p.vnorm, L.d1, OSSCAR_FP32) != OSSCAR_OK) { rc = OSSCAR_E_CUDA; break; }
            if (fast && bootstrap_g1() != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            after_kernel = false;
        }
        cudaEvent_t* pe = nullptr;
        if (next_prof < nprof && prof_it[next_prof] == it) pe = evp[next_prof++];
        int slot = 0;
        auto mark = [&]() { if (pe) { cudaEventRecord(pe[slot], st); after_kernel = false; } ++slot; };
        mark();
        if (block) {
            if (enqueue_block_step(ctx, p, bp, prm->accept_mode, tol, obj_trace, swap_trace, mark) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
        } else if (fast && sharded) {
            // column shards: the same five launches, with the two sums over shards where a decision needs them --
            // the cross term of the chosen pair before the accept test, the row norms before the next scores
            const unsigned nbV = (unsigned)((L.nI + G1_RB - 1) / G1_RB), nbR = (unsigned)((L.nJ + G1_RB - 1) / G1_RB), nbH = nbR + 1;
            k_decide_g1<<<1, 1024, 0, st>>>(p, prm->accept_mode, tol, obj_trace, swap_trace, 1);
            if (shard_reduce(ctx, p.shard, 1, OSSCAR_FP64) != OSSCAR_OK) { rc = OSSCAR_E_CUDA; break; }
            k_decide_g1<<<1, 1024, 0, st>>>(p, prm->accept_mode, tol, obj_trace, swap_trace, 2);
            after_kernel = true;                                                                 mark();
            launch_l1(nbV, nbH);                                                                 mark();
            launch_l2(nbR);                                                                      mark();
            if (shard_reduce(ctx, p.vnorm, L.d1, OSSCAR_FP32) != OSSCAR_OK) { rc = OSSCAR_E_CUDA; break; }
            k_scores_sharded_g1<<<(unsigned)((L.d1 + 255) / 256), 256, 0, st>>>(p);
            k_select_in_g1<<<1, 1024, 0, st>>>(p);
            after_kernel = true;                                                                 mark();
            launch_l4();        mark();
            after_kernel = false;               // the next step opens with ordinary launches
            count_launches(7);
        } else if (fast) {
            // single-row groups: decide, {H pass || V}, {R || slot exchange}, next entering group, {Hinv + next y}
            // G1_RB rows per block; the H pass has one more block for the leaving row
            const unsigned nbV = (unsigned)((L.nI + G1_RB - 1) / G1_RB), nbR = (unsigned)((L.nJ + G1_RB - 1) / G1_RB), nbH = nbR + 1;
            launch_pdl(dep(), k_decide_g1, dim3(1), dim3(1024), st, p, (int)prm->accept_mode, tol, obj_trace, swap_trace, 0);   mark();
            launch_l1(nbV, nbH);                                                                 mark();
            launch_l2(nbR);                                                                      mark();
            launch_pdl(dep(), k_select_in_g1, dim3(1), dim3(1024), st, p);                              mark();
            launch_l4();                                                     mark();
            count_launches(5);
        } else {
            if (pair) { if (pair_scores() != cudaSuccess) { rc = OSSCAR_E_CUDA; break; } after_kernel = false; }
            else launch_pdl(dep(), k_select, dim3(1), dim3(1024), st, p);
            mark();
            launch_pdl(dep(), k_pairgram, dim3((unsigned)((3 * g * g + 7) / 8)), dim3(256), st, p);                          mark();
            if (g > 1) {
                const int R = tile_rows(L.nI);
                if (R == 4) launch_pdl(dep(), k_ypass_g<4>, dim3(tile_blocks(L.nI, 4), gtiles), dim3(32 * TP_W), st, p);
                else if (R == 2) launch_pdl(dep(), k_ypass_g<2>, dim3(tile_blocks(L.nI, 2), gtiles), dim3(32 * TP_W), st, p);
                else launch_pdl(dep(), k_ypass_g<1>, dim3(tile_blocks(L.nI, 1), gtiles), dim3(32 * TP_W), st, p);
            }
            else launch_pdl(dep(), k_ypass, dim3(yblocks, 1), dim3(256), st, p);
            mark();
            launch_pdl_smem(dep(), k_small, dim3(1), dim3(small_threads(g)), inv_smem, st, p, prm->accept_mode, tol, max_swaps, obj_trace, swap_trace);
            mark();
            launch_pdl(dep(), k_prep, dim3(prep_blocks), dim3(256), st, p);                                                  mark();
            if (g > 1) {
                const int R = tile_rows(L.nJ + g);
                if (R == 4) launch_pdl(dep(), k_hpass_g<4>, dim3(tile_blocks(L.nJ + g, 4), gtiles), dim3(32 * TP_W), st, p);
                else if (R == 2) launch_pdl(dep(), k_hpass_g<2>, dim3(tile_blocks(L.nJ + g, 2), gtiles), dim3(32 * TP_W), st, p);
                else launch_pdl(dep(), k_hpass_g<1>, dim3(tile_blocks(L.nJ + g, 1), gtiles), dim3(32 * TP_W), st, p);
            }
            else launch_pdl(dep(), k_hpass<RPW>, dim3(hblocks, 1), dim3(256), st, p);
            mark();
            if (g > 1) {
                const size_t sm_t = 2 * (size_t)g * TG_RT * sizeof(float);
                const unsigned hx = (unsigned)((L.ldh / 4 + TG_T - 1) / TG_T), hy = (unsigned)((L.nI + TG_RT - 1) / TG_RT);
                const unsigned mx = (unsigned)((L.ldm / 4 + TG_T - 1) / TG_T), ry = (unsigned)((L.nJ + TG_RT - 1) / TG_RT);
                if (pe) {           // a profiled step times the three updates one by one
                    launch_pdl_smem(dep(), k_update_hinv_g, dim3(hx, hy), dim3(TG_T), sm_t, st, p);          mark();
                    launch_pdl_smem(dep(), k_update_rows_g, dim3(mx, hy), dim3(TG_T), sm_t, st, p, 0);       mark();
                    launch_pdl_smem(dep(), k_update_rows_g, dim3(mx, ry), dim3(TG_T), sm_t, st, p, 1);       mark();
                } else {
                    launch_pdl_smem(dep(), k_update_all_g, dim3(hx * hy + mx * hy + mx * ry), dim3(TG_T), sm_t, st, p, hx * hy, mx * hy, hx, mx);
                    mark(); mark(); mark();
                }
            } else {
                launch_pdl(dep(), k_update_hinv, dim3((unsigned)((L.ldh / 4 + 255) / 256), (unsigned)((L.nI + HI_RT - 1) / HI_RT)), dim3(256), st, p);
                mark();
                launch_pdl(dep(), k_update_rows, dim3((unsigned)((L.nI + UP_ROWS - 1) / UP_ROWS)), dim3(256), st, p, 0);          mark();
                launch_pdl(dep(), k_update_rows, dim3((unsigned)((L.nJ + UP_ROWS - 1) / UP_ROWS)), dim3(256), st, p, 1);          mark();
            }
            count_launches(g > 1 && !pe ? 7 : 9);
            if (g > 1) {
                launch_pdl_smem(dep(), k_update_c, dim3((unsigned)(L.ng - L.k)), dim3(small_threads(g)), 2 * (size_t)g * g * sizeof(double), st, p);
                count_launches(1);
            }
            if (g > 1 || pair) {
                if (enqueue_scores(ctx, p, false, pair, true, dep()) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            }
            mark();
            launch_pdl(dep(), k_hswap, dim3((unsigned)((L.ldp * g + 255) / 256)), dim3(256), st, p, 0);                       mark();
            launch_pdl(dep(), k_hswap, dim3((unsigned)((L.ldp * g + 255) / 256)), dim3(256), st, p, 1);                       mark();
            count_launches(2);
        }
        if (pe) nmarks = slot;
        if (cudaGetLastError() != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
        if ((it + 1) % batch == 0) {
            if (cudaMemcpyAsync((void*)(ctx->done_flag_host + 1 + ((it / batch) & 1)), &ctx->ctl->done, sizeof(int32_t),
                                cudaMemcpyDeviceToHost, st) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            if (cudaEventRecord(evb[(it / batch) & 1], st) != cudaSuccess) { rc = OSSCAR_E_CUDA; break; }
            after_kernel = false;
        }
    }
    cudaEventDestroy(evb[0]);
    cudaEventDestroy(evb[1]);
    if (rc != OSSCAR_OK) {
        if (own_limit) k_search_wait_limit<<<1, 1, 0, st>>>(ctx->ctl, ctx->wait_limit);
        cudaStreamSynchronize(st);
        for (int i = 0; i < nprof; ++i) for (int j = 0; j <= NK; ++j) cudaEventDestroy(evp[i][j]);
        return rc;
    }
    CK(cudaEventRecord(ctx->ev1, st));
    if (fast && max_swaps > 0) {       // the fp32 inverse follows its fp64 copy (state reader, other drivers)
        k_hinv_from_d<<<(unsigned)L.nI, 256, 0, st>>>(p.Hd, p.Hinv, L.ldh, nullptr);
        count_launches(1);
    }

    // results: weights, support, objective recomputed from the final state
    CK(cudaMemsetAsync(W_out, 0, sizeof(float) * L.d1 * L.m, st));
    k_scatter_rows<<<(unsigned)L.nI, 256, 0, st>>>(p, W_out);
    k_sorted_support<<<(L.k + 255) / 256, 256, 0, st>>>(p, support_out);
    {
        float* big = (float*)((char*)ctx->ws + L.off_big);
        // G_I in slot order, then Tr(G_I^T V)
        CK(gather_rows(st, ctx->G, L.m, L.g, p.perm, 0, L.nI, big, L.ldm));
        CK(trace_product(st, big, L.ldm, p.V, L.ldm, L.nI, L.m, ctx->partials, &ctx->ctl->acc[1]));
        if (sharded) {      // Tr(G_I^T V) is a sum over this shard's columns
            k_shard_scalar<<<1, 1, 0, st>>>(ctx->ctl, p.shard, 0);
            if (shard_reduce(ctx, p.shard, 1, OSSCAR_FP64) != OSSCAR_OK) return OSSCAR_E_CUDA;
            k_shard_scalar<<<1, 1, 0, st>>>(ctx->ctl, p.shard, 1);
            count_launches(2);
        }
        k_final_obj<<<1, 1, 0, st>>>(ctx->ctl);
        count_launches(3);
    }
    if (own_limit) { k_search_wait_limit<<<1, 1, 0, st>>>(ctx->ctl, ctx->wait_limit); count_launches(1); }
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(ctx->ctl_host, ctx->ctl, sizeof(SearchCtl), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, ctx->ev0, ctx->ev1));
    res->n_swaps = ctx->ctl_host->n_swaps;
    res->stop_reason = ctx->ctl_host->stop_reason;
    res->n_refresh = ctx->ctl_host->n_refresh;
    res->status = ctx->ctl_host->status;
    res->obj_init = ctx->ctl_host->acc[2];
    res->obj_final = ctx->ctl_host->acc[3];
    res->ms_search = ms;
    res->loop_driver = persistent ? OSSCAR_LOOP_PERSISTENT : OSSCAR_LOOP_LAUNCHES;
    // kernel times of the sampled steps that really swapped (a stopped loop runs empty kernels)
    int used = 0;
    for (int i = 0; i < nprof; ++i) {
        if (i < next_prof && prof_it[i] < res->n_swaps / bs) {
            for (int j = 0; j + 1 < nmarks && j < NK; ++j) {
                float t = 0.f;
                if (cudaEventElapsedTime(&t, evp[i][j], evp[i][j + 1]) == cudaSuccess) res->ms_kernel[j] += t;
            }
            ++used;
        }
        for (int j = 0; j <= NK; ++j) cudaEventDestroy(evp[i][j]);
    }
    for (int j = 0; j < NK && used > 0; ++j) res->ms_kernel[j] /= (float)used;
    res->n_profiled = used;
    if (persistent && max_swaps > 0) {      // phase times of the persistent loop (block 0's clock), mean over its steps
        unsigned long long prof[8] = {0};
        CK(cudaMemcpy(prof, loop_prof, sizeof(prof), cudaMemcpyDeviceToHost));
        const double steps = prof[4] > 0 ? (double)prof[4] : 1.0;
        res->ms_kernel[0] = (float)(prof[0] / steps * 1e-6);      // decide + staging
        res->ms_kernel[1] = (float)(prof[1] / steps * 1e-6);      // H pass || V update
        res->ms_kernel[2] = (float)(prof[2] / steps * 1e-6);      // R update || slot exchange
        res->ms_kernel[3] = 0.f;                                  // (the selection rides on the other phases)
        res->ms_kernel[4] = (float)(prof[3] / steps * 1e-6);      // Hinv update + next y
        res->n_profiled = (int32_t)prof[4];
    }
    return ctx->ctl_host->status;
}

}  // namespace osscar
