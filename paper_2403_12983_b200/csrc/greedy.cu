// Nested (greedy) phase of Algorithm 1 (t_i = p_i = t_hat): start with every group kept, H^-1 and W* = H^-1 G,
// and per iteration prune the t_hat kept groups whose removal raises obj least (Eq. impact through Case 1 /
// Lemma A.1: D_i = Tr(V_r^T (Hinv_rr)^-1 V_r)), all chosen from the scores of the current support, then move
// (Hinv, V) to the smaller support with the joint Case-1 downdate over the T = t_hat * g removed rows:
//   Hinv' = Hinv - B C^-1 B^T,   V' = V - B C^-1 V_r,   obj' = obj + Tr(V_r^T C^-1 V_r),   B = Hinv[:, r], C = Hinv[r, r].
// Live groups occupy slots [0, n_live); the holes left by pruned groups are refilled from the tail, so both
// matrices stay dense.  When k groups remain the slot permutation is handed to the regular state build.
#include "osscar_internal.cuh"
#include "small_mat.cuh"
#include <math.h>
#include <limits.h>

namespace osscar {
namespace {

using namespace smallmat;

constexpr int kMaxT = 256;          // rows removed per iteration (t_hat * g)
constexpr int UT_COLS = 1024, UT_ROWS = 8;

struct GPtrs {
    float* A; int64_t lda;          // Hinv of the live rows (d1 x lda storage)
    float* V; int64_t ldv;          // optimal weights of the live rows
    int64_t m;
    float* B;                       // T x lda: rows r of A (= columns, A symmetric)
    float* BC;                      // T x lda: C^-1 B
    float* KT;                      // T x ldv: C^-1 V_r
    float* BCT; float* BT;          // n x T: transposes of BC and B (left operands of the tensor-core downdates)
    double* gram;                   // ngroups x g x g
    double* D;                      // ngroups
    double* Cm;                     // 3 x T x T doubles: C, work, C^-1
    int32_t* sel;                   // [0]: t, [1..t]: chosen slots (descending), [1+kMaxT ..]: move sources
    int32_t* perm;
    int32_t* drop_trace;            // may be null
    SearchCtl* ctl;
    int g;
};

__global__ void k_identity_perm(int32_t* perm, int32_t* slotof, int64_t ng)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < ng) { perm[i] = (int32_t)i; slotof[i] = (int32_t)i; }
}
__global__ void k_copy_pad2(const float* __restrict__ src, int64_t lds, int64_t cols, float* __restrict__ dst, int64_t ldd)
{
    const int64_t i = blockIdx.x;
    for (int64_t c = threadIdx.x; c < ldd; c += blockDim.x) dst[i * ldd + c] = c < cols ? src[i * lds + c] : 0.f;
}

// gram[grp][a][b] = V[grp*g+a,:] . V[grp*g+b,:]; grid (live groups, g).
__global__ void k_gr_gram(GPtrs p)
{
    const int g = p.g;
    const int64_t grp = blockIdx.x;
    const int a = blockIdx.y;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const float4* ra = reinterpret_cast<const float4*>(p.V + (grp * g + a) * p.ldv);
    if (g == 1) {                    // a single squared norm: the whole block shares the row
        __shared__ float red[32];
        float s = 0.f;
        for (int64_t c = threadIdx.x; c < p.ldv / 4; c += blockDim.x) {
            const float4 x = ra[c];
            s += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
        }
        s = warp_sum(s);
        if (lane == 0) red[w] = s;
        __syncthreads();
        if (threadIdx.x == 0) { float t = 0.f; for (int i = 0; i < nw; ++i) t += red[i]; p.gram[grp] = (double)t; }
        return;
    }
    for (int b = w; b < g; b += nw) {
        const float4* rb = reinterpret_cast<const float4*>(p.V + (grp * g + b) * p.ldv);
        float s = 0.f;
        for (int64_t c = lane; c < p.ldv / 4; c += 32) {
            const float4 x = ra[c], z = rb[c];
            s += x.x * z.x + x.y * z.y + x.z * z.z + x.w * z.w;
        }
        s = warp_sum(s);
        if (lane == 0) p.gram[(grp * g + a) * g + b] = (double)s;
    }
}
// D[grp] = Tr((Hinv_rr)^-1 Gram); one block per live group (dynamic smem 3 g^2 doubles).
__global__ void k_gr_score(GPtrs p)
{
    extern __shared__ double smd[];
    __shared__ double red[32];
    const int g = p.g, gg = g * g;
    double* M = smd; double* Lw = smd + gg; double* Out = Lw + gg;
    const int64_t grp = blockIdx.x;
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        M[idx] = 0.5 * ((double)p.A[(grp * g + i) * p.lda + grp * g + j] + (double)p.A[(grp * g + j) * p.lda + grp * g + i]);
    }
    __syncthreads();
    const double piv = spd_inverse(M, Lw, Out, g);
    const double tr = mat_trace_prod(Out, p.gram + grp * gg, g, red);
    if (threadIdx.x == 0) p.D[grp] = piv > 0.0 ? tr : INFINITY;
}

// The t cheapest live groups (ties -> smaller id), stored in descending slot order, and the tail slots that
// refill their holes.  One block.
__global__ void __launch_bounds__(1024) k_gr_select(GPtrs p, int n_live, int t, int trace_pos)
{
    __shared__ double sv[32]; __shared__ int sid[32], sidx[32];
    __shared__ int chosen[kMaxT];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    // every thread keeps the best of its own strided share; only the owner of a round's winner rescans its share
    double mine = INFINITY; int mid = INT_MAX, midx = -1;
    auto rescan = [&]() {
        mine = INFINITY; mid = INT_MAX; midx = -1;
        for (int i = tid; i < n_live; i += blockDim.x) {
            const double v = p.D[i]; const int id = p.perm[i];
            if (v < mine || (v == mine && id < mid)) { mine = v; mid = id; midx = i; }
        }
    };
    rescan();
    __shared__ int winner;
    for (int round = 0; round < t; ++round) {
        double best = mine; int bid = mid, bidx = midx;
        for (int o = 16; o > 0; o >>= 1) {
            const double ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oid = __shfl_xor_sync(0xffffffffu, bid, o), oidx = __shfl_xor_sync(0xffffffffu, bidx, o);
            if (ov < best || (ov == best && oid < bid)) { best = ov; bid = oid; bidx = oidx; }
        }
        __syncthreads();
        if (lane == 0) { sv[w] = best; sid[w] = bid; sidx[w] = bidx; }
        __syncthreads();
        if (tid == 0) {
            for (int i = 1; i < (int)(blockDim.x >> 5); ++i)
                if (sv[i] < best || (sv[i] == best && sid[i] < bid)) { best = sv[i]; bid = sid[i]; bidx = sidx[i]; }
            if (bidx < 0 || !isfinite(best)) { p.ctl->status = OSSCAR_E_NOTPD; bidx = n_live - 1 - round; }
            chosen[round] = bidx;
            if (p.drop_trace) p.drop_trace[trace_pos + round] = p.perm[bidx];
            p.D[bidx] = INFINITY;                 // not again in this iteration
            winner = bidx;
        }
        __syncthreads();
        if (winner % (int)blockDim.x == tid) rescan();
    }
    if (tid == 0) {
        // refill plan: the new live range is [0, n_new); every chosen slot below n_new is a hole, every slot of
        // [n_new, n_live) that was not chosen is a survivor; pair them one to one (all moves are independent)
        const int n_new = n_live - t;
        p.sel[0] = t;
        int nh = 0;
        for (int i = 0; i < t; ++i) { p.sel[1 + i] = chosen[i]; p.sel[1 + kMaxT + i] = -1; }
        int surv = n_new;
        for (int i = 0; i < t; ++i) {
            if (chosen[i] >= n_new) continue;                 // already in the tail: no move
            while (true) {                                    // next tail slot that was not chosen
                bool taken = false;
                for (int j = 0; j < t; ++j) taken |= chosen[j] == surv;
                if (!taken) break;
                ++surv;
            }
            p.sel[1 + kMaxT + i] = surv++;
            ++nh;
        }
    }
}

// B[e] = A[row r_e, :] (T rows), C = A[r, r] -> C^-1 (fp64), in one block for the small part.
__global__ void k_gr_stage_b(GPtrs p, int n_live)
{
    const int g = p.g, t = p.sel[0], T = t * g;
    const int e = blockIdx.x;
    if (e >= T) return;
    const int64_t r = (int64_t)p.sel[1 + e / g] * g + e % g;
    const int64_t n = (int64_t)n_live * g;
    for (int64_t c = threadIdx.x; c < p.lda; c += blockDim.x) p.B[(int64_t)e * p.lda + c] = c < n ? p.A[r * p.lda + c] : 0.f;
}
__global__ void __launch_bounds__(1024) k_gr_cinv(GPtrs p, int in_smem)
{
    extern __shared__ double smg[];           // T^2 + 2 T doubles when the matrix fits
    const int g = p.g, t = p.sel[0], T = t * g;
    double* C = in_smem ? smg : p.Cm; double* Lw = in_smem ? smg + T * T : p.Cm + kMaxT * kMaxT; double* Cinv = p.Cm + 2 * kMaxT * kMaxT;
    for (int idx = threadIdx.x; idx < T * T; idx += blockDim.x) {
        const int a = idx / T, b = idx % T;
        const int64_t ra = (int64_t)p.sel[1 + a / g] * g + a % g, rb = (int64_t)p.sel[1 + b / g] * g + b % g;
        C[idx] = 0.5 * ((double)p.A[ra * p.lda + rb] + (double)p.A[rb * p.lda + ra]);
    }
    __syncthreads();
    const double piv = spd_inverse(C, Lw, Cinv, T);
    if (threadIdx.x == 0 && !(piv > 0.0)) p.ctl->status = OSSCAR_E_NOTPD;
}
// BC[e][s] = sum_f Cinv[e][f] B[f][s]  and  KT[e][c] = sum_f Cinv[e][f] V[r_f][c];  obj += sum_e KT[e] . V[r_e].
__global__ void k_gr_stage_bc(GPtrs p, int n_live)
{
    const int g = p.g, t = p.sel[0], T = t * g;
    const double* Cinv = p.Cm + 2 * kMaxT * kMaxT;
    const int64_t nA = (int64_t)T * p.lda, nV = (int64_t)T * p.ldv;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < nA + nV; idx += (int64_t)gridDim.x * blockDim.x) {
        if (idx < nA) {
            const int e = (int)(idx / p.lda); const int64_t s = idx % p.lda;
            double acc = 0.0;
            for (int f = 0; f < T; ++f) acc += Cinv[e * T + f] * (double)p.B[(int64_t)f * p.lda + s];
            p.BC[idx] = (float)acc;
            if (s < (int64_t)n_live * g) { p.BCT[s * T + e] = (float)acc; p.BT[s * T + e] = p.B[(int64_t)e * p.lda + s]; }
        } else {
            const int64_t j = idx - nA;
            const int e = (int)(j / p.ldv); const int64_t c = j % p.ldv;
            double acc = 0.0;
            for (int f = 0; f < T; ++f) {
                const int64_t rf = (int64_t)p.sel[1 + f / g] * g + f % g;
                acc += Cinv[e * T + f] * (double)p.V[rf * p.ldv + c];
            }
            p.KT[j] = (float)acc;
        }
    }
}
__global__ void __launch_bounds__(256) k_gr_obj(GPtrs p, double* __restrict__ partial)
{
    __shared__ double red[32];
    const int g = p.g, t = p.sel[0], T = t * g;
    double acc = 0.0;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < (int64_t)T * p.ldv; idx += (int64_t)gridDim.x * blockDim.x) {
        const int e = (int)(idx / p.ldv); const int64_t c = idx % p.ldv;
        const int64_t re = (int64_t)p.sel[1 + e / g] * g + e % g;
        acc += (double)p.KT[idx] * (double)p.V[re * p.ldv + c];
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) { double s = 0.0; for (int i = 0; i < (int)(blockDim.x >> 5); ++i) s += red[i]; partial[blockIdx.x] = s; }
}
__global__ void k_gr_obj_add(SearchCtl* ctl, const double* __restrict__ partial, int n)
{
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += partial[i];      // fixed order
    ctl->obj += s;
}

// M[s][c] -= sum_e left[e][s] * right[e][c] for live rows s and columns c < ncols (M = A with right = B, or
// M = V with right = KT).  Block: 1024 columns x 8 rows; the right-hand pieces of a thread are reused by its 8 rows.
__global__ void __launch_bounds__(256)
k_gr_update(float* __restrict__ M, int64_t ld, int64_t ncols4, int64_t nrows, const float* __restrict__ left, int64_t ldl,
            const float* __restrict__ right, int64_t ldr, const int32_t* __restrict__ sel, int g)
{
    const int T = sel[0] * g;
    const int64_t c4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c4 >= ncols4) return;
    const int64_t row0 = (int64_t)blockIdx.y * UT_ROWS;
    float4 acc[UT_ROWS];
#pragma unroll
    for (int i = 0; i < UT_ROWS; ++i) {
        const int64_t s = row0 + i;
        acc[i] = s < nrows ? reinterpret_cast<const float4*>(M + s * ld)[c4] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int e = 0; e < T; ++e) {
        const float4 rv = __ldg(reinterpret_cast<const float4*>(right + (int64_t)e * ldr) + c4);
#pragma unroll
        for (int i = 0; i < UT_ROWS; ++i) {
            const int64_t s = row0 + i;
            const float l = s < nrows ? -__ldg(left + (int64_t)e * ldl + s) : 0.f;
            acc[i].x = fmaf(l, rv.x, acc[i].x); acc[i].y = fmaf(l, rv.y, acc[i].y);
            acc[i].z = fmaf(l, rv.z, acc[i].z); acc[i].w = fmaf(l, rv.w, acc[i].w);
        }
    }
#pragma unroll
    for (int i = 0; i < UT_ROWS; ++i) {
        const int64_t s = row0 + i;
        if (s < nrows) reinterpret_cast<float4*>(M + s * ld)[c4] = acc[i];
    }
}

// Refill the holes: phase 0 copies whole rows of A and V from the tail slots into the holes and exchanges the
// permutation entries; phase 1 copies the matching columns of A for every remaining live row.
__global__ void k_gr_compact(GPtrs p, int phase, int64_t n_new_rows /* live groups after the iteration */)
{
    const int g = p.g, t = p.sel[0];
    for (int i = blockIdx.y; i < t; i += gridDim.y) {
        const int dst = p.sel[1 + i], src = p.sel[1 + kMaxT + i];
        if (src < 0) continue;
        if (phase == 0) {
            const int64_t n = (p.lda + p.ldv) * g;
            for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (int64_t)gridDim.x * blockDim.x) {
                const int e = (int)(idx / (p.lda + p.ldv)); const int64_t x = idx % (p.lda + p.ldv);
                if (x < p.lda) p.A[((int64_t)dst * g + e) * p.lda + x] = p.A[((int64_t)src * g + e) * p.lda + x];
                else p.V[((int64_t)dst * g + e) * p.ldv + (x - p.lda)] = p.V[((int64_t)src * g + e) * p.ldv + (x - p.lda)];
            }
            if (blockIdx.x == 0 && threadIdx.x == 0) {
                const int a = p.perm[dst], b = p.perm[src];
                p.perm[dst] = b; p.perm[src] = a;
            }
        } else {
            const int64_t n = n_new_rows * g * g;          // every live row (n_new groups x g) times the g moved columns
            for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (int64_t)gridDim.x * blockDim.x) {
                const int64_t row = idx / g; const int e = (int)(idx % g);
                p.A[row * p.lda + (int64_t)dst * g + e] = p.A[row * p.lda + (int64_t)src * g + e];
            }
        }
    }
}
// Groups pruned without a refill (the hole was the tail itself) still have to leave the kept part of the
// permutation: they already sit at positions >= the new live count, nothing to do.

__global__ void k_sorted_prefix(const int32_t* __restrict__ perm, int k, int32_t* __restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= k) return;
    const int id = perm[i];
    int rank = 0;
    for (int j = 0; j < k; ++j) rank += perm[j] < id;
    out[rank] = id;
}
__global__ void k_sort_perm_prefix(int32_t* __restrict__ perm, const int32_t* __restrict__ sorted, int k)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < k) perm[i] = sorted[i];
}
__global__ void k_fix_pruned_order(int32_t* __restrict__ perm, int32_t* __restrict__ slotof, int k, int64_t ng, int32_t* __restrict__ tmp)
{
    // pruned groups in ascending id order behind the kept ones (the order the regular initialiser uses)
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= ng) return;
    if (i >= k) {
        const int id = perm[i];
        int rank = 0;
        for (int64_t j = k; j < ng; ++j) rank += perm[j] < id;
        tmp[k + rank] = id;
    } else tmp[i] = perm[i];
}
__global__ void k_store_perm(int32_t* __restrict__ perm, int32_t* __restrict__ slotof, const int32_t* __restrict__ tmp, int64_t ng)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < ng) { perm[i] = tmp[i]; slotof[tmp[i]] = (int32_t)i; }
}
__global__ void k_set_obj0(SearchCtl* ctl) { ctl->const_term = ctl->acc[0]; ctl->obj = ctl->acc[0] - ctl->acc[1]; }

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) return OSSCAR_E_CUDA; } while (0)

}  // namespace

size_t greedy_scratch_bytes(int64_t d1, int64_t m, int g)
{
    const int64_t ng = d1 / g;
    return sizeof(double) * (size_t)(ng * g * g + ng + 3 * kMaxT * kMaxT) + sizeof(int32_t) * (size_t)(2 * kMaxT + 16 + 2 * ng) + 4096;
}

// Runs the nested phase down to L.k groups; leaves the slot permutation (kept groups sorted in slots [0, k)) in the
// workspace and the sorted kept ids in `support`.  The caller then builds the regular search state.
int greedy_support(osscar_ctx* ctx, int t_hat, int32_t* support, int32_t* drop_trace, int32_t* n_iters_out)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    char* ws = (char*)ctx->ws;
    const int g = L.g;
    const int64_t d1 = L.d1, ng = L.ng;
    if (t_hat < 1 || (int64_t)t_hat * g > kMaxT) return OSSCAR_E_SHAPE;
    const int64_t T = (int64_t)t_hat * g;
    // scratch carved from `big` (2 d1 ldm floats at least): V of all rows, then B, BC (T x ldp each), KT (T x ldm)
    float* big = (float*)(ws + L.off_big);
    const size_t big_floats = (L.off_Hp - L.off_big) / sizeof(float);
    const size_t need = (size_t)d1 * L.ldm + 2 * (size_t)T * L.ldp + (size_t)T * L.ldm + 2 * (size_t)d1 * T;
    if (need > big_floats) return OSSCAR_E_WORKSPACE;
    GPtrs p;
    p.A = (float*)(ws + L.off_Hp); p.lda = L.ldp;
    p.V = big; p.ldv = L.ldm; p.m = L.m;
    p.B = big + (size_t)d1 * L.ldm; p.BC = p.B + (size_t)T * L.ldp; p.KT = p.BC + (size_t)T * L.ldp;
    p.BCT = p.KT + (size_t)T * L.ldm; p.BT = p.BCT + (size_t)d1 * T;
    char* gs = ws + L.off_greedy;
    p.gram = (double*)gs; p.D = p.gram + ng * g * g; p.Cm = p.D + ng;
    p.sel = (int32_t*)(p.Cm + 3 * kMaxT * kMaxT);
    int32_t* tmp = p.sel + 2 * kMaxT + 16;
    p.perm = (int32_t*)(ws + L.off_perm);
    int32_t* slotof = (int32_t*)(ws + L.off_slotof);
    p.drop_trace = drop_trace; p.ctl = ctx->ctl; p.g = g;

    const unsigned nbg = (unsigned)((ng + 255) / 256);
    k_identity_perm<<<nbg, 256, 0, st>>>(p.perm, slotof, ng);
    k_copy_pad2<<<(unsigned)d1, 256, 0, st>>>(ctx->H, d1, d1, p.A, p.lda);
    count_launches(2);
    // fp32 pipes for the rank-64 updates: no correction of the inverse follows here
    int rc = invert_spd_inplace(ctx, p.A, p.lda, d1, ctx->H, d1, nullptr, false);
    if (rc != OSSCAR_OK) return rc;
    // W* = H^-1 G (Algorithm 1, line 1)
    if (L.ldm != L.m) CK(cudaMemsetAsync(p.V, 0, sizeof(float) * d1 * L.ldm, st));
    CK(sgemm(st, false, false, d1, L.m, d1, 1.f, p.A, p.lda, ctx->G, L.m, 0.f, p.V, L.ldm));
    if (ctx->have_const) CK(set_device_double(st, &ctx->ctl->acc[0], ctx->user_const));
    else CK(trace_product(st, ctx->W, L.m, ctx->G, L.m, d1, L.m, ctx->partials, &ctx->ctl->acc[0]));
    CK(trace_product(st, ctx->G, L.m, p.V, L.ldm, d1, L.m, ctx->partials, &ctx->ctl->acc[1]));
    k_set_obj0<<<1, 1, 0, st>>>(ctx->ctl);
    count_launches(1);

    const size_t smem_score = 3 * (size_t)g * g * sizeof(double);
    CK(cudaFuncSetAttribute(k_gr_score, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_score));
    CK(cudaFuncSetAttribute(k_gr_cinv, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    int n_live = (int)ng, iters = 0, trace_pos = 0;
    while (n_live > L.k) {
        const int t = n_live - L.k < t_hat ? n_live - L.k : t_hat;
        const int64_t nrows = (int64_t)n_live * g;
        k_gr_gram<<<dim3((unsigned)n_live, (unsigned)g), 128, 0, st>>>(p);
        k_gr_score<<<(unsigned)n_live, g == 1 ? 32 : 256, smem_score, st>>>(p);
        k_gr_select<<<1, 1024, 0, st>>>(p, n_live, t, trace_pos);
        k_gr_stage_b<<<(unsigned)(t * g), 256, 0, st>>>(p, n_live);
        {
            const size_t cs = ((size_t)t * g * t * g + 2 * (size_t)t * g) * sizeof(double);
            const bool fits = cs <= 200 * 1024;
            k_gr_cinv<<<1, fits ? 1024 : 256, fits ? cs : 0, st>>>(p, fits ? 1 : 0);
        }
        k_gr_stage_bc<<<(unsigned)(((int64_t)t * g * (p.lda + p.ldv) + 255) / 256 < 2368 ? ((int64_t)t * g * (p.lda + p.ldv) + 255) / 256 : 2368), 256, 0, st>>>(p, n_live);
        k_gr_obj<<<128, 256, 0, st>>>(p, ctx->partials);
        k_gr_obj_add<<<1, 1, 0, st>>>(ctx->ctl, ctx->partials, 128);
        const int64_t Tt = (int64_t)t * g;
        if (Tt >= 32) {
            // wide downdates: A -= BC^T B and V -= B^T KT as products with inner dimension T on the tensor cores
            void* tc = ws + L.off_tc;
            if (rank_update_tc(st, nrows, round_up(nrows, 4), Tt, -1.f, p.BCT, Tt, p.B, p.lda, p.A, p.lda, tc, L.tc_bytes, ctx->ctl)
                    != cudaSuccess) return OSSCAR_E_CUDA;
            if (rank_update_tc(st, nrows, p.ldv, Tt, -1.f, p.BT, Tt, p.KT, p.ldv, p.V, p.ldv, tc, L.tc_bytes, ctx->ctl)
                    != cudaSuccess) return OSSCAR_E_CUDA;
        } else {
            const int64_t nc4 = (round_up(nrows, 4)) / 4;
            dim3 ga((unsigned)((nc4 + 255) / 256), (unsigned)((nrows + UT_ROWS - 1) / UT_ROWS));
            k_gr_update<<<ga, 256, 0, st>>>(p.A, p.lda, nc4, nrows, p.BC, p.lda, p.B, p.lda, p.sel, g);
            const int64_t nv4 = p.ldv / 4;
            dim3 gv((unsigned)((nv4 + 255) / 256), (unsigned)((nrows + UT_ROWS - 1) / UT_ROWS));
            k_gr_update<<<gv, 256, 0, st>>>(p.V, p.ldv, nv4, nrows, p.B, p.lda, p.KT, p.ldv, p.sel, g);     // V -= B (C^-1 V_r)
        }
        const int n_new = n_live - t;
        k_gr_compact<<<dim3(64, (unsigned)t), 256, 0, st>>>(p, 0, (int64_t)n_new);
        k_gr_compact<<<dim3(64, (unsigned)t), 256, 0, st>>>(p, 1, (int64_t)n_new);
        count_launches(12);
        CK(cudaGetLastError());
        n_live = n_new; trace_pos += t; ++iters;
    }
    // kept groups sorted into slots [0, k), pruned groups ascending behind them
    k_sorted_prefix<<<(L.k + 255) / 256, 256, 0, st>>>(p.perm, L.k, support);
    k_sort_perm_prefix<<<(L.k + 255) / 256, 256, 0, st>>>(p.perm, support, L.k);
    k_fix_pruned_order<<<nbg, 256, 0, st>>>(p.perm, slotof, L.k, ng, tmp);
    k_store_perm<<<nbg, 256, 0, st>>>(p.perm, slotof, tmp, ng);
    count_launches(4);
    CK(cudaGetLastError());
    if (n_iters_out) *n_iters_out = iters;
    return OSSCAR_OK;
}

}  // namespace osscar
