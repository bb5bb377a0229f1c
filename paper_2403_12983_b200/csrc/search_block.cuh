// Block exchanges: local-search iterations of Algorithm 1 with p_hat = 0 and t_hat = 2 s (Eq. local, Eq. impact).
// The s kept groups with the lowest drop score leave and the s pruned groups with the highest add score enter in ONE
// rank-2G update (G = s g rows on each side), so every matrix of the state is streamed once per s swaps.
// Included by search.cu (same translation unit: uses its Ptrs, small-matrix slots and reductions).
//
// The algebra is that of a single swap (header of search.cu) with r = the G leaving rows and q = the G entering
// rows, given by index lists instead of one contiguous group; the joint Schur complement of the entering rows,
// c_qq = H_qq - H_qI Hinv H_Iq, is formed from y because the state only carries its diagonal blocks.
// Panels (row-major, one staged vector per row):
//   hT, yT (G x ldh)   h = Hp[q, 0:n_I],  y = Hinv h
//   PB (2G x ldh)      [ b ; u2 ]          b = rows r of Hinv
//   PA (2G x ldh)      [ b C^-1 ; -u2 c1^-1 ]
//   KV (2G x ldm)      [ K ; Vq ]
//   PBT, PAT (n_I x 2G) the transposes of PB and PA (left operands of the update GEMMs)
//   UD ((n_J+G) x 2G)  [ u | -d ] for the pruned rows, then the leaving rows
//   Hinv' = Hinv - PA^T PB,   V' = V - PB^T KV,   R' = R + UD KV      (three GEMMs with inner dimension 2G)
#pragma once

struct BlockPtrs {
    int32_t *rslot, *tslot;        // kept slots that leave (cheapest first), pruned slots that enter (best first)
    float *hT, *yT, *HrT, *PB, *PA, *PBT, *PAT, *KV, *Vr, *Rq, *UD;
    double* small;                 // kBlockSmall matrices of G x G doubles
    int s, G;
};
constexpr int kBlockSmall = 18;
constexpr int kBlockMaxPairs = OSSCAR_MAX_GROUP;      // s g <= OSSCAR_MAX_GROUP rows per side, hence at most that many groups
enum { B_CQ = 16, B_HY = 17 };     // joint Schur complement of the entering rows, h^T y

size_t block_bytes_for(const Layout& L, int G) { return osscar::block_region_bytes(L.ldh, L.ldm, L.nJ, G); }

BlockPtrs make_block_ptrs(osscar_ctx* ctx, int s)
{
    const Layout& L = ctx->L;
    const int G = s * L.g;
    char* base = (char*)ctx->ws + L.off_block;
    size_t off = 0;
    auto take = [&](size_t b) { char* q = base + off; off += (b + 255) / 256 * 256; return q; };
    BlockPtrs bp;
    bp.s = s; bp.G = G;
    bp.rslot = (int32_t*)take(sizeof(int32_t) * (size_t)G);
    bp.tslot = (int32_t*)take(sizeof(int32_t) * (size_t)G);
    bp.hT = (float*)take(sizeof(float) * (size_t)G * L.ldh);
    bp.yT = (float*)take(sizeof(float) * (size_t)G * L.ldh);
    bp.HrT = (float*)take(sizeof(float) * (size_t)G * L.ldh);
    bp.PB = (float*)take(sizeof(float) * 2 * (size_t)G * L.ldh);
    bp.PA = (float*)take(sizeof(float) * 2 * (size_t)G * L.ldh);
    bp.PBT = (float*)take(sizeof(float) * 2 * (size_t)G * L.ldh);
    bp.PAT = (float*)take(sizeof(float) * 2 * (size_t)G * L.ldh);
    bp.KV = (float*)take(sizeof(float) * 2 * (size_t)G * L.ldm);
    bp.Vr = (float*)take(sizeof(float) * (size_t)G * L.ldm);
    bp.Rq = (float*)take(sizeof(float) * (size_t)G * L.ldm);
    bp.UD = (float*)take(sizeof(float) * (size_t)(L.nJ + G) * 2 * G);
    bp.small = (double*)take(sizeof(double) * kBlockSmall * (size_t)G * G);
    return bp;
}

// row of the e-th leaving row among the kept slots / of the e-th entering row among the pruned slots
__device__ __forceinline__ int64_t blk_rrow(const Ptrs& p, const BlockPtrs& bp, int e) { return (int64_t)bp.rslot[e / p.g] * p.g + e % p.g; }
__device__ __forceinline__ int64_t blk_qrow(const Ptrs& p, const BlockPtrs& bp, int e) { return (int64_t)bp.tslot[e / p.g] * p.g + e % p.g; }

// Monotone map of a double onto an unsigned integer (smaller value, smaller key); -0 counts as +0.
__device__ __forceinline__ unsigned long long blk_ordered_key(double v)
{
    const unsigned long long u = (unsigned long long)__double_as_longlong(v + 0.0);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// One digit of a radix selection over the block: among the n items that `in_class` admits, the digit (0..255) whose
// bin holds the item of rank `want` (1-based, ascending), how many admitted items lie in the bins below it and how many
// in that bin.  hist is [32 warps][256] in shared memory; every thread of the block calls this with the same n and want.
template <class Digit>
__device__ __forceinline__ void blk_radix_digit(int n, int want, Digit&& digit_of, unsigned* hist, unsigned* bcast, int& digit, int& below,
                                                int& in_bin)
{
    const int t = threadIdx.x, lane = t & 31, w = t >> 5, nt = blockDim.x, nw = nt >> 5;
    for (int i = t; i < nw * 256; i += nt) hist[i] = 0;
    __syncthreads();
    constexpr int RB = 8;                                 // items per thread whose loads are in flight together
    for (int i0 = 0; i0 < n; i0 += nt * RB) {             // whole warps stay together for the lane vote
        int d[RB];
#pragma unroll
        for (int b = 0; b < RB; ++b) {
            const int i = i0 + b * nt + t;
            d[b] = i < n ? digit_of(i) : -1;              // -1: not in the class
        }
#pragma unroll
        for (int b = 0; b < RB; ++b) {
            const unsigned peers = __match_any_sync(0xffffffffu, d[b]);
            if (d[b] >= 0 && lane == __ffs(peers) - 1) hist[w * 256 + d[b]] += __popc(peers);    // one lane per distinct digit
            __syncwarp();
        }
    }
    __syncthreads();
    if (t < 256) { unsigned c = 0; for (int ww = 0; ww < nw; ++ww) c += hist[ww * 256 + t]; hist[t] = c; }
    __syncthreads();
    if (w == 0) {                                         // lane owns bins 8 lane .. 8 lane + 7
        unsigned c[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = hist[lane * 8 + j]; sum += c[j]; }
        unsigned incl = sum;
        for (int o = 1; o < 32; o <<= 1) { const unsigned v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
        unsigned run = incl - sum;                        // items in the bins of the lanes before this one
        const bool mine = run < (unsigned)want && (unsigned)want <= incl;
        if (mine) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (run < (unsigned)want && (unsigned)want <= run + c[j]) { bcast[0] = lane * 8 + j; bcast[1] = run; bcast[2] = c[j]; }
                run += c[j];
            }
        }
    }
    __syncthreads();
    digit = (int)bcast[0]; below = (int)bcast[1]; in_bin = (int)bcast[2];
    __syncthreads();
}

// The s cheapest kept slots (block 0) and the s most valuable pruned slots (block 1), from the scores at the current
// support; ties go to the smaller group id; the lists come out in the order in which a repeated arg-min would draw
// them.  Radix selection: 8-bit digits of the ordered key, most significant first, narrow down the value of the s-th
// item until the bin of the current digit holds only items that belong; if several items share that value exactly,
// digits of their group ids fix the last id that still belongs; the members are then gathered and ranked among
// themselves.
__global__ void __launch_bounds__(1024) k_blk_select(Ptrs p, BlockPtrs bp)
{
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ unsigned hist[32 * 256];
    __shared__ unsigned bcast[3];
    __shared__ int guard;
    __shared__ unsigned long long selk[kBlockMaxPairs];
    __shared__ int selid[kBlockMaxPairs], selix[kBlockMaxPairs];
    __shared__ int nsel;
    const int side = blockIdx.x;
    const int n = side == 0 ? p.k : (int)(p.ng - p.k);
    double* val = side == 0 ? p.D : p.A;
    const int32_t* ids = side == 0 ? p.perm : p.perm + p.k;
    int32_t* out = side == 0 ? bp.rslot : bp.tslot;
    const int t = threadIdx.x, nt = blockDim.x, s = bp.s;
    if (p.g == 1) {                       // single-row groups: scores from the row norms
        constexpr int SB = 8;             // diagonal entries (one DRAM sector each) requested together
        for (int i0 = 0; i0 < n; i0 += nt * SB) {
            float hd[SB];
#pragma unroll
            for (int b = 0; b < SB; ++b) {
                const int64_t i = i0 + b * nt + t;
                hd[b] = i < n ? (side == 0 ? p.Hinv[i * p.ldh + i] : p.Hp[(p.nI + i) * p.ldp + p.nI + i]) : 0.f;
            }
#pragma unroll
            for (int b = 0; b < SB; ++b) {
                const int i = i0 + b * nt + t;
                if (i >= n) continue;
                if (side == 0) val[i] = hd[b] > 0.f ? (double)p.vnorm[i] / (double)hd[b] : INFINITY;
                else {
                    const double cc = p.c[i];
                    val[i] = cc > kAddPivotTol * (double)hd[b] ? (double)p.rnorm[i] / cc : -INFINITY;
                }
            }
        }
        __syncthreads();
    }
    const double sign = side == 0 ? 1.0 : -1.0;
    auto key_of = [&](int i) { return blk_ordered_key(sign * val[i]); };
    // Leading digits of the s-th smallest key.  As soon as the bin of the current digit holds no more items than are
    // still wanted, every item of it belongs and the remaining digits need not be resolved (usually after 3-4 of 8).
    unsigned long long T = 0;
    int want = s, kshift = 0;
    bool open = true;                     // the bin of the last digit still holds items that do not belong
    for (int pass = 0; pass < 8 && open; ++pass) {
        const int shift = 56 - 8 * pass;
        int digit, below, in_bin;
        blk_radix_digit(n, want, [&](int i) {
            const unsigned long long k = key_of(i);
            return (pass == 0 || (k >> (shift + 8)) == (T >> (shift + 8))) ? (int)((k >> shift) & 255) : -1;
        }, hist, bcast, digit, below, in_bin);
        T |= (unsigned long long)digit << shift;
        want -= below;
        kshift = shift;
        open = in_bin > want;
    }
    // still open after the last digit: several items have exactly the value T and `want` of them belong, those with
    // the smallest ids
    unsigned idT = 0;
    int ishift = 32;                      // 32: no id digit was needed
    for (int pass = 0; pass < 4 && open; ++pass) {
        const int shift = 24 - 8 * pass;
        int digit, below, in_bin;
        blk_radix_digit(n, want, [&](int i) {
            if (key_of(i) != T) return -1;
            const unsigned id = (unsigned)ids[i];
            return (pass == 0 || (id >> (shift + 8)) == (idT >> (shift + 8))) ? (int)((id >> shift) & 255) : -1;
        }, hist, bcast, digit, below, in_bin);
        idT |= (unsigned)digit << shift;
        want -= below;
        ishift = shift;
        open = in_bin > want;
    }
    if (t == 0) { nsel = 0; guard = 0; }
    __syncthreads();
    const unsigned long long kInf = blk_ordered_key(INFINITY);
    for (int i = t; i < n; i += nt) {
        const unsigned long long k = key_of(i);
        const int id = ids[i];
        const bool member = ishift == 32 ? (k >> kshift) <= (T >> kshift)
                                         : (k < T || (k == T && ((unsigned)id >> ishift) <= (idT >> ishift)));
        if (member) {
            const int at = atomicAdd(&nsel, 1);
            if (at < kBlockMaxPairs) { selk[at] = k; selid[at] = id; selix[at] = i; }
            if (k >= kInf) guard = 1;     // fewer than s candidates with a finite score
        }
    }
    __syncthreads();
    if (guard) {
        if (t == 0) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
        return;
    }
    if (t < s) {                          // exactly s members; rank each among them by (value, id)
        int rank = 0;
        for (int j = 0; j < s; ++j) rank += (selk[j] < selk[t] || (selk[j] == selk[t] && selid[j] < selid[t])) ? 1 : 0;
        out[rank] = selix[t];
    }
}

// Rows of the exchange copied into the panels: hT, HrT (rows of Hp), b (rows of Hinv), V_r, R_q.  grid (G, 5).
__global__ void __launch_bounds__(256) k_blk_gather(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int e = blockIdx.x, which = blockIdx.y;
    const int64_t rrow = blk_rrow(p, bp, e), qrow = blk_qrow(p, bp, e);
    const float* src; float* dst; int64_t n, valid;
    switch (which) {
    case 0:  src = p.Hp + (p.nI + qrow) * p.ldp; dst = bp.hT + (int64_t)e * p.ldh;  n = p.ldh; valid = p.nI; break;
    case 1:  src = p.Hp + rrow * p.ldp;          dst = bp.HrT + (int64_t)e * p.ldh; n = p.ldh; valid = p.nI; break;
    case 2:  src = p.Hinv + rrow * p.ldh;        dst = bp.PB + (int64_t)e * p.ldh;  n = p.ldh; valid = p.nI; break;
    case 3:  src = p.V + rrow * p.ldm;           dst = bp.Vr + (int64_t)e * p.ldm;  n = p.ldm; valid = p.m; break;
    default: src = p.R + qrow * p.ldm;           dst = bp.Rq + (int64_t)e * p.ldm;  n = p.ldm; valid = p.m; break;
    }
    for (int64_t x = threadIdx.x; x < n; x += blockDim.x) dst[x] = x < valid ? src[x] : 0.f;
}

// G x G Grams of the panels, one warp per entry: GV = V_r V_r^T, GX = V_r R_q^T, GR = R_q R_q^T, HY = h^T y.
__global__ void __launch_bounds__(256) k_blk_gram(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= 4LL * G * G) return;
    const int which = (int)(wid / (G * G)), a = (int)((wid / G) % G), b = (int)(wid % G);
    const int lane = threadIdx.x & 31;
    const float *x, *z; int64_t n;
    if (which == 3) { x = bp.hT + (int64_t)a * p.ldh; z = bp.yT + (int64_t)b * p.ldh; n = p.ldh; }
    else {
        x = (which == 2 ? bp.Rq : bp.Vr) + (int64_t)a * p.ldm;
        z = (which == 0 ? bp.Vr : bp.Rq) + (int64_t)b * p.ldm;
        n = p.ldm;
    }
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const float4* z4 = reinterpret_cast<const float4*>(z);
    float s0 = 0.f, s1 = 0.f;
    int64_t c = lane;
    for (; c + 32 < n / 4; c += 64) {
        const float4 xa = x4[c], zb = z4[c], xc = x4[c + 32], zd = z4[c + 32];
        s0 += xa.x * zb.x + xa.y * zb.y + xa.z * zb.z + xa.w * zb.w;
        s1 += xc.x * zd.x + xc.y * zd.y + xc.z * zd.z + xc.w * zd.w;
    }
    for (; c < n / 4; c += 32) {
        const float4 xa = x4[c], zb = z4[c];
        s0 += xa.x * zb.x + xa.y * zb.y + xa.z * zb.z + xa.w * zb.w;
    }
    s0 = warp_sum(s0 + s1);
    const int slot = which == 0 ? S_GV : which == 1 ? S_GX : which == 2 ? S_GR : B_HY;
    if (lane == 0) bp.small[(int64_t)slot * G * G + a * G + b] = (double)s0;
}

// C = op(A) * op(B) (G x G, fp64) with both operands staged in shared memory (2 G^2 doubles at `sm`).
__device__ void blk_mat_mul(const double* A, bool tA, const double* B, bool tB, double* C, int g, double* sm)
{
    const int gg = g * g;
    __syncthreads();
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) { sm[idx] = A[idx]; sm[gg + idx] = B[idx]; }
    __syncthreads();
    mat_mul(sm, tA, sm + gg, tB, C, g);
}

// One block: the G x G algebra of the exchange, its exact change of obj and the accept decision.
__global__ void __launch_bounds__(1024)
k_blk_small(Ptrs p, BlockPtrs bp, int accept_mode, double accept_tol, double* __restrict__ obj_trace, int32_t* __restrict__ swap_trace)
{
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ double red[32];
    extern __shared__ double smw[];          // 2 G^2 doubles: the matrix being factorised and its work array
    const int g = bp.G, gg = g * g;
    double* S = bp.small;
    double *Cinv = S + S_CINV * gg, *c1inv = S + S_C1INV * gg, *Q1 = S + S_Q1 * gg, *Q1c = S + S_Q1C * gg, *M2 = S + S_M2 * gg;
    double *GV = S + S_GV * gg, *GX = S + S_GX * gg, *GR = S + S_GR * gg, *C = S + S_C * gg, *P = S + S_P * gg;
    double *T1 = S + S_T1 * gg, *T2 = S + S_T2 * gg, *T3 = S + S_T3 * gg, *c1 = S + S_C1 * gg, *Lw = S + S_L * gg;
    double *cq = S + B_CQ * gg, *HY = S + B_HY * gg;
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        const int64_t ri = blk_rrow(p, bp, i), rj = blk_rrow(p, bp, j);
        const int64_t qi = p.nI + blk_qrow(p, bp, i), qj = p.nI + blk_qrow(p, bp, j);
        C[idx] = 0.5 * ((double)bp.PB[(int64_t)i * p.ldh + rj] + (double)bp.PB[(int64_t)j * p.ldh + ri]);
        P[idx] = (double)bp.yT[(int64_t)i * p.ldh + rj];                  // P[a][b] = y_a[r_b]
        cq[idx] = (double)p.Hp[qi * p.ldp + qj] - 0.5 * (HY[idx] + HY[j * g + i]);
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) smw[idx] = C[idx];
    __syncthreads();
    const double pivC = spd_inverse(smw, smw + gg, Cinv, g);
    const double Ds = mat_trace_prod(Cinv, GV, g, red);               // Tr(C^-1 V_r V_r^T)
    blk_mat_mul(Cinv, false, GX, false, T1, g, smw);                           // K R_q^T
    blk_mat_mul(P, false, T1, false, T2, g, smw);                              // P K R_q^T
    blk_mat_mul(P, false, Cinv, false, T1, g, smw);                            // P Cinv
    blk_mat_mul(T1, false, GV, false, T3, g, smw);                             // P Cinv GV
    blk_mat_mul(T3, false, T1, true, Lw, g, smw);                              // P Cinv GV Cinv P^T
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        T3[idx] = GR[idx] + T2[idx] + T2[j * g + i] + Lw[idx];        // R1 R1^T
    }
    __syncthreads();
    blk_mat_mul(T1, false, P, true, T2, g, smw);                               // P Cinv P^T
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        const int i = idx / g, j = idx % g;
        c1[idx] = cq[idx] + 0.5 * (T2[idx] + T2[j * g + i]);
    }
    __syncthreads();
    // the smallest pivot of c1 is compared with the diagonal of H on the entering rows (eligibility of the joint add)
    double scale = 0.0;
    {
        double hd = 0.0;
        for (int i = threadIdx.x; i < g; i += blockDim.x) {
            const int64_t qi = p.nI + blk_qrow(p, bp, i);
            hd = fmax(hd, (double)p.Hp[qi * p.ldp + qi]);
        }
        for (int o = 16; o > 0; o >>= 1) hd = fmax(hd, __shfl_xor_sync(0xffffffffu, hd, o));
        __syncthreads();
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = hd;
        __syncthreads();
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) scale = fmax(scale, red[i]);
        __syncthreads();
    }
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) smw[idx] = c1[idx];
    __syncthreads();
    const double pivc1 = spd_inverse(smw, smw + gg, c1inv, g);
    const double gain = mat_trace_prod(c1inv, T3, g, red);
    const double delta = Ds - gain;
    blk_mat_mul(Cinv, false, P, true, Q1, g, smw);                             // Q1 = Cinv P^T
    blk_mat_mul(Q1, false, c1inv, false, Q1c, g, smw);                         // Q1 c1inv
    blk_mat_mul(c1inv, false, T1, false, M2, g, smw);                          // c1inv P Cinv
    const double obj = ctl->obj;
    const int n = ctl->n_swaps;
    bool stop = false; int reason = 0;
    if (!(pivC > 0.0) || !(pivc1 > kAddPivotTol * scale) || !isfinite(delta)) { stop = true; reason = OSSCAR_STOP_GUARD; }
    else if (accept_mode == OSSCAR_ACCEPT_IMPROVING && !(delta <= -accept_tol * obj)) { stop = true; reason = OSSCAR_STOP_NO_IMPROVEMENT; }
    if (!stop) {
        for (int t = threadIdx.x; t < bp.s; t += blockDim.x) {
            swap_trace[2 * (n + t)] = p.perm[bp.rslot[t]];
            swap_trace[2 * (n + t) + 1] = p.perm[p.k + bp.tslot[t]];
        }
    }
    __syncthreads();                     // every thread has read obj and n_swaps
    if (threadIdx.x == 0) {
        ctl->delta = delta;
        if (stop) { ctl->done = 1; ctl->stop_reason = reason; *p.done_host = 1; }
        else {
            obj_trace[n / bp.s + 1] = obj + delta;
            ctl->obj = obj + delta;
            ctl->n_swaps = n + bp.s;
        }
    }
}

// Staged panels.  Part A (kept rows i): b C^-1, u2 = y - b Q1 (0 on r), -u2 c1^-1.  Part B (columns): K, Vq.
__global__ void __launch_bounds__(256) k_blk_prep(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G, gg = G * G;
    const double* S = bp.small;
    const double *Cinv = S + S_CINV * gg, *c1inv = S + S_C1INV * gg, *Q1 = S + S_Q1 * gg, *Q1c = S + S_Q1C * gg, *M2 = S + S_M2 * gg;
    const int64_t nA = p.ldh * G, nB = p.ldm * G;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < nA + nB; idx += (int64_t)gridDim.x * blockDim.x) {
        if (idx < nA) {
            const int e = (int)(idx / p.ldh); const int64_t i = idx % p.ldh;
            float vbc = 0.f, vu2 = 0.f, vnu = 0.f;
            if (i < p.nI) {
                double bc = 0.0, bq = 0.0, bqc = 0.0, yc = 0.0;
                for (int f = 0; f < G; ++f) {
                    const double bf = (double)bp.PB[(int64_t)f * p.ldh + i];
                    bc += bf * Cinv[f * G + e];
                    bq += bf * Q1[f * G + e];
                    bqc += bf * Q1c[f * G + e];
                    yc += (double)bp.yT[(int64_t)f * p.ldh + i] * c1inv[f * G + e];
                }
                vbc = (float)bc;                 // the entries of u2 on the leaving rows are cleared by k_blk_zero_r
                vu2 = (float)((double)bp.yT[(int64_t)e * p.ldh + i] - bq); vnu = (float)(bqc - yc);
            }
            bp.PA[(int64_t)e * p.ldh + i] = vbc;
            bp.PB[(int64_t)(G + e) * p.ldh + i] = vu2;
            bp.PA[(int64_t)(G + e) * p.ldh + i] = vnu;
            if (i < p.nI) {
                bp.PBT[i * 2 * G + e] = bp.PB[(int64_t)e * p.ldh + i];
                bp.PBT[i * 2 * G + G + e] = vu2;
                bp.PAT[i * 2 * G + e] = vbc;
                bp.PAT[i * 2 * G + G + e] = vnu;
            }
        } else {
            const int64_t j = idx - nA;
            const int e = (int)(j / p.ldm); const int64_t c = j % p.ldm;
            double kk = 0.0, vq = 0.0;
            for (int f = 0; f < G; ++f) {
                const double vr = (double)bp.Vr[(int64_t)f * p.ldm + c];
                const double rq = (double)bp.Rq[(int64_t)f * p.ldm + c];
                kk += Cinv[e * G + f] * vr;
                vq += c1inv[e * G + f] * rq + M2[e * G + f] * vr;
            }
            bp.KV[(int64_t)e * p.ldm + c] = (float)kk;
            bp.KV[(int64_t)(G + e) * p.ldm + c] = (float)vq;
        }
    }
}

// u2 vanishes on the leaving rows (y_r - C C^-1 y_r = 0): make the zeros exact, and put the block c1^-1 there in
// the -u2 c1^-1 panel.  G x G entries.
__global__ void __launch_bounds__(256) k_blk_zero_r(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= G * G) return;
    const int e = idx / G, a = idx % G;
    const int64_t i = blk_rrow(p, bp, a);
    const double* c1inv = bp.small + (int64_t)S_C1INV * G * G;
    bp.PB[(int64_t)(G + e) * p.ldh + i] = 0.f;
    // this row of PA doubles as the new rows / columns r of Hinv (k_blk_fix): -u2 c1^-1 off r, c1^-1 on r
    bp.PA[(int64_t)(G + e) * p.ldh + i] = (float)(0.5 * (c1inv[a * G + e] + c1inv[e * G + a]));
    bp.PBT[i * 2 * G + G + e] = 0.f;
    bp.PAT[i * 2 * G + G + e] = 0.f;
}

// H pass of the G leaving rows: UD[n_J + a][G + e] = Hp[r_a, 0:n_I] . u2_e, one warp per entry.
__global__ void __launch_bounds__(256) k_blk_leave_d(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (int64_t)G * G) return;
    const int a = (int)(wid / G), e = (int)(wid % G), lane = threadIdx.x & 31;
    const float4* x4 = reinterpret_cast<const float4*>(bp.HrT + (int64_t)a * p.ldh);
    const float4* z4 = reinterpret_cast<const float4*>(bp.PB + (int64_t)(G + e) * p.ldh);
    float s0 = 0.f, s1 = 0.f;
    int64_t c = lane;
    for (; c + 32 < p.ldh / 4; c += 64) {
        const float4 xa = x4[c], zb = z4[c], xc = x4[c + 32], zd = z4[c + 32];
        s0 += xa.x * zb.x + xa.y * zb.y + xa.z * zb.z + xa.w * zb.w;
        s1 += xc.x * zd.x + xc.y * zd.y + xc.z * zd.z + xc.w * zd.w;
    }
    for (; c < p.ldh / 4; c += 32) {
        const float4 xa = x4[c], zb = z4[c];
        s0 += xa.x * zb.x + xa.y * zb.y + xa.z * zb.z + xa.w * zb.w;
    }
    s0 = warp_sum(s0 + s1);
    if (lane == 0) bp.UD[(p.nJ + a) * 2 * G + G + e] = s0;
}

// After the H pass: UD[l][G+e] = Hp[l, I] u2_e  ->  -(d_l)_e = that - Hp[l, q_e]; the u part of a leaving row is e_l.
__global__ void __launch_bounds__(256) k_blk_finish_d(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G;
    const int64_t n = (p.nJ + G) * G;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t l = idx / G; const int e = (int)(idx % G);
        const int64_t row = l < p.nJ ? p.nI + l : blk_rrow(p, bp, (int)(l - p.nJ));
        float* ud = bp.UD + l * 2 * G;
        ud[G + e] -= p.Hp[row * p.ldp + p.nI + blk_qrow(p, bp, e)];
        if (l >= p.nJ) ud[e] = (l - p.nJ == e) ? 1.f : 0.f;
    }
}

// Rows and columns r of Hinv' = -u2 c1^-1 (block rr: c1^-1), rows r of V' = Vq, rows q of R' = the leaving rows'
// residual (staged in Rq).  One launch: blocks [0, G) per leaving row.
__global__ void __launch_bounds__(256) k_blk_fix(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    const int G = bp.G, t = blockIdx.x;
    const int64_t row = blk_rrow(p, bp, t), qrow = blk_qrow(p, bp, t);
    const float* nu = bp.PA + (int64_t)(G + t) * p.ldh;
    for (int64_t i = threadIdx.x; i < p.nI; i += blockDim.x) {       // on the leaving rows the panel holds c1^-1 (symmetric)
        const float v = nu[i];
        p.Hinv[i * p.ldh + row] = v;
        p.Hinv[row * p.ldh + i] = v;
    }
    const float* vq = bp.KV + (int64_t)(G + t) * p.ldm;
    const float* rn = bp.Rq + (int64_t)t * p.ldm;
    float sv = 0.f, sr = 0.f;
    for (int64_t c = threadIdx.x; c < p.m; c += blockDim.x) {
        const float a = vq[c], b = rn[c];
        p.V[row * p.ldm + c] = a;
        p.R[qrow * p.ldm + c] = b;
        sv = fmaf(a, a, sv); sr = fmaf(b, b, sr);
    }
    if (p.g == 1) {                      // single-row groups are scored from the row norms
        __shared__ float red[32];
        sv = block_sum_f(sv, red);
        sr = block_sum_f(sr, red);
        if (threadIdx.x == 0) { p.vnorm[row] = sv; p.rnorm[qrow] = sr; }
    }
}

// c_l' = c_l + u_l C^-1 u_l^T - d_l c1^-1 d_l^T for every pruned slot; an entering slot receives the leaving group
// (old c = 0, u_l = unit rows).  One block per pruned slot; dynamic shared memory 2 g G doubles.
__global__ void __launch_bounds__(128) k_blk_update_c(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    extern __shared__ double smc[];
    const int g = p.g, G = bp.G;
    double* TU = smc; double* TD = smc + g * G;
    const int64_t t = blockIdx.x;
    int pos = -1;
    for (int a = 0; a < bp.s; ++a) if (bp.tslot[a] == t) pos = a;
    const int64_t base = pos >= 0 ? p.nJ + (int64_t)pos * g : t * g;
    const double* Cinv = bp.small + (int64_t)S_CINV * G * G;
    const double* c1inv = bp.small + (int64_t)S_C1INV * G * G;
    const float* ud = bp.UD + base * 2 * G;
    for (int idx = threadIdx.x; idx < g * G; idx += blockDim.x) {
        const int a = idx / G, f = idx % G;
        double tu = 0.0, td = 0.0;
        for (int e = 0; e < G; ++e) {
            tu += (double)ud[a * 2 * G + e] * Cinv[e * G + f];
            td += (double)ud[a * 2 * G + G + e] * c1inv[e * G + f];
        }
        TU[idx] = tu; TD[idx] = td;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < g * g; idx += blockDim.x) {
        const int a = idx / g, b2 = idx % g;
        double s = pos >= 0 ? 0.0 : p.c[t * g * g + idx];
        for (int f = 0; f < G; ++f)
            s += TU[a * G + f] * (double)ud[b2 * 2 * G + f] - TD[a * G + f] * (double)ud[b2 * 2 * G + G + f];
        p.c[t * g * g + idx] = s;
    }
}

// Single-row groups: c_l' = c_l + u_l C^-1 u_l^T - d_l c1^-1 d_l^T, one warp per four pruned rows; C^-1 and c1^-1
// sit in shared memory as fp32 (u and d are fp32 values already) and the sums run in fp32, the update of c in fp64.
__global__ void __launch_bounds__(256) k_blk_update_c_g1(Ptrs p, BlockPtrs bp)
{
    if (p.ctl->done) return;
    extern __shared__ float smf[];
    const int G = bp.G, gg = G * G;
    float* Ci = smf; float* c1i = smf + gg;
    for (int idx = threadIdx.x; idx < gg; idx += blockDim.x) {
        Ci[idx] = (float)bp.small[(int64_t)S_CINV * gg + idx];
        c1i[idx] = (float)bp.small[(int64_t)S_C1INV * gg + idx];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t nw = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t t0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 4; t0 < p.nJ; t0 += nw * 4) {
        const float* ud[4]; bool enter[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int64_t t = t0 + r < p.nJ ? t0 + r : p.nJ - 1;
            int pos = -1;
            for (int a = 0; a < bp.s; ++a) if (bp.tslot[a] == t) pos = a;
            enter[r] = pos >= 0;
            ud[r] = bp.UD + (pos >= 0 ? p.nJ + pos : t) * 2 * G;
        }
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        for (int e = lane; e < G; e += 32) {
            float tu[4] = {0.f, 0.f, 0.f, 0.f}, td[4] = {0.f, 0.f, 0.f, 0.f};
            for (int f = 0; f < G; ++f) {
                const float ci = Ci[f * G + e], c1 = c1i[f * G + e];
#pragma unroll
                for (int r = 0; r < 4; ++r) { tu[r] = fmaf(ud[r][f], ci, tu[r]); td[r] = fmaf(ud[r][G + f], c1, td[r]); }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) s[r] += tu[r] * ud[r][e] - td[r] * ud[r][G + e];
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const float v = warp_sum(s[r]);
            if (lane == 0 && t0 + r < p.nJ) p.c[t0 + r] = (enter[r] ? 0.0 : p.c[t0 + r]) + (double)v;
        }
    }
}

// Exchange the rows (phase 0) or columns (phase 1) of Hp of every leaving / entering pair; phase 1 also exchanges
// the groups in the slot permutation.  Phase 0: grid (pieces of a row, G), a block moves 256 consecutive floats of the
// two rows of one pair.  Phase 1: a warp owns one row of Hp and its lanes take the pairs, so that the 2 G scattered
// floats a warp touches lie in one row of the matrix (one DRAM page neighbourhood) instead of in 32 rows.
__global__ void __launch_bounds__(256) k_blk_hswap(Ptrs p, BlockPtrs bp, int phase)
{
    if (p.ctl->done) return;
    const int G = bp.G;
    if (phase == 0) {
        const int e = blockIdx.y;
        const int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        if (x < p.ldp) {
            float* pa = p.Hp + blk_rrow(p, bp, e) * p.ldp + x;
            float* pb = p.Hp + (p.nI + blk_qrow(p, bp, e)) * p.ldp + x;
            const float va = *pa, vb = *pb;
            *pa = vb; *pb = va;
        }
    } else {
        __shared__ int32_t sa[OSSCAR_MAX_GROUP], sb[OSSCAR_MAX_GROUP];
        for (int e = threadIdx.x; e < G; e += blockDim.x) { sa[e] = (int32_t)blk_rrow(p, bp, e); sb[e] = (int32_t)(p.nI + blk_qrow(p, bp, e)); }
        __syncthreads();
        const int lane = threadIdx.x & 31;
        const int64_t x = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
        if (x < p.nI + p.nJ) {
            float* row = p.Hp + x * p.ldp;
            for (int e = lane; e < G; e += 32) {
                const float va = row[sa[e]], vb = row[sb[e]];
                row[sa[e]] = vb; row[sb[e]] = va;
            }
        }
    }
    if (phase == 1 && blockIdx.x == 0 && threadIdx.x == 0) {
        for (int t = 0; t < bp.s; ++t) {
            const int s = bp.rslot[t], u = p.k + bp.tslot[t];
            const int gi = p.perm[s], gj = p.perm[u];
            p.perm[s] = gj; p.perm[u] = gi;
            p.slotof[gj] = s; p.slotof[gi] = u;
        }
    }
}

// One iteration of the block exchange on the stream; `mark` records an event after each stage when profiling.
template <class Mark>
cudaError_t enqueue_block_step(osscar_ctx* ctx, const Ptrs& p, const BlockPtrs& bp, int accept_mode, double tol,
                               double* obj_trace, int32_t* swap_trace, Mark&& mark)
{
    const Layout& L = ctx->L;
    cudaStream_t st = ctx->stream;
    const int G = bp.G;
    const int32_t* done = &ctx->ctl->done;
    cudaError_t e;
#define BK(x) do { e = (x); if (e != cudaSuccess) return e; } while (0)
    k_blk_select<<<2, 1024, 0, st>>>(p, bp);                                                    mark();
    k_blk_gather<<<dim3((unsigned)G, 5), 256, 0, st>>>(p, bp);
    void* tc = (char*)ctx->ws + L.off_tc;                       // free between state builds: bf16 terms and partial sums
    SearchCtl* stat = ctx->ctl;
    BK(panel_dot_tc(st, L.nI, G, L.nI, p.Hinv, L.ldh, bp.hT, L.ldh, bp.yT, 1, L.ldh, tc, L.tc_bytes, stat, done));     mark();   // y^T (Hinv symmetric)
    k_blk_gram<<<(unsigned)((4 * G * G + 7) / 8), 256, 0, st>>>(p, bp);
    k_blk_small<<<1, 1024, 2 * (size_t)G * G * sizeof(double), st>>>(p, bp, accept_mode, tol, obj_trace, swap_trace);
    k_blk_prep<<<(unsigned)(((L.ldh + L.ldm) * G + 255) / 256), 256, 0, st>>>(p, bp);
    k_blk_zero_r<<<(unsigned)((G * G + 255) / 256), 256, 0, st>>>(p, bp);                        mark();
    // H pass: [u | H u2] for the pruned rows and the leaving rows, then -d
    BK(panel_dot_tc(st, L.nJ, 2 * G, L.nI, p.Hp + L.nI * L.ldp, L.ldp, bp.PB, L.ldh, bp.UD, 2 * G, 1, tc, L.tc_bytes, stat, done));
    k_blk_leave_d<<<(unsigned)((G * G + 7) / 8), 256, 0, st>>>(p, bp);
    k_blk_finish_d<<<(unsigned)(((L.nJ + G) * G + 255) / 256), 256, 0, st>>>(p, bp);            mark();
    // the three rank-2G updates; the residual rows of the leaving groups go through the Rq panel
    BK(rank_update_tc(st, L.nI, L.ldh, 2 * G, -1.f, bp.PAT, 2 * G, bp.PB, L.ldh, p.Hinv, L.ldh, tc, L.tc_bytes, stat, done));   mark();
    // single-row groups: the squared row norms of V' and R' (the next scores) come out of the update passes
    float* sq = (float*)((char*)tc + (L.tc_bytes / 2 / 1024) * 1024);
    const size_t sq_floats = (L.tc_bytes - (L.tc_bytes / 2 / 1024) * 1024) / sizeof(float);
    const int64_t nseg = 2 * ((L.ldm + 127) / 128);
    const bool fused_norms = L.g == 1 && 2 * G <= 128 && (size_t)((L.nJ > L.nI ? L.nJ : L.nI) * nseg) <= sq_floats;
    BK(rank_update_tc(st, L.nI, L.ldm, 2 * G, -1.f, bp.PBT, 2 * G, bp.KV, L.ldm, p.V, L.ldm, tc, L.tc_bytes / 2, stat, done,
                      fused_norms ? p.vnorm : nullptr, sq));                                                              mark();
    BK(rank_update_tc(st, L.nJ, L.ldm, 2 * G, 1.f, bp.UD, 2 * G, bp.KV, L.ldm, p.R, L.ldm, tc, L.tc_bytes / 2, stat, done,
                      fused_norms ? p.rnorm : nullptr, sq));
    BK(sgemm(st, false, false, G, L.m, 2 * G, 1.f, bp.UD + L.nJ * 2 * G, 2 * G, bp.KV, L.ldm, 0.f, bp.Rq, L.ldm, done));   mark();
    if (L.g == 1) k_blk_update_c_g1<<<296, 256, 2 * (size_t)G * G * sizeof(float), st>>>(p, bp);
    else k_blk_update_c<<<(unsigned)(L.ng - L.k), 128, 2 * (size_t)L.g * G * sizeof(double), st>>>(p, bp);
    k_blk_fix<<<(unsigned)G, 256, 0, st>>>(p, bp);                                              mark();
    k_blk_hswap<<<dim3((unsigned)((L.ldp + 255) / 256), (unsigned)G), 256, 0, st>>>(p, bp, 0);
    k_blk_hswap<<<(unsigned)((L.d1 + 7) / 8), 256, 0, st>>>(p, bp, 1);                           mark();
    count_launches(12);
    BK(enqueue_scores(ctx, p, !fused_norms, false));                                           mark();
#undef BK
    return cudaGetLastError();
}
