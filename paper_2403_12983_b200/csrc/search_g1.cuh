// Swap step for single-row groups (g = 1): five launches per swap, each matrix streamed once.
// Included by search.cu (same translation unit: uses its Ptrs, reductions and small-matrix slots).
//
//   decide      one block: i* = argmin D, exact change of obj, accept test, staged vectors b, u2, K, Vq
//   L1          H pass (u_l, d_l for every pruned row and the leaving row)  ||  V update + drop scores D
//   L2          R update + Schur complements + add scores A                 ||  slot exchange in Hp
//   select_in   q* = argmax A for the NEXT step
//   L4          Hinv update fused with y_next = Hinv' * Hp[q_next, 0:n_I]^T (the next step's y pass)
//
// Scalars of a step live in p.small (doubles): [S_CINV] = 1/C, [S_C1INV] = 1/c1, [G1_Q1] = P/C,
// [G1_M2] = P/(C c1), [G1_HDIAG] = H diagonal entry of the leaving row.
#pragma once

constexpr int G1_Q1 = 2, G1_M2 = 3, G1_HDIAG = 4;

__device__ __forceinline__ void fma4(float4& v, float a, const float4& x) {
    v.x = fmaf(a, x.x, v.x); v.y = fmaf(a, x.y, v.y); v.z = fmaf(a, x.z, v.z); v.w = fmaf(a, x.w, v.w);
}
__device__ __forceinline__ float dot4(const float4& a, const float4& b) {
    return a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
}

// D[s] = ||V_s||^2 / Hinv_ss and A[t] = ||R_t||^2 / c_t from the row norms (start of a search / after a refresh).
__global__ void k_scores_g1(Ptrs p)
{
    if (p.ctl->done) return;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.nI) {
        const double hd = p.Hd[i * p.ldh + i];
        p.D[i] = hd > 0.0 ? (double)p.vnorm[i] / hd : INFINITY;
    } else if (i < p.nI + p.nJ) {
        const int64_t t = i - p.nI;
        const double cc = p.c[t];
        const double hd = p.Hp[(p.nI + t) * p.ldp + p.nI + t];
        p.A[t] = cc > kAddPivotTol * hd ? (double)p.rnorm[t] / cc : -INFINITY;
    }
}

// Column shards: after the row norms of V' and R' have been summed over shards, the scores of the new state.  The
// inverse has not been updated yet (that pass needs the next entering group, which these scores decide), so its new
// diagonal comes from the rank-two formula, as in the row update's own epilogue.
__global__ void k_scores_sharded_g1(Ptrs p)
{
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const double Cinv = p.small[S_CINV], c1inv = p.small[S_C1INV];
    if (i < p.nI) {
        const double bs = p.b[i], us = p.u2[i];
        const double hd = i == p.ctl->sel_slot ? c1inv : p.Hd[i * p.ldh + i] - bs * bs * Cinv + us * us * c1inv;
        p.D[i] = hd > 0.0 ? (double)p.vnorm[i] / hd : INFINITY;
    } else if (i < p.nI + p.nJ) {
        const int64_t t = i - p.nI;
        const double cc = p.c[t];
        const double hd = p.Hp[(p.nI + t) * p.ldp + p.nI + t];
        p.A[t] = cc > kAddPivotTol * hd ? (double)p.rnorm[t] / cc : -INFINITY;
    }
}

// Block-wide arg-min of val[i] (ties -> smaller group id); result broadcast through shared memory.
__device__ void block_argmin(const double* val, const int32_t* ids, int n, bool negate,
                             double* best_out, int* idx_out)
{
    __shared__ double sv[32]; __shared__ int sid[32]; __shared__ int sidx[32];
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    double best = INFINITY; int bid = INT_MAX, bidx = -1;
    for (int i0 = t; i0 < n; i0 += 4 * blockDim.x) {          // four independent loads in flight per thread
        double vv[4]; int ii[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = i0 + j * blockDim.x;
            vv[j] = i < n ? val[i] : (negate ? -INFINITY : INFINITY);
            ii[j] = i < n ? ids[i] : INT_MAX;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = i0 + j * blockDim.x;
            const double v = negate ? -vv[j] : vv[j];
            if (i < n && (v < best || (v == best && ii[j] < bid))) { best = v; bid = ii[j]; bidx = i; }
        }
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
        sv[0] = best; sidx[0] = bidx;
    }
    __syncthreads();
    *best_out = negate ? -sv[0] : sv[0];
    *idx_out = sidx[0];
    __syncthreads();
}

// q* = argmax A (the group that enters at the next step).
__global__ void __launch_bounds__(1024) k_select_in_g1(Ptrs p)
{
    pdl_wait_then_release();
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    double best; int idx;
    block_argmin(p.A, p.perm + p.k, (int)p.nJ, true, &best, &idx);
    if (threadIdx.x == 0) {
        ctl->sel_t = idx;
        if (idx < 0 || !isfinite(best)) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
    }
}

// One block: leaving row, exact change of obj, accept test, traces, staged vectors.
// part 0: the whole decision; column shards run it in two parts around the sum of the cross term over shards:
// part 1 picks the leaving row and leaves this shard's V_r . R_q in p.shard[0], part 2 continues from the summed value.
__global__ void __launch_bounds__(1024)
k_decide_g1(Ptrs p, int accept_mode, double accept_tol, double* __restrict__ obj_trace, int32_t* __restrict__ swap_trace, int part)
{
    pdl_wait_then_release();
    SearchCtl* ctl = p.ctl;
    if (ctl->done) return;
    __shared__ float redf[32];
    __shared__ int s_stop;
    double Dbest = 0.0; int slot;
    if (part == 2) slot = ctl->sel_slot;
    else {
        block_argmin(p.D, p.perm, p.k, false, &Dbest, &slot);
        if (slot < 0 || !isfinite(Dbest)) {
            if (threadIdx.x == 0) { ctl->done = 1; ctl->stop_reason = OSSCAR_STOP_GUARD; *p.done_host = 1; }
            return;
        }
    }
    const int64_t t = ctl->sel_t;
    const int64_t r0 = slot;
    double GX;
    if (part == 2) GX = p.shard[0];
    else {          // cross term V_r . R_q
        const float4* vr = reinterpret_cast<const float4*>(p.V + r0 * p.ldm);
        const float4* rq = reinterpret_cast<const float4*>(p.R + t * p.ldm);
        float acc = 0.f;
        for (int64_t c = threadIdx.x; c < p.ldm / 4; c += blockDim.x) acc += dot4(vr[c], rq[c]);
        GX = (double)block_sum_f(acc, redf);
    }
    if (part == 1) {
        if (threadIdx.x == 0) { ctl->sel_slot = slot; p.shard[0] = GX; }
        return;
    }
    if (threadIdx.x == 0) {
        const double C = p.Hd[r0 * p.ldh + r0], P = p.y[r0], cq = p.c[t];
        const double GV = p.vnorm[r0], GR = p.rnorm[t];
        const double Cinv = 1.0 / C;
        const double Ds = GV * Cinv;
        const double RR1 = GR + 2.0 * P * Cinv * GX + P * P * Cinv * Cinv * GV;
        const double c1 = cq + P * P * Cinv;
        const double c1inv = 1.0 / c1;
        const double delta = Ds - c1inv * RR1;
        const double obj = ctl->obj;
        bool stop = false; int reason = 0;
        if (!(C > 0.0) || !(c1 > 0.0) || !isfinite(delta)) { stop = true; reason = OSSCAR_STOP_GUARD; }
        else if (accept_mode == OSSCAR_ACCEPT_IMPROVING && !(delta <= -accept_tol * obj)) { stop = true; reason = OSSCAR_STOP_NO_IMPROVEMENT; }
        ctl->delta = delta; ctl->sel_D = Ds; ctl->sel_slot = slot;
        if (stop) { ctl->done = 1; ctl->stop_reason = reason; *p.done_host = 1; }
        else {
            const int n = ctl->n_swaps;
            swap_trace[2 * n] = p.perm[slot];
            swap_trace[2 * n + 1] = p.perm[p.k + t];
            obj_trace[n + 1] = obj + delta;
            ctl->obj = obj + delta;
            ctl->n_swaps = n + 1;
            p.small[S_CINV] = Cinv; p.small[S_C1INV] = c1inv;
            p.small[G1_Q1] = Cinv * P; p.small[G1_M2] = c1inv * P * Cinv;
            p.small[G1_HDIAG] = p.Hp[r0 * p.ldp + r0];
        }
        s_stop = stop;
    }
    __syncthreads();
    if (s_stop) return;
    const float Q1 = (float)p.small[G1_Q1];
    const double Cinv = p.small[S_CINV], c1inv = p.small[S_C1INV], M2 = p.small[G1_M2];
    // float4 wide (pads of Hinv rows, y, V, R are zero, so the padded tails stay zero); the inverse is kept in fp64
    const double2* hrow2 = reinterpret_cast<const double2*>(p.Hd + r0 * p.ldh);
    const float4* y4 = reinterpret_cast<const float4*>(p.y);
    float4* b4 = reinterpret_cast<float4*>(p.b);
    float4* u4 = reinterpret_cast<float4*>(p.u2);
    for (int64_t c = threadIdx.x; c < p.ldh / 4; c += blockDim.x) {
        const double2 h0 = hrow2[2 * c], h1 = hrow2[2 * c + 1];
        const float4 bs = make_float4((float)h0.x, (float)h0.y, (float)h1.x, (float)h1.y), yy = y4[c];
        float4 uu = make_float4(fmaf(-bs.x, Q1, yy.x), fmaf(-bs.y, Q1, yy.y), fmaf(-bs.z, Q1, yy.z), fmaf(-bs.w, Q1, yy.w));
        const int64_t rc = r0 - c * 4;
        uu.x = rc == 0 ? 0.f : uu.x; uu.y = rc == 1 ? 0.f : uu.y; uu.z = rc == 2 ? 0.f : uu.z; uu.w = rc == 3 ? 0.f : uu.w;
        b4[c] = bs;
        u4[c] = uu;
    }
    const float4* v4 = reinterpret_cast<const float4*>(p.V + r0 * p.ldm);
    const float4* r4 = reinterpret_cast<const float4*>(p.R + t * p.ldm);
    float4* k4 = reinterpret_cast<float4*>(p.K);
    float4* q4 = reinterpret_cast<float4*>(p.Vq);
    const float fC = (float)Cinv, fc1 = (float)c1inv, fM2 = (float)M2;
    for (int64_t c = threadIdx.x; c < p.ldm / 4; c += blockDim.x) {
        const float4 v = v4[c], r = r4[c];
        k4[c] = make_float4(fC * v.x, fC * v.y, fC * v.z, fC * v.w);
        q4[c] = make_float4(fmaf(fc1, r.x, fM2 * v.x), fmaf(fc1, r.y, fM2 * v.y), fmaf(fc1, r.z, fM2 * v.z), fmaf(fc1, r.w, fM2 * v.w));
    }
}

// Streaming layout of the three big kernels: a block of 256 threads owns whole rows, every thread requests its (up to)
// eight or nine 16-byte pieces of a row at once, one block-wide reduction per row at the end.  Measured on the R update
// shape (20070 x 7168): 6.7 TB/s for a row per block against 5.7 TB/s for a warp per row and 6.0 TB/s for a plain copy.
// Two rows per block halve the L2 reads of the step's vectors: measured at the OPT-30B FC2 shape that pays for the Hinv
// update with its three vectors (0.122 -> 0.115 ms) and costs the V / R updates and the H pass 12-17 % (half as many
// resident blocks), so G1_RB = 1 there and G1_RB4 = 2 for the Hinv update.
constexpr int G1_U = 8;
constexpr int G1_UH = 9;            // pieces per thread for rows of Hinv / Hp: 9 x 256 x 4 floats cover n_I = 8602 in one pass
constexpr int G1_T = 256;           // most threads per block; rows of up to 512 / 1024 pieces run with 64 / 128 threads, so that
                                    // a thread still requests about eight pieces and twice or four times as many rows are in flight per SM
__host__ __device__ inline int g1_threads(int64_t pieces) { return pieces <= 512 ? 64 : (pieces <= 1024 ? 128 : 256); }

// Block-wide sum for blocks of 64, 128 or 256 threads (the launch picks the size by the row length).
template <int TB>
__device__ __forceinline__ float block_sum_256(float v, float* red /*[8]*/)
{
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < TB / 32; ++i) t += red[i];
    __syncthreads();
    return t;
}

// Row update M'[s] = M[s] + ck_s K + cq_s Vq with the squared norm of the new row, RB rows per block (every piece of
// K and Vq fetched from L2 serves the RB rows).  kind 0: V (ck = -b_s, cq = -u2_s, row r0 := Vq, D' written),
// kind 1: R (ck = u_l, cq = -d_l, row of the entering slot := K - d_r Vq, c' and A' written).
template <int RB, int TB>
__device__ __forceinline__ void update_row_g1(const Ptrs& p, int kind, int64_t s0, float* red)
{
    float* M = kind == 0 ? p.V : p.R;
    const int64_t nrows = kind == 0 ? p.nI : p.nJ;
    const int64_t n4 = p.ldm / 4;
    const float4* K4 = reinterpret_cast<const float4*>(p.K);
    const float4* Q4 = reinterpret_cast<const float4*>(p.Vq);
    float4* row[RB];
    int64_t srow[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        srow[r] = s0 + r < nrows ? s0 + r : nrows - 1;
        row[r] = reinterpret_cast<float4*>(M + srow[r] * p.ldm);
    }
    float nrm[RB], ck[RB], cq[RB];
    bool sp[RB];
    float dr = 0.f;
#pragma unroll
    for (int r = 0; r < RB; ++r) { nrm[r] = 0.f; ck[r] = 0.f; cq[r] = 0.f; sp[r] = false; }
    for (int64_t base = threadIdx.x; base < n4; base += (int64_t)TB * G1_U) {
        float4 v[RB][G1_U];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int j = 0; j < G1_U; ++j) {
                const int64_t c = base + TB * j;
                v[r][j] = c < n4 ? row[r][c] : make_float4(0.f, 0.f, 0.f, 0.f);     // requested before the step's scalars arrive
            }
        if (base == threadIdx.x) {           // first pass: the scalars of these rows, loaded behind the rows themselves
            pdl_wait_then_release();
            if (p.ctl->done) return;             // a stopped loop only read; nothing is written
            const int64_t special = kind == 0 ? (int64_t)p.ctl->sel_slot : (int64_t)p.ctl->sel_t;
            if (kind == 1) dr = p.d[p.nJ];
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                const int64_t s = srow[r];
                sp[r] = s == special;
                if (kind == 0) { ck[r] = -p.b[s]; cq[r] = -p.u2[s]; }
                else { ck[r] = p.u[s]; cq[r] = -p.d[s]; }
                if (sp[r]) { ck[r] = kind == 0 ? 0.f : 1.f; cq[r] = kind == 0 ? 1.f : -dr; }      // new row = ck K + cq Vq
            }
        }
#pragma unroll
        for (int j = 0; j < G1_U; ++j) {
            const int64_t c = base + TB * j;
            if (c < n4) {
                const float4 kk = K4[c], qq = Q4[c];
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    if (sp[r]) v[r][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    fma4(v[r][j], ck[r], kk);
                    fma4(v[r][j], cq[r], qq);
                    if (s0 + r < nrows) row[r][c] = v[r][j];
                    nrm[r] += dot4(v[r][j], v[r][j]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        const float nr = block_sum_256<TB>(nrm[r], red);
        if (threadIdx.x == 0 && s0 + r < nrows) {
            const int64_t s = s0 + r;
            const double Cinv = p.small[S_CINV], c1inv = p.small[S_C1INV];
            if (kind == 0) {
                p.vnorm[s] = nr;
                double hd;
                if (sp[r]) hd = c1inv;
                else {
                    const double bs = p.b[s], us = p.u2[s];
                    hd = p.Hd[s * p.ldh + s] - bs * bs * Cinv + us * us * c1inv;
                }
                p.D[s] = hd > 0.0 ? (double)nr / hd : INFINITY;
            } else {
                p.rnorm[s] = nr;
                double cc, hd;
                if (sp[r]) { cc = Cinv - (double)dr * (double)dr * c1inv; hd = p.small[G1_HDIAG]; }
                else {
                    const double uu = p.u[s], dd = p.d[s];
                    cc = p.c[s] + uu * uu * Cinv - dd * dd * c1inv;
                    hd = p.Hp[(p.nI + s) * p.ldp + p.nI + s];
                }
                p.c[s] = cc;
                p.A[s] = cc > kAddPivotTol * hd ? (double)nr / cc : -INFINITY;
            }
        }
    }
}

// u_l = Hp[l, 0:n_I] . b and d_l = Hp[l, q] - Hp[l, 0:n_I] . u2 for RB rows (pruned rows l0.., or the single leaving
// row, l = n_J); every piece of b and u2 serves the RB rows.
template <int RB, int TB>
__device__ __forceinline__ void hpass_stream(const Ptrs& p, const float4* const (&row)[RB], int64_t l0, int nvalid, float* red /*[16]*/)
{
    const float4* bv = reinterpret_cast<const float4*>(p.b);
    const float4* uv = reinterpret_cast<const float4*>(p.u2);
    const int64_t n4 = p.ldh / 4;
    float au[RB], ad[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) { au[r] = 0.f; ad[r] = 0.f; }
    for (int64_t base = threadIdx.x; base < n4; base += (int64_t)TB * G1_UH) {
        float4 x[RB][G1_UH];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int j = 0; j < G1_UH; ++j) {
                const int64_t c = base + TB * j;
                x[r][j] = c < n4 ? row[r][c] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        if (base == threadIdx.x) pdl_wait_then_release();          // b and u2 come from the kernel before this one
#pragma unroll
        for (int j = 0; j < G1_UH; ++j) {
            const int64_t c = base + TB * j;
            if (c < n4) {
                const float4 bb = bv[c], uu = uv[c];
#pragma unroll
                for (int r = 0; r < RB; ++r) { au[r] += dot4(x[r][j], bb); ad[r] += dot4(x[r][j], uu); }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        const float a = warp_sum(au[r]), d = warp_sum(ad[r]);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = a; red[8 + (threadIdx.x >> 5)] = d; }
        __syncthreads();
        if (threadIdx.x == 0 && r < nvalid && !p.ctl->done) {
            float su = 0.f, sd = 0.f;
#pragma unroll
            for (int i = 0; i < TB / 32; ++i) { su += red[i]; sd += red[8 + i]; }
            const int64_t qcol = p.nI + (int64_t)p.ctl->sel_t;
            p.u[l0 + r] = su;
            p.d[l0 + r] = reinterpret_cast<const float*>(row[r])[qcol] - sd;
        }
    }
}

// L1: blocks [0, nbV) update G1_RB rows of V each; then one block per G1_RB pruned rows of the H pass (their addresses
// need no control-block read, so their streams start at once) and a last block for the leaving row.
constexpr int G1_RB = 1;            // rows per block of the V / R updates and the H pass
constexpr int G1_RB4 = 1;           // rows per block of the Hinv update
template <int TB>
__global__ void __launch_bounds__(TB, 1024 / TB) k_l1_g1(Ptrs p, unsigned nbV)      // 64 registers: four resident blocks per SM
{
    __shared__ float red[16];
    if (blockIdx.x < nbV) { update_row_g1<G1_RB, TB>(p, 0, (int64_t)blockIdx.x * G1_RB, red); return; }
    const int64_t l0 = (int64_t)(blockIdx.x - nbV) * G1_RB;
    if (l0 < p.nJ) {
        const float4* rows[G1_RB];
        int nvalid = 0;
#pragma unroll
        for (int r = 0; r < G1_RB; ++r) {
            const int64_t l = l0 + r < p.nJ ? l0 + r : p.nJ - 1;
            rows[r] = reinterpret_cast<const float4*>(p.Hp + (p.nI + l) * p.ldp);
            nvalid += l0 + r < p.nJ;
        }
        hpass_stream<G1_RB, TB>(p, rows, l0, nvalid, red);
    } else {
        pdl_wait_then_release();             // the leaving row is named by the control block
        const float4* rows[1] = { reinterpret_cast<const float4*>(p.Hp + (int64_t)p.ctl->sel_slot * p.ldp) };
        hpass_stream<1, TB>(p, rows, p.nJ, 1, red);
    }
}

// Exchange of the leaving kept slot a and the entering pruned slot b in Hp (rows and columns) and in the
// slot permutation.  Work item ranges: [0, ldp) the two rows, [ldp, 2 ldp) the two columns.
__device__ __forceinline__ void hswap_g1_at(const Ptrs& p, const int64_t a, const int64_t b, int64_t idx, int64_t stride)
{
    const int64_t d1 = p.nI + p.nJ;
    for (; idx < 2 * p.ldp; idx += stride) {
        if (idx < p.ldp) {
            const int64_t x = idx;
            if (x == a) {           // the 2 x 2 intersection, one thread: new[a][a]=old[b][b], new[a][b]=old[b][a], ...
                const float aa = p.Hp[a * p.ldp + a], ab = p.Hp[a * p.ldp + b], ba = p.Hp[b * p.ldp + a], bb = p.Hp[b * p.ldp + b];
                p.Hp[a * p.ldp + a] = bb; p.Hp[a * p.ldp + b] = ba; p.Hp[b * p.ldp + a] = ab; p.Hp[b * p.ldp + b] = aa;
            } else if (x != b) {
                const float va = p.Hp[a * p.ldp + x], vb = p.Hp[b * p.ldp + x];
                p.Hp[a * p.ldp + x] = vb; p.Hp[b * p.ldp + x] = va;
            }
        } else {
            const int64_t x = idx - p.ldp;
            if (x < d1 && x != a && x != b) {
                const float va = p.Hp[x * p.ldp + a], vb = p.Hp[x * p.ldp + b];
                p.Hp[x * p.ldp + a] = vb; p.Hp[x * p.ldp + b] = va;
            }
        }
    }
}

__device__ __forceinline__ void hswap_g1(const Ptrs& p, int64_t idx, int64_t stride)
{
    hswap_g1_at(p, p.ctl->sel_slot, p.nI + (int64_t)p.ctl->sel_t, idx, stride);
}

// L2: blocks [0, nbR) update G1_RB rows of R each (+ c, A); the remaining blocks exchange the two slots in Hp.
template <int TB>
__global__ void __launch_bounds__(TB, 1024 / TB) k_l2_g1(Ptrs p, unsigned nbR)
{
    __shared__ float red[8];
    if (blockIdx.x < nbR) { update_row_g1<G1_RB, TB>(p, 1, (int64_t)blockIdx.x * G1_RB, red); return; }
    pdl_wait_then_release();
    if (p.ctl->done) return;
    const int64_t nsw = gridDim.x - nbR;
    hswap_g1(p, (int64_t)(blockIdx.x - nbR) * blockDim.x + threadIdx.x, nsw * blockDim.x);
    if (blockIdx.x == nbR && threadIdx.x == 0) {
        const int s = p.ctl->sel_slot, t = p.k + p.ctl->sel_t;
        const int gi = p.perm[s], gj = p.perm[t];
        p.perm[s] = gj; p.perm[t] = gi;
        p.slotof[gj] = s; p.slotof[gi] = t;
    }
}

// L4: Hinv' = Hinv - (b/C) b^T + (u2/c1) u2^T (row and column r0: -u2/c1, corner 1/c1) on the fp64 copy of the inverse and,
// in the same pass, y_next = Hinv' h with h = Hp[row of the next entering group, 0:n_I].  RB rows per block; a piece is a
// double2, nine pieces per thread and pass.
template <int RB, int TB>
__global__ void __launch_bounds__(TB) k_l4_g1(Ptrs p)
{
    __shared__ double red[8];
    const int64_t s0 = (int64_t)blockIdx.x * RB;
    const float2* b2 = reinterpret_cast<const float2*>(p.b);
    const float2* u2v = reinterpret_cast<const float2*>(p.u2);
    const int64_t n2 = p.ldh / 2;
    double2* row[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) row[r] = reinterpret_cast<double2*>(p.Hd + (s0 + r < p.nI ? s0 + r : p.nI - 1) * p.ldh);
    int64_t r0 = 0;
    const float2* h2 = nullptr;
    bool srow[RB];
    double nb[RB], us[RB], corner[RB], yacc[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) { srow[r] = false; nb[r] = 0.0; us[r] = 0.0; corner[r] = 0.0; yacc[r] = 0.0; }
    for (int64_t base = threadIdx.x; base < n2; base += (int64_t)TB * G1_UH) {
        double2 h[RB][G1_UH];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int j = 0; j < G1_UH; ++j) {
                const int64_t c = base + TB * j;
                h[r][j] = c < n2 ? row[r][c] : make_double2(0.0, 0.0);    // requested before the step's scalars arrive
            }
        if (base == threadIdx.x) {
            pdl_wait_then_release();
            if (p.ctl->done) return;
            r0 = p.ctl->sel_slot;
            const double Cinv = p.small[S_CINV], c1inv = p.small[S_C1INV];
            h2 = reinterpret_cast<const float2*>(p.Hp + (p.nI + (int64_t)p.ctl->sel_t) * p.ldp);
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                const int64_t s = s0 + r < p.nI ? s0 + r : p.nI - 1;
                srow[r] = s == r0;
                // row r0 becomes -u2/c1: treat it as 0 * old - 0 * b + (-1/c1) * u2
                nb[r] = srow[r] ? 0.0 : -(double)p.b[s] * Cinv;
                us[r] = srow[r] ? -c1inv : (double)p.u2[s] * c1inv;
                corner[r] = srow[r] ? c1inv : -us[r];                            // value of column r0 in this row
            }
        }
#pragma unroll
        for (int j = 0; j < G1_UH; ++j) {
            const int64_t c = base + TB * j;
            if (c < n2) {
                const float2 bb = b2[c], uu = u2v[c], hh = h2[c];
                const int64_t rc = r0 - c * 2;           // position of column r0 inside this piece, if any
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
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        double t = warp_sum(yacc[r]);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
        __syncthreads();
        if (threadIdx.x == 0 && s0 + r < p.nI) {
            double sum = 0.0;
#pragma unroll
            for (int i = 0; i < TB / 32; ++i) sum += red[i];
            p.y[s0 + r] = (float)sum;
        }
    }
}

// y = Hd h for the entering group chosen by the bootstrap (one warp per row; runs once per state build).
__global__ void __launch_bounds__(256) k_ypass_d(Ptrs p)
{
    if (p.ctl->done) return;
    const int lane = threadIdx.x & 31;
    const int64_t s = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (s >= p.nI) return;
    const float* hrow = p.Hp + (p.nI + (int64_t)p.ctl->sel_t) * p.ldp;
    const double* arow = p.Hd + s * p.ldh;
    double acc = 0.0;
    for (int64_t c = lane; c < p.nI; c += 32) acc = fma(arow[c], (double)hrow[c], acc);
    acc = warp_sum(acc);
    if (lane == 0) p.y[s] = (float)acc;
}

// Hd := (double) Hinv + (double) Dlt, symmetrised (second Newton-Schulz step, summed in fp64), and the reverse copy.
__global__ void k_hinv_to_d(const float* __restrict__ Hinv, const float* __restrict__ Dlt, double* __restrict__ Hd, int64_t ldh, int64_t n,
                            const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t r = blockIdx.x;
    for (int64_t c = threadIdx.x; c < ldh; c += blockDim.x) {
        double v = 0.0;
        if (c < n) v = 0.5 * (((double)Hinv[r * ldh + c] + (double)Hinv[c * ldh + r]) + ((double)Dlt[r * ldh + c] + (double)Dlt[c * ldh + r]));
        Hd[r * ldh + c] = v;
    }
}
__global__ void k_hinv_from_d(const double* __restrict__ Hd, float* __restrict__ Hinv, int64_t ldh, const int32_t* __restrict__ done)
{
    if (done && *done) return;
    const int64_t r = blockIdx.x;
    for (int64_t c = threadIdx.x; c < ldh; c += blockDim.x) Hinv[r * ldh + c] = (float)Hd[r * ldh + c];
}
