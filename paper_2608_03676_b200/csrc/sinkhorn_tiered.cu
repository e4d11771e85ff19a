// Sinkhorn-Knopp (Appendix A.2) for a tiered cost matrix: O(R) work per half-step, several warps per problem.
//
// The paper's cost is a topology cost: C_ij depends only on whether i and j share a node (8 ranks), a rail
// group (4 nodes) or neither.  With supply and demand on disjoint rank sets the diagonal never takes part, so a
// row sum of the absorbed kernel matrix  K~_ij = exp(alpha_i + beta_j - C_ij/eps)  splits by tier:
//
//   (K~ v~)_i = e1_i * N_n(i) + e2_i * (G_g(i) - f_n(i) N_n(i)) + e3_i * (T - F_g(i) G_g(i))
//
// N_n  = sum over demand ranks j of node n of  exp(beta_j - m1_n) v~_j          (m1_n = max beta in the node)
// G_g  = sum over the nodes of group g of  f_n N_n,   f_n = exp(m1_n - m2_g)     (m2_g = max m1 in the group)
// T    = sum over the groups of  F_g G_g,             F_g = exp(m2_g - m3)       (m3   = max m2)
// e1_i = exp(alpha_i - c1/eps + m1_n(i)),  e2_i = exp(alpha_i - c2/eps + m2_g(i)),  e3_i = exp(alpha_i - c3/eps + m3)
//
// and the column sums the same way with the roles of alpha and beta exchanged.  The shifts m keep every factor
// inside the fp32 range: a term that underflows is smaller by e^-87 than another term of the same sum.  The two
// differences lose nothing that matters: e1_i N_n >= e2_i f_n N_n * exp((c2 - c1)/eps) >= e2_i f_n N_n, so the
// rounding error of G (relative to G) enters the row sum with a weight no larger than the row sum itself, and
// likewise for T.
//
// The iteration, its stopping rule, the drift fold of u~, v~ into the fp64 potentials (which recomputes every
// factor above), the first iteration in the log domain and the column cap follow the register-tile kernels;
// problems this kernel cannot take (a rank with both supply and demand, sums outside the safe fp32 range) are
// handed back (iters = -1) to the general kernel.
//
// The ranks of a problem are spread over the lanes of KW warps (8, 4 or 2: see launch_mw_ranks for which).
// Lane gl = 32 * warp + lane owns RPL = R / (32 KW) consecutive ranks: a node of 8 ranks is 8 / RPL adjacent lanes,
// a rail group 32 / RPL lanes, a warp holds RPL whole groups.  A half-step is lane-local products, five xor-shuffle levels (node, group, groups of the warp), one shared-memory exchange of
// the KW warp totals (one named barrier), one multiply-add and a reciprocal per rank.  The iteration is one
// dependent chain on a nearly empty SM, so everything that is not on the chain is kept out of the loop:
//   * the loop body holds no rare case: a thread that sees its u~ or v~ drift out of range stores the number of the
//     next exchange in a flag word, every thread reads that word (and the stop word) after the exchange's barrier,
//     and any event -- drift, stop, last iteration -- leaves the loop for code that all threads run together;
//   * with a tolerance, the row error of an iterate is not reduced by these warps at all: each lane stores
//     its term, and one more warp, which otherwise only takes part in the barriers, sums the terms after
//     half-step 2's barrier and posts the iteration number in the stop word if the error is within the tolerance.
//     The others see the word after the next barrier, half a step into iteration t + 1, and put iterate t back.
#include "sinkhorn_common.cuh"

using namespace taot_sk;

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float exp_or_zero(double x) { return x == -INFINITY ? 0.0f : exp_split(x); }

struct TierCosts {
    double c1, c2, c3;            // cost / eps of the three tiers off the diagonal
};

// C_ij / eps for i != j, from the indices alone: kNode ranks per node, kGroup ranks per rail group
template <int kNode, int kGroup>
__device__ __forceinline__ double tier_cost(const TierCosts& tc, int i, int j)
{
    return (i / kNode == j / kNode) ? tc.c1 : ((i / kGroup == j / kGroup) ? tc.c2 : tc.c3);
}

// Iteration 1, second half, in the log domain (Appendix A.2 with v = 1 on every rank in the first half):
// psi_q = log d_q - LSE_i(phi_i - C_iq/eps) over the Hn supply ranks hot[], phi = alpha.
template <int kNode, int kGroup>
__device__ __forceinline__ double first_column_potential(const TierCosts& tc, const double* alpha, const int32_t* hot, int Hn,
                                                         int q, float dq)
{
    double mx = -INFINITY;
    for (int h = 0; h < Hn; ++h) {
        const int r = hot[h];
        const double v = alpha[r] - tier_cost<kNode, kGroup>(tc, r, q);
        mx = v > mx ? v : mx;
    }
    double acc = 0.0;
    for (int h = 0; h < Hn; ++h) {
        const int r = hot[h];
        acc += (double)exp_split(alpha[r] - tier_cost<kNode, kGroup>(tc, r, q) - mx);
    }
    return log((double)dq) - (mx + log(acc));
}


template <int LO, int HI>
__device__ __forceinline__ float xor_sum(float v)           // all-reduce over lane bits LO <= offset < HI
{
#pragma unroll
    for (int o = LO; o < HI; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
template <int LO, int HI>
__device__ __forceinline__ double xor_max(double v)
{
#pragma unroll
    for (int o = LO; o < HI; o <<= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// ((a0 + a2) + (a4 + a6)) + ((a1 + a3) + (a5 + a7)) with packed fp32 additions: four instructions, three levels
__device__ __forceinline__ float sum8(const float4 lo, const float4 hi)
{
    unsigned long long p0, p1, p2, p3;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p0) : "f"(lo.x), "f"(lo.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(p1) : "f"(lo.z), "f"(lo.w));
    asm("mov.b64 %0, {%1, %2};" : "=l"(p2) : "f"(hi.x), "f"(hi.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(p3) : "f"(hi.z), "f"(hi.w));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(p0) : "l"(p0), "l"(p1));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(p2) : "l"(p2), "l"(p3));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(p0) : "l"(p0), "l"(p2));
    float x, y;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(p0));
    return x + y;
}

// one of the two barriers of an iteration: every thread of the block, whatever code it is in
__device__ __forceinline__ void bar_loop(const int nthreads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// kNode ranks per node, kGroup ranks per rail group (powers of two, kNode < kGroup, a group inside one warp)
template <int kNode, int kGroup, int KW, int RPL, bool TOL>
__global__ void __launch_bounds__(KW * 32 + 32)
sinkhorn_tiered_mw_kernel(SinkArgs a, TierCosts tc, int64_t nprob)
{
    constexpr int kWarps = KW, kThreads = KW * 32;
    static_assert(KW == 2 || KW == 4 || KW == 8, "the warp totals are exchanged as one or two 16-byte words");
    static_assert(kGroup / RPL <= 32 && kGroup > kNode && kGroup % kNode == 0, "a rail group is held by the lanes of one warp");
    constexpr int LPN = kNode / RPL;              // lanes per node
    constexpr int LPG = kGroup / RPL;             // lanes per rail group
    static_assert(RPL >= 1 && RPL <= kNode && kNode % RPL == 0, "a lane holds part of one node");
    constexpr int NW = kWarps + (TOL ? 1 : 0);    // warps of the block: with a tolerance, one more that sums the error
    constexpr int NT = NW * 32;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int R = a.R, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool mainw = warp < kWarps;             // this warp owns ranks
    const int64_t b = blockIdx.x;
    if (b >= nprob) return;
    double* alpha = reinterpret_cast<double*>(smem_raw);          // [R] potentials by rank (supply ranks; -inf elsewhere)
    double* beta = alpha + R;                                      // [R] (demand ranks)
    float* fgs = reinterpret_cast<float*>(beta + R);               // [R] column cap of the final plan, 0 off the demand ranks
    int32_t* hot = reinterpret_cast<int32_t*>(fgs + R);            // [R] supply ranks, ascending
    __shared__ __align__(16) float xtot[2][kWarps + 4];  // what a warp hands to the others in one half-step: its share of the total
    __shared__ __align__(16) float xe[kThreads];         // each lane's term of the row error of the iterate
    __shared__ int xev[4];                               // events of the iteration loop (see there)
    __shared__ double dred[2][NW];
    __shared__ int ired[NW];

    // block-wide reductions for the set-up and the folds (two barriers each; not used inside an iteration)
    auto block_sum2 = [&](double& p, double& q) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            p += __shfl_xor_sync(kFull, p, o);
            q += __shfl_xor_sync(kFull, q, o);
        }
        if (lane == 0) { dred[0][warp] = p; dred[1][warp] = q; }
        __syncthreads();
        p = 0.0; q = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) { p += dred[0][w]; q += dred[1][w]; }
        __syncthreads();
    };
    auto block_max2 = [&](double& p, double& q) {               // p, q already reduced over the warp
        if (lane == 0) { dred[0][warp] = p; dred[1][warp] = q; }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < NW; ++w) { p = fmax(p, dred[0][w]); q = fmax(q, dred[1][w]); }
        __syncthreads();
    };

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)); masses of this lane's ranks
    const int q0 = tid * RPL;                     // first rank of this lane
    float x[RPL];
    unsigned hotm = 0u, coldm = 0u;
    int both = 0;
    double ps = 0.0, pd = 0.0;
#pragma unroll
    for (int i = 0; i < RPL; ++i) {
        const float sv = mainw ? a.s[b * R + q0 + i] : 0.0f, dv = mainw ? a.d[b * R + q0 + i] : 0.0f;
        if (sv > 0.0f) { ps += (double)sv; hotm |= 1u << i; }
        if (dv > 0.0f) { pd += (double)dv; coldm |= 1u << i; }
        both |= (sv > 0.0f && dv > 0.0f) ? 1 : 0;
        x[i] = sv > 0.0f ? sv : (dv > 0.0f ? dv : 0.0f);
    }
    block_sum2(ps, pd);
    if (__syncthreads_or(both)) {                 // the diagonal would take part: not this kernel's case
        if (tid == 0) a.iters[b] = kHandBack;
        return;
    }
    const double sum_s = ps, sum_d = pd;
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, (double)a.eps0));
#pragma unroll
    for (int i = 0; i < RPL; ++i)
        if ((hotm >> i) & 1u) x[i] = (float)(gamma * (double)x[i]);
    int info = 0;
    if (sum_s > sum_d) info |= TAOT_INFO_SUPPLY_SCALED;
    float* out = a.plan + b * (int64_t)R * R;
    // supply ranks in ascending order: prefix over the lanes of a warp, then over the warps
    const int Hn_lane = __popc(hotm), Cn_lane = __popc(coldm);
    int incl = Hn_lane, Cw = Cn_lane;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += up;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Cw += __shfl_xor_sync(kFull, Cw, o);
    if (lane == 31) ired[warp] = incl;
    if (lane == 0) dred[0][warp] = (double)Cw;
    __syncthreads();
    int Hn = 0, hbase = incl - Hn_lane, Cn = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        if (w < warp) hbase += ired[w];
        Hn += ired[w];
        Cn += (int)dred[0][w];
    }
    __syncthreads();
    if (Hn == 0 || Cn == 0) {
        for (int q = tid; q < R * R; q += NT) out[q] = 0.0f;
        if (tid == 0) {
            a.iters[b] = 0;
            a.row_err[b] = 0.0f;
            if (info) atomicOr(a.info + b, info);
        }
        return;
    }
    {
        int k = hbase;
#pragma unroll
        for (int i = 0; i < RPL; ++i)
            if ((hotm >> i) & 1u) hot[k++] = q0 + i;
    }
    double sum_st = 0.0, unused = 0.0;
#pragma unroll
    for (int i = 0; i < RPL; ++i)
        if ((hotm >> i) & 1u) sum_st += (double)x[i];
    block_sum2(sum_st, unused);
    const double tol_abs = (double)a.tol * sum_st;
    const float tol_abs_f = (float)tol_abs;

    // ---- iteration 1 in the log domain (v = 1 on every rank): phi = log s~ - LSE_j(-C_ij/eps) over all j,
    //      psi_j = log d_j - LSE_i(phi_i - C_ij/eps)
    if (mainw) {
#pragma unroll
        for (int i = 0; i < RPL; ++i)
            alpha[q0 + i] = ((hotm >> i) & 1u) ? log((double)x[i]) - a.rowlse0[q0 + i] : -INFINITY;
    }
    __syncthreads();
    if (mainw) {
#pragma unroll 1
        for (int i = 0; i < RPL; ++i) {
            const int q = q0 + i;
            double bj = -INFINITY;
            if ((coldm >> i) & 1u) bj = first_column_potential<kNode, kGroup>(tc, alpha, hot, Hn, q, a.d[b * R + q]);
            beta[q] = bj;
        }
    }
    __syncthreads();
    // ---- per-rank state: z = u~ or v~; pr / pc = this rank's term of its node sum for the next row / column sums
    // (weight times scaling: zero unless the rank is a demand / supply rank); wrx / wcx = that weight times the rank's
    // mass, so that the term follows from the reciprocal of a sum in one multiplication; kA, kB, k3 = coefficients of
    // its own sum on the node sum, the group sum and the total:
    //   own sum = k1 N + k2 (G - f N) + k3 (T - F G) = (k1 - k2 f) N + (k2 - k3 F) G + k3 T,
    // with f, F the node and group factors of the tree the sum is taken over (b: demand side, feeds the row sums; a:
    // supply side, feeds the column sums).  k1 >= k2 f exp((c2 - c1)/eps) and k2 >= k3 F exp((c3 - c2)/eps), so the two
    // differences are formed without cancellation that matters.
    float z[RPL], pr[RPL], pc[RPL], wrx[RPL], wcx[RPL], wc[RPL], kA[RPL], kB[RPL], k3[RPL];
    float fb = 0.0f, fa = 0.0f, Fb = 0.0f, Fa = 0.0f;
#pragma unroll
    for (int i = 0; i < RPL; ++i) z[i] = 1.0f;

    // (keep: also store what the final plan is written from -- a supply rank's three tier coefficients, a demand
    // rank's weight and that weight times its node factor and times node and group factor)
    float pf1[RPL], pf2[RPL], pf3[RPL];
    auto rebuild = [&](const bool keep) {          // block-uniform: holds barriers; expects z = 1
        double m1 = -INFINITY, p1 = -INFINITY;
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            if ((coldm >> i) & 1u) m1 = fmax(m1, beta[q0 + i]);
            if ((hotm >> i) & 1u) p1 = fmax(p1, alpha[q0 + i]);
        }
        m1 = xor_max<1, LPN>(m1); p1 = xor_max<1, LPN>(p1);
        const double m2 = xor_max<LPN, LPG>(m1), p2 = xor_max<LPN, LPG>(p1);
        double m3 = xor_max<LPG, 32>(m2), p3 = xor_max<LPG, 32>(p2);
        block_max2(m3, p3);
        fb = exp_or_zero(m1 == -INFINITY ? -INFINITY : m1 - m2);
        fa = exp_or_zero(p1 == -INFINITY ? -INFINITY : p1 - p2);
        Fb = exp_or_zero(m2 == -INFINITY ? -INFINITY : m2 - m3);
        Fa = exp_or_zero(p2 == -INFINITY ? -INFINITY : p2 - p3);
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const bool ish = (hotm >> i) & 1u, isc = (coldm >> i) & 1u;
            float wrow = 0.0f, wcol = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
            if (ish) {
                const double al = alpha[q0 + i];
                wcol = exp_or_zero(al - p1);
                a1 = exp_or_zero(m1 == -INFINITY ? -INFINITY : al - tc.c1 + m1);
                a2 = exp_or_zero(m2 == -INFINITY ? -INFINITY : al - tc.c2 + m2);
                a3 = exp_or_zero(m3 == -INFINITY ? -INFINITY : al - tc.c3 + m3);
            } else if (isc) {
                const double be = beta[q0 + i];
                wrow = exp_or_zero(be - m1);
                a1 = exp_or_zero(p1 == -INFINITY ? -INFINITY : be - tc.c1 + p1);
                a2 = exp_or_zero(p2 == -INFINITY ? -INFINITY : be - tc.c2 + p2);
                a3 = exp_or_zero(p3 == -INFINITY ? -INFINITY : be - tc.c3 + p3);
            }
            // a supply rank's own sum is a row sum (demand-side tree), a demand rank's a column sum
            kA[i] = fmaf(-a2, ish ? fb : fa, a1);
            kB[i] = fmaf(-a3, ish ? Fb : Fa, a2);
            k3[i] = a3;
            wc[i] = wcol;
            wrx[i] = wrow * x[i]; wcx[i] = wcol * x[i];
            pr[i] = wrow; pc[i] = wcol;            // z = 1
            if (keep) {
                pf1[i] = ish ? a1 : wrow;
                pf2[i] = ish ? a2 : fb * wrow;
                pf3[i] = ish ? a3 : Fb * (fb * wrow);
            }
        }
    };
    auto fold = [&](const bool keep) {             // u~, v~ into the fp64 potentials, then every factor anew
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            if ((hotm >> i) & 1u) alpha[q0 + i] += log((double)z[i]);
            if ((coldm >> i) & 1u) beta[q0 + i] += log((double)z[i]);
            z[i] = 1.0f;
        }
        rebuild(keep);
    };
    // First part of a half-step, everything that does not need the other warps: the lane's node sum and group sum by
    // five xor-shuffle levels, the warp's share of the total (the same value in all of its lanes when a warp is one
    // rail group) and `base[i]`, each rank's own sum without the total's term.
    auto partial = [&](const bool rows, const float (&term)[RPL], float (&base)[RPL]) {
        float p = term[0];
#pragma unroll
        for (int i = 1; i < RPL; ++i) p += term[i];
#pragma unroll
        for (int o = 1; o < LPN; o <<= 1) p += __shfl_xor_sync(kFull, p, o);
        const float N = p;
        // every node appears LPN times among the lanes of its group: sum one copy per node
        float g = (rows ? fb : fa) * N;
#pragma unroll
        for (int o = LPN; o < LPG; o <<= 1) g += __shfl_xor_sync(kFull, g, o);
        const float G = g;
        float tt = (rows ? Fb : Fa) * G;           // every group appears once per LPG lanes
#pragma unroll
        for (int o = LPG; o < 32; o <<= 1) tt += __shfl_xor_sync(kFull, tt, o);
#pragma unroll
        for (int i = 0; i < RPL; ++i) base[i] = fmaf(kA[i], N, kB[i] * G);
        return tt;
    };
    // second part: the eight warp totals, summed pairwise (the same in every thread)
    auto total_of = [&](const int buf) {
        if constexpr (KW == 8) {
            const float4 lo = *reinterpret_cast<const float4*>(&xtot[buf][0]);
            const float4 hi = *reinterpret_cast<const float4*>(&xtot[buf][4]);
            return sum8(lo, hi);
        } else if constexpr (KW == 4) {
            const float4 v = *reinterpret_cast<const float4*>(&xtot[buf][0]);
            return (v.x + v.y) + (v.z + v.w);
        } else {
            const float2 v = *reinterpret_cast<const float2*>(&xtot[buf][0]);
            return v.x + v.y;
        }
    };
    // exact row error of the iterate (u~, v~) = z whose row sums are r, and whether a row sum left the safe range:
    // block-wide, for the iterate that is the result
    auto exact_error = [&](const float (&r)[RPL], double& err, int& bad) {
        double e = 0.0, unused = 0.0;
        int b2 = 0;
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const bool ish = (hotm >> i) & 1u;
            e += ish ? (double)fabsf(fmaf(z[i], r[i], -x[i])) : 0.0;
            b2 |= (ish && !(r[i] > kSumLo && r[i] < kSumHi)) ? 1 : 0;
        }
        block_sum2(e, unused);
        err = e;
        bad = __syncthreads_or(b2);
    };
    rebuild(false);

    // ---- the iterations; t = iteration in progress.  xev[0] = the iteration whose half-step 1 ends with an event: the
    // last one unless a thread that saw its u~ or v~ drift (xev[2]) or the ninth warp that found the previous iterate
    // within the tolerance (xev[1]) put the next iteration there.
    int t = 1;
    int until_check = a.check_every;
    const bool every = a.check_every <= 1;
    float err_out = 0.0f;
    const uint32_t lo_bits = __float_as_uint(kDriftLo), span_bits = __float_as_uint(kDriftHi) - lo_bits;
    float r[RPL], zkeep[RPL], base[RPL];
#pragma unroll
    for (int i = 0; i < RPL; ++i) { r[i] = 1.0f; zkeep[i] = 1.0f; base[i] = 0.0f; }
    if (tid == 0) { xev[0] = a.max_iters; xev[1] = -1; xev[2] = -1; }
    __syncthreads();
    for (;;) {
        float T = 0.0f;
        if (mainw) {
            for (;;) {
                // ================= half-step 1: r = K~ v~ on the supply ranks; these row sums belong to iterate t
                xtot[0][warp] = partial(true, pr, base);
                bar_loop(NT);
                T = total_of(0);
                if (xev[0] <= t) break;
                float rr[RPL];
#pragma unroll
                for (int i = 0; i < RPL; ++i) {
                    r[i] = fmaf(k3[i], T, base[i]);
                    rr[i] = rcp_fast(r[i]);
                    pc[i] = ((hotm >> i) & 1u) ? wcx[i] * rr[i] : 0.0f;
                }
                // ================= half-step 2: c = K~^T u' on the demand ranks, v' = d / c
                xtot[1][warp] = partial(false, pc, base);
                if (TOL) {
                    bool check_now = true;
                    if (!every) {
                        check_now = until_check == 1;
                        until_check = check_now ? a.check_every : until_check - 1;
                    }
                    if (check_now) {               // this lane's term of the row error, for the ninth warp
                        float e = 0.0f;
#pragma unroll
                        for (int i = 0; i < RPL; ++i) {
                            e += ((hotm >> i) & 1u) ? fabsf(fmaf(z[i], r[i], -x[i])) : 0.0f;
                            zkeep[i] = z[i];
                        }
                        xe[tid] = e;
                    }
                }
                float zn[RPL];
#pragma unroll
                for (int i = 0; i < RPL; ++i) zn[i] = ((hotm >> i) & 1u) ? x[i] * rr[i] : z[i];
                bar_loop(NT);
                T = total_of(1);
                // a sum outside the safe range shows in its reciprocal (zero, infinite or not a number), so the
                // drift test catches it too; a rank that takes no part keeps z = 1
                ++t;
                bool drift = false;
#pragma unroll
                for (int i = 0; i < RPL; ++i) {
                    const float c = fmaf(k3[i], T, base[i]);
                    const float rc = rcp_fast(c);
                    pr[i] = ((coldm >> i) & 1u) ? wrx[i] * rc : 0.0f;
                    z[i] = ((coldm >> i) & 1u) ? x[i] * rc : zn[i];
                    drift |= (__float_as_uint(z[i]) - lo_bits) > span_bits;
                }
                if (drift) { xev[2] = t; xev[0] = t; }     // read after the next barrier; every writer stores the same t
            }
        } else {
            // the ninth warp: the same barriers, the same events; between half-step 2's barrier and the next one it
            // sums the 256 terms of the row error (eight per lane, then five shuffle levels: one fixed order)
            for (;;) {
                bar_loop(NT);
                if (xev[0] <= t) break;
                bool check_now = true;
                if (!every) {
                    check_now = until_check == 1;
                    until_check = check_now ? a.check_every : until_check - 1;
                }
                bar_loop(NT);
                ++t;
                if (check_now) {
                    float e;
                    if constexpr (KW == 8) {
                        const float4 lo = *reinterpret_cast<const float4*>(&xe[lane * 8]);
                        const float4 hi = *reinterpret_cast<const float4*>(&xe[lane * 8 + 4]);
                        e = ((lo.x + lo.y) + (lo.z + lo.w)) + ((hi.x + hi.y) + (hi.z + hi.w));
                    } else if constexpr (KW == 4) {
                        const float4 v = *reinterpret_cast<const float4*>(&xe[lane * 4]);
                        e = (v.x + v.y) + (v.z + v.w);
                    } else {
                        const float2 v = *reinterpret_cast<const float2*>(&xe[lane * 2]);
                        e = v.x + v.y;
                    }
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) e += __shfl_xor_sync(kFull, e, o);
                    if (lane == 0 && e <= tol_abs_f) { xev[1] = t; xev[0] = t; }
                }
            }
        }
        // ---- an event: every thread of the block is here, after the barrier of half-step 1 of iteration t
        const int ev_stop = xev[1], ev_drift = xev[2];
        __syncthreads();
        if (TOL && ev_stop == t) {                 // iterate t - 1 met the tolerance: it is the result
            --t;
#pragma unroll
            for (int i = 0; i < RPL; ++i) z[i] = zkeep[i];
            double err;
            int bad;
            exact_error(r, err, bad);
            if (bad) { if (tid == 0) a.iters[b] = kHandBack; return; }
            err_out = (float)(err / sum_st);
            break;
        }
        if (ev_drift == t) {
            // Some u~ or v~ of the previous update left [e^-40, e^40].  Either a sum left the safe range -- its
            // reciprocal is then zero, infinite, not a number or far outside any drift -- and the problem is handed
            // back, or the factors drifted: fold them into the potentials and take the half-step again.
            int range = 0;
#pragma unroll
            for (int i = 0; i < RPL; ++i)
                range |= (!(z[i] > x[i] * kSumLo && z[i] < x[i] * kSumHi) && ((hotm | coldm) >> i & 1u)) ? 1 : 0;
            if (__syncthreads_or(range)) {
                if (tid == 0) a.iters[b] = kHandBack;
                return;
            }
            if (tid == 0) { xev[0] = a.max_iters; xev[2] = -1; }
            fold(false);
            continue;
        }
        // the last iteration: iterate t is the result whatever its error
#pragma unroll
        for (int i = 0; i < RPL; ++i) r[i] = fmaf(k3[i], T, base[i]);
        double err;
        int bad;
        exact_error(r, err, bad);
        if (bad) { if (tid == 0) a.iters[b] = kHandBack; return; }
        err_out = (float)(err / sum_st);
        if (TOL && !((float)err <= tol_abs_f)) info |= TAOT_INFO_SINKHORN_CAP;
        break;
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap.  With the shifts of the tier sums an
    // entry is a product of fp32 factors that are all in range: T_ij = a1_i w_j (same node), a2_i f_n(j) w_j (same rail
    // group), a3_i F_g(j) f_n(j) w_j (neither), times the cap of column j; a factor that underflows belongs to an
    // entry e^-87 below the largest of its row.  The factors go to shared memory (over the potentials, which are no
    // longer needed) and a row costs one multiplication per entry.
    fold(true);
    float cap[RPL];
    {
        xtot[0][warp] = partial(false, wc, base);                               // column sums of K~ itself (u~ = 1)
        __syncthreads();                                                        // (also: every potential has been read)
        const float T = total_of(0);
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const float c = fmaf(k3[i], T, base[i]);
            cap[i] = ((coldm >> i) & 1u) ? (float)fmin(1.0, (double)x[i] / ((double)c + (double)a.eps0)) : 0.0f;
        }
    }
    float* rowf = reinterpret_cast<float*>(smem_raw);     // [3][R] tier coefficients of a supply rank's row; [0] < 0: no row
    float* colf = rowf + 3 * R;                            // [3][R] column factors by tier, zero off the demand ranks
    if (mainw) {
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const bool ish = (hotm >> i) & 1u, isc = (coldm >> i) & 1u;
            const int q = q0 + i;
            rowf[q] = ish ? pf1[i] : -1.0f; rowf[R + q] = ish ? pf2[i] : 0.0f; rowf[2 * R + q] = ish ? pf3[i] : 0.0f;
            colf[q] = isc ? pf1[i] * cap[i] : 0.0f; colf[R + q] = isc ? pf2[i] * cap[i] : 0.0f;
            colf[2 * R + q] = isc ? pf3[i] * cap[i] : 0.0f;
        }
    }
    __syncthreads();
    int nonfinite = 0;
    for (int row = warp; row < R; row += NW) {
        float* orow = out + (int64_t)row * R;
        const float a1 = rowf[row];
        if (a1 < 0.0f) {
            for (int j = lane; j < R; j += 32) orow[j] = 0.0f;
            continue;
        }
        const float a2 = rowf[R + row], a3 = rowf[2 * R + row];
        const int node = row / kNode, group = row / kGroup;
#pragma unroll 4
        for (int j = lane; j < R; j += 32) {
            const bool sn = j / kNode == node, sg = j / kGroup == group;
            const float v = sn ? a1 * colf[j] : (sg ? a2 * colf[R + j] : a3 * colf[2 * R + j]);
            if (!isfinite(v)) nonfinite = 1;
            orow[j] = v;
        }
    }
    if (__syncthreads_or(nonfinite)) info |= TAOT_INFO_NONFINITE;
    if (tid == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
}

constexpr size_t kExclusiveSmem = 200 * 1024;

template <int kNode, int kGroup, int KW, int RPL>
int launch_mw(const SinkArgs& a, const TierCosts& tc, int32_t B, cudaStream_t st)
{
    constexpr int kThreads = KW * 32;
    size_t smem = (size_t)a.R * (2 * sizeof(double) + sizeof(float) + sizeof(int32_t));
    // A batch far smaller than the GPU is one dependent chain per problem: give each problem an SM to itself (a
    // shared-memory request no two CTAs of any kernel can share an SM with), so that neither the problems of other
    // launches in flight nor the bandwidth-bound kernels of other layer groups take issue slots from the chain.
    int dev = 0, sms = 0;
    TAOT_CUDA_OK(cudaGetDevice(&dev));
    TAOT_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (2 * B <= sms && smem < kExclusiveSmem) smem = kExclusiveSmem;
    if (a.tol > 0.0f) {
        TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_tiered_mw_kernel<kNode, kGroup, KW, RPL, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sinkhorn_tiered_mw_kernel<kNode, kGroup, KW, RPL, true><<<B, kThreads + 32, smem, st>>>(a, tc, (int64_t)B);
    } else {
        TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_tiered_mw_kernel<kNode, kGroup, KW, RPL, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sinkhorn_tiered_mw_kernel<kNode, kGroup, KW, RPL, false><<<B, kThreads, smem, st>>>(a, tc, (int64_t)B);
    }
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

// Warps per problem by batch size (measured, 500 fixed iterations, B = 1 / 64 / 1024 / 4096, ms):
//   256 ranks:  8 warps 0.175 / 0.177 / 0.478 / 1.77,  4 warps 0.174 / 0.175 / 0.285 / 0.981,  2 warps 0.216 / 0.218 / 0.287 / 0.843
//               (one warp with 8 ranks per lane, a kernel of its own until then: - / - / 0.414 / 0.988)
//   512 ranks:  8 warps 0.214 / 0.218 / 0.779 / 2.63,  4 warps 0.236 / 0.240 / 0.619 / 1.88,   2 warps 0.318 / 0.324 / 0.811 / 2.09
//   1024 ranks: 8 warps 0.343 / 0.359 / 1.68 / 5.92,   4 warps 0.384 / 0.412 / 1.61 / 5.11
// A problem that has an SM to itself is one dependent chain and wants the fewest instructions per warp (8 warps; with a
// tolerance also at 256 ranks, 0.381 against 0.391 ms at config 4); a batch that fills the GPU wants the fewest
// instructions per problem that still leave enough warps to hide each other's latency (4 warps, 2 for the largest
// batches at 256 ranks).
template <int kNode, int kGroup>
int launch_mw_ranks(const SinkArgs& a, const TierCosts& tc, int32_t B, cudaStream_t st)
{
    int dev = 0, sms = 0;
    TAOT_CUDA_OK(cudaGetDevice(&dev));
    TAOT_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const bool alone = 2 * B <= sms;               // every problem gets an SM to itself
    const bool huge = B >= 16 * sms;
    switch (a.R) {
        case 256:
            if constexpr (kNode >= 4) {
                if (huge) return launch_mw<kNode, kGroup, 2, 4>(a, tc, B, st);
            }
            if constexpr (kNode >= 2) {
                if (!alone) return launch_mw<kNode, kGroup, 4, 2>(a, tc, B, st);
            }
            return launch_mw<kNode, kGroup, 8, 1>(a, tc, B, st);
        case 512:
            if constexpr (kNode >= 4) {
                if (!alone) return launch_mw<kNode, kGroup, 4, 4>(a, tc, B, st);
            }
            if constexpr (kNode >= 2) return launch_mw<kNode, kGroup, 8, 2>(a, tc, B, st); else return 0;
        case 1024:
            if constexpr (kNode >= 8) {
                if (!alone) return launch_mw<kNode, kGroup, 4, 8>(a, tc, B, st);
            }
            if constexpr (kNode >= 4) return launch_mw<kNode, kGroup, 8, 4>(a, tc, B, st); else return 0;
        default: return 0;
    }
}

}  // namespace

// Launches the tiered-cost kernel if the handle's cost matrix has the node / rail-group structure (checked at
// taot_create, which also requires 256, 512 or 1024 ranks); returns the number of kernels launched (0: not
// applicable or a hierarchy that is not built, the caller takes the general kernels).
int taot_launch_sinkhorn_tiered(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st)
{
    if (!h->tier_ok) return 0;
    const float* tier_cost3 = h->tier_cost;
    const int node = h->tier_node, group = h->tier_group;
    TierCosts tc;
    tc.c1 = (double)tier_cost3[0] * a.inv_eps;
    tc.c2 = (double)tier_cost3[1] * a.inv_eps;
    tc.c3 = (double)tier_cost3[2] * a.inv_eps;
    if (node == 8 && group == 32) return launch_mw_ranks<8, 32>(a, tc, B, st);
    if (node == 4 && group == 16) return launch_mw_ranks<4, 16>(a, tc, B, st);
    if (node == 4 && group == 32) return launch_mw_ranks<4, 32>(a, tc, B, st);
    if (node == 16 && group == 32) return launch_mw_ranks<16, 32>(a, tc, B, st);
    return 0;
}
