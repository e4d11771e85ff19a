// Sinkhorn-Knopp (Appendix A.2) for a tiered cost matrix: one warp per problem, O(R) work per half-step.
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
// likewise for T.  A lane owns R/32 consecutive ranks (a node at 256 ranks, the size this kernel is launched for:
// large batches; sinkhorn_tiered_mw.cu spreads a problem over eight warps for small batches and larger R); node
// sums are lane-local, group and total sums are xor-shuffle all-reduces (5 levels per half-step).
//
// The iteration, its stopping rule, the drift fold of u~, v~ into the fp64 potentials (which recomputes every
// factor above), the first iteration in the log domain and the final plan follow the register-tile kernels;
// problems this kernel cannot take (a rank with both supply and demand, sums outside the safe fp32 range) are
// handed back (iters = -1) to the general kernel.
#include "sinkhorn_tiered_common.cuh"

using namespace taot_sk;

namespace {

constexpr int kNode = 8;          // ranks per node
constexpr int kGroup = 32;        // ranks per rail group

// all-reduce over the lanes of one rail group (LPG lanes), and over the groups (one value per group, held by all
// of its lanes)
template <int LPG>
__device__ __forceinline__ float group_sum(float v)
{
#pragma unroll
    for (int o = 1; o < LPG; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
template <int LPG>
__device__ __forceinline__ float across_groups_sum(float v)
{
#pragma unroll
    for (int o = LPG; o < 32; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
template <int LPG>
__device__ __forceinline__ double group_max(double v)
{
#pragma unroll
    for (int o = 1; o < LPG; o <<= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
template <int LPG>
__device__ __forceinline__ double across_groups_max(double v)
{
#pragma unroll
    for (int o = LPG; o < 32; o <<= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

template <int RPL, bool TOL>
__global__ void __launch_bounds__(32)
sinkhorn_tiered_kernel(SinkArgs a, TierCosts tc, int64_t nprob)
{
    constexpr int NPL = RPL / kNode;              // nodes per lane
    constexpr int LPG = kGroup / RPL;             // lanes per rail group
    static_assert(RPL % kNode == 0 && kGroup % RPL == 0, "a lane holds whole nodes of one rail group");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int R = a.R, lane = threadIdx.x;
    const int64_t b = blockIdx.x;
    if (b >= nprob) return;
    double* alpha = reinterpret_cast<double*>(smem_raw);          // [R] potentials by rank (supply ranks)
    double* beta = alpha + R;                                      // [R] (demand ranks)
    float* fgs = reinterpret_cast<float*>(beta + R);               // [R] column cap of the final plan, 0 off the demand ranks
    int32_t* hot = reinterpret_cast<int32_t*>(fgs + R);            // [R] supply ranks, ascending

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)); masses of this lane's ranks
    float x[RPL];                                 // s~ on a supply rank, d on a demand rank
    unsigned hotm = 0u, coldm = 0u;
    bool both = false;
    double ps = 0.0, pd = 0.0;
#pragma unroll
    for (int i = 0; i < RPL; ++i) {
        const float sv = a.s[b * R + lane * RPL + i], dv = a.d[b * R + lane * RPL + i];
        if (sv > 0.0f) { ps += (double)sv; hotm |= 1u << i; }
        if (dv > 0.0f) { pd += (double)dv; coldm |= 1u << i; }
        both |= sv > 0.0f && dv > 0.0f;
        x[i] = sv > 0.0f ? sv : (dv > 0.0f ? dv : 0.0f);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ps += __shfl_xor_sync(kFull, ps, o);
        pd += __shfl_xor_sync(kFull, pd, o);
    }
    if (__any_sync(kFull, both)) {                // the diagonal would take part: not this kernel's case
        if (lane == 0) a.iters[b] = kHandBack;
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
    const int Hn_lane = __popc(hotm), Cn_lane = __popc(coldm);
    int Hn = Hn_lane, Cn = Cn_lane, hbase = 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(kFull, Hn, o);
        if (lane >= o) Hn += up;
    }
    hbase = Hn - Hn_lane;                          // exclusive prefix of the supply ranks
    Hn = __shfl_sync(kFull, Hn, 31);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Cn += __shfl_xor_sync(kFull, Cn, o);
    if (Hn == 0 || Cn == 0) {
        for (int q = lane; q < R * R; q += 32) out[q] = 0.0f;
        if (lane == 0) {
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
            if ((hotm >> i) & 1u) hot[k++] = lane * RPL + i;
    }
    double sum_st = 0.0;
#pragma unroll
    for (int i = 0; i < RPL; ++i)
        if ((hotm >> i) & 1u) sum_st += (double)x[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum_st += __shfl_xor_sync(kFull, sum_st, o);
    const double tol_abs = (double)a.tol * sum_st;
    const float tol_abs_f = (float)tol_abs;

    // ---- iteration 1 in the log domain (v = 1 on every rank): phi = log s~ - LSE_j(-C_ij/eps) over all j,
    //      psi_j = log d_j - LSE_i(phi_i - C_ij/eps)
#pragma unroll
    for (int i = 0; i < RPL; ++i) {
        const int q = lane * RPL + i;
        alpha[q] = ((hotm >> i) & 1u) ? log((double)x[i]) - a.rowlse0[q] : -INFINITY;
    }
    __syncwarp();
#pragma unroll 1
    for (int i = 0; i < RPL; ++i) {
        const int q = lane * RPL + i;
        double bj = -INFINITY;
        if ((coldm >> i) & 1u) bj = first_column_potential<kNode, kGroup>(tc, alpha, hot, Hn, q, a.d[b * R + q]);
        beta[q] = bj;
    }
    __syncwarp();

    // ---- per-rank state in registers: z = u~ (supply rank) or v~ (demand rank), w = its weight inside the node
    // sum, k1..k3 = the three tier coefficients of its own sum; per node f, per lane's group F (both directions)
    float z[RPL], w[RPL], k1[RPL], k2[RPL], k3[RPL];
    float fb[NPL], fa[NPL];           // node factors of the demand-side (row sums) and supply-side (column sums) trees
    float Fb = 0.0f, Fa = 0.0f;
#pragma unroll
    for (int i = 0; i < RPL; ++i) z[i] = 1.0f;

    auto rebuild = [&]() {
        double m1[NPL], p1[NPL];
#pragma unroll
        for (int n = 0; n < NPL; ++n) { m1[n] = -INFINITY; p1[n] = -INFINITY; }
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const int q = lane * RPL + i;
            if ((coldm >> i) & 1u) m1[i / kNode] = fmax(m1[i / kNode], beta[q]);
            if ((hotm >> i) & 1u) p1[i / kNode] = fmax(p1[i / kNode], alpha[q]);
        }
        double m2 = -INFINITY, p2 = -INFINITY;
#pragma unroll
        for (int n = 0; n < NPL; ++n) { m2 = fmax(m2, m1[n]); p2 = fmax(p2, p1[n]); }
        m2 = group_max<LPG>(m2); p2 = group_max<LPG>(p2);
        const double m3 = across_groups_max<LPG>(m2), p3 = across_groups_max<LPG>(p2);
#pragma unroll
        for (int n = 0; n < NPL; ++n) {
            fb[n] = exp_or_zero(m1[n] == -INFINITY ? -INFINITY : m1[n] - m2);
            fa[n] = exp_or_zero(p1[n] == -INFINITY ? -INFINITY : p1[n] - p2);
        }
        Fb = exp_or_zero(m2 == -INFINITY ? -INFINITY : m2 - m3);
        Fa = exp_or_zero(p2 == -INFINITY ? -INFINITY : p2 - p3);
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const int q = lane * RPL + i, n = i / kNode;
            const bool ish = (hotm >> i) & 1u, isc = (coldm >> i) & 1u;
            float wv = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
            if (ish) {
                const double al = alpha[q];
                wv = exp_or_zero(al - p1[n]);
                a1 = exp_or_zero(m1[n] == -INFINITY ? -INFINITY : al - tc.c1 + m1[n]);
                a2 = exp_or_zero(m2 == -INFINITY ? -INFINITY : al - tc.c2 + m2);
                a3 = exp_or_zero(m3 == -INFINITY ? -INFINITY : al - tc.c3 + m3);
            } else if (isc) {
                const double be = beta[q];
                wv = exp_or_zero(be - m1[n]);
                a1 = exp_or_zero(p1[n] == -INFINITY ? -INFINITY : be - tc.c1 + p1[n]);
                a2 = exp_or_zero(p2 == -INFINITY ? -INFINITY : be - tc.c2 + p2);
                a3 = exp_or_zero(p3 == -INFINITY ? -INFINITY : be - tc.c3 + p3);
            }
            w[i] = wv; k1[i] = a1; k2[i] = a2; k3[i] = a3;
        }
    };

    // sums of the absorbed kernel matrix against the current scalings: ROWS: (K~ v~)_i on the supply ranks (sources
    // are the demand ranks), else (K~^T u~)_j on the demand ranks; zsrc = scalings of the sources
    // `carry` (if with_carry): one more value summed over the warp in the same shuffle levels (the row-error partial)
    auto tier_sums = [&](const bool rows, const bool with_carry, const float (&zsrc)[RPL], float (&res)[RPL], float& carry) {
        const unsigned srcm = rows ? coldm : hotm;
        float N[NPL];
#pragma unroll
        for (int n = 0; n < NPL; ++n) {
            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
            for (int i = 0; i < kNode; i += 2) {
                const int i0 = n * kNode + i, i1 = i0 + 1;
                acc0 += ((srcm >> i0) & 1u) ? w[i0] * zsrc[i0] : 0.0f;
                acc1 += ((srcm >> i1) & 1u) ? w[i1] * zsrc[i1] : 0.0f;
            }
            N[n] = acc0 + acc1;
        }
        float g = 0.0f;
#pragma unroll
        for (int n = 0; n < NPL; ++n) g = fmaf(rows ? fb[n] : fa[n], N[n], g);
#pragma unroll
        for (int o = 1; o < LPG; o <<= 1) {
            g += __shfl_xor_sync(kFull, g, o);
            if (with_carry) carry += __shfl_xor_sync(kFull, carry, o);
        }
        const float G = g;
        const float FG = (rows ? Fb : Fa) * G;
        float tt = FG;
#pragma unroll
        for (int o = LPG; o < 32; o <<= 1) {
            tt += __shfl_xor_sync(kFull, tt, o);
            if (with_carry) carry += __shfl_xor_sync(kFull, carry, o);
        }
        const float Tx = tt - FG;
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const int n = i / kNode;
            const float Gx = G - (rows ? fb[n] : fa[n]) * N[n];
            res[i] = fmaf(k1[i], N[n], fmaf(k2[i], Gx, k3[i] * Tx));
        }
    };
    auto fold = [&]() {                            // u~, v~ into the fp64 potentials, then every factor anew
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const int q = lane * RPL + i;
            if ((hotm >> i) & 1u) alpha[q] += log((double)z[i]);
            if ((coldm >> i) & 1u) beta[q] += log((double)z[i]);
            z[i] = 1.0f;
        }
        rebuild();
    };
    rebuild();

    int t = 1;
    int until_check = a.check_every;
    float err_out = 0.0f;
    const uint32_t lo_bits = __float_as_uint(kDriftLo), span_bits = __float_as_uint(kDriftHi) - lo_bits;
    const unsigned anym = hotm | coldm;
    for (;;) {
        // ================= half-step 1: r = K~ v~ on the supply ranks; these row sums belong to iterate t
        float r[RPL];
        float nocarry = 0.0f;
        tier_sums(true, false, z, r, nocarry);
        auto rows_bad = [&]() {
            bool bad = false;
#pragma unroll
            for (int i = 0; i < RPL; ++i) bad |= ((hotm >> i) & 1u) && !(r[i] > kSumLo && r[i] < kSumHi);
            return __any_sync(kFull, bad) != 0;
        };
        const bool last = t >= a.max_iters;
        bool check_now = false;
        if (TOL) {
            check_now = until_check == 1;
            until_check = check_now ? a.check_every : until_check - 1;
        }
        // the error of iterate t is formed here but tested only after half-step 2 has been issued, so that its
        // reduction does not sit on the dependent chain (a stop discards that half-step)
        const bool test = last || check_now;
        float err = 0.0f;
        if (test) {
            float e = 0.0f;
#pragma unroll
            for (int i = 0; i < RPL; ++i) e += ((hotm >> i) & 1u) ? fabsf(fmaf(z[i], r[i], -x[i])) : 0.0f;
            err = e;                               // summed over the warp inside half-step 2's reduction
        }
        float zn[RPL];
#pragma unroll
        for (int i = 0; i < RPL; ++i) zn[i] = ((hotm >> i) & 1u) ? x[i] * rcp_fast(r[i]) : z[i];
        // ================= half-step 2: c = K~^T u' on the demand ranks, v' = d / c
        float c[RPL];
        if (test) tier_sums(false, true, zn, c, err);
        else tier_sums(false, false, zn, c, nocarry);
        if (test && (last || err <= tol_abs_f)) {
            if (rows_bad()) { if (lane == 0) a.iters[b] = kHandBack; return; }
            err_out = (float)((double)err / sum_st);
            if (TOL && !(err <= tol_abs_f)) info |= TAOT_INFO_SINKHORN_CAP;
            break;
        }
        // a sum outside the safe range shows in its reciprocal (zero, infinite or not a number), so the drift test
        // catches it too and the range test itself stays off the common path
        bool odd = false;
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const bool isc = (coldm >> i) & 1u;
            zn[i] = isc ? x[i] * rcp_fast(c[i]) : zn[i];
            odd |= ((anym >> i) & 1u) && (__float_as_uint(zn[i]) - lo_bits) > span_bits;
        }
        const bool drift = __any_sync(kFull, odd) != 0;
        if (drift) {
            bool bad = false;
#pragma unroll
            for (int i = 0; i < RPL; ++i)
                bad |= (((hotm >> i) & 1u) && !(r[i] > kSumLo && r[i] < kSumHi)) ||
                       (((coldm >> i) & 1u) && !(c[i] > kSumLo && c[i] < kSumHi));
            if (__any_sync(kFull, bad)) { if (lane == 0) a.iters[b] = kHandBack; return; }
        }
#pragma unroll
        for (int i = 0; i < RPL; ++i) z[i] = zn[i];
        ++t;
        if (drift) fold();
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
    fold();
    {
        float c[RPL];
        float nocarry = 0.0f;
        tier_sums(false, false, z, c, nocarry);    // column sums of K~ itself (u~ = 1)
#pragma unroll
        for (int i = 0; i < RPL; ++i) {
            const int q = lane * RPL + i;
            fgs[q] = ((coldm >> i) & 1u) ? (float)fmin(1.0, (double)x[i] / ((double)c[i] + (double)a.eps0)) : 0.0f;
        }
    }
    __syncwarp();
    const int nonfinite = write_plan_rows<kNode, kGroup>(tc, alpha, beta, fgs, R, 0, 1, lane, out);
    if (__any_sync(kFull, nonfinite != 0)) info |= TAOT_INFO_NONFINITE;
    if (lane == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
}

template <int RPL>
int launch_rpl(const SinkArgs& a, const TierCosts& tc, int32_t B, cudaStream_t st)
{
    const size_t smem = (size_t)a.R * (2 * sizeof(double) + sizeof(float) + sizeof(int32_t));
    if (a.tol > 0.0f) {
        if (smem > 48 * 1024)
            TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_tiered_kernel<RPL, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sinkhorn_tiered_kernel<RPL, true><<<B, 32, smem, st>>>(a, tc, (int64_t)B);
    } else {
        if (smem > 48 * 1024)
            TAOT_CUDA_OK(cudaFuncSetAttribute(sinkhorn_tiered_kernel<RPL, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        sinkhorn_tiered_kernel<RPL, false><<<B, 32, smem, st>>>(a, tc, (int64_t)B);
    }
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}

}  // namespace

// Launches a tiered-cost kernel if the handle's cost matrix has the node / rail-group structure (checked at
// taot_create, which also requires 256, 512 or 1024 ranks); returns the number of kernels launched (0: not
// applicable, the caller takes the general kernels).
int taot_launch_sinkhorn_tiered_mw(const SinkArgs& a, const float* tier_cost3, int node, int group, int32_t B, cudaStream_t st);

int taot_launch_sinkhorn_tiered(taot_handle_t h, const SinkArgs& a, int32_t B, cudaStream_t st)
{
    if (!h->tier_ok) return 0;
    // few problems per call: eight warps per problem (a lone warp is bound by the instructions it issues); batches
    // of 256-rank problems that fill the GPU several times over: one warp per problem (fewest instructions per
    // problem).  Beyond 256 ranks the eight-warp kernel wins at every batch size (32 ranks per lane do not fit the registers).
    // (the one-warp kernel is built for nodes of 8 and rail groups of 32 ranks: a lane is a node)
    if (B < 4 * h->sm_count || h->p.R > 256 || h->tier_node != 8 || h->tier_group != 32)
        return taot_launch_sinkhorn_tiered_mw(a, h->tier_cost, h->tier_node, h->tier_group, B, st);
    TierCosts tc;
    tc.c1 = (double)h->tier_cost[0] * a.inv_eps;
    tc.c2 = (double)h->tier_cost[1] * a.inv_eps;
    tc.c3 = (double)h->tier_cost[2] * a.inv_eps;
    return launch_rpl<8>(a, tc, B, st);
}
