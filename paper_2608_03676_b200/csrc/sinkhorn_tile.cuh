// Phase 1 fast path: Sinkhorn-Knopp (Appendix A.2) with the absorbed kernel matrix K~ held in
// REGISTERS.  Same arithmetic as the shared-memory kernel in sinkhorn.cu (absorbed potentials,
// fp32 mat-vecs, fp64 folds), different data placement.  Two layouts:
//
// grid_solve (one warp per problem, up to 64 ranks): a 4 x 8 lane grid; lane (lr, lc) holds K~ for rows
//   ra*4 + lr and columns cg*8 + lc.  Row sums reduce over the 8 column lanes and column sums over the 4 row
//   lanes by xor-butterflies, after which every lane of a group holds the same bits, so u~ and v~ are computed
//   where they are needed and nothing is broadcast.  No barrier, no shared memory and (besides one rarely taken
//   exit) no branch in the loop.
//
// tile_solve (4 or 16 warps per problem, up to 128 / 256 ranks):
//   warp w owns compact rows [w*RPW, (w+1)*RPW)  (rows = ranks with supply),
//   lane l owns compact columns l + 32*g, g < CG (columns = ranks with demand),
//   K[a][g] in registers; every warp keeps v~ for its lane's columns in registers.
//   Half-step 1 (row sums) is warp-local: RPW partial sums per lane are reduced across the 32 lanes
//   by a transposing butterfly (RPW-1 + log2(32/RPW) shuffles for all rows together), after which
//   lane a holds row a's sum and computes u~_a = s~_a / r_a.  Half-step 2 (column sums) is
//   lane-local over the warp's rows (u~_a broadcast by shuffle); the partials of the warps
//   meet in shared memory (two block barriers per iteration).
//
// A problem that does not fit the tile (too many rows with supply), or whose fp32 sums leave the
// safe range, is handed back (iters[b] = -1) and solved by the next kernel of the chain, in the end
// by the shared-memory kernel, which holds any problem.
#pragma once
#include "sinkhorn_common.cuh"

using namespace taot_sk;

namespace {

constexpr unsigned kFull = 0xffffffffu;

// Sum over the 32 lanes of N per-lane values at once: on return the value is the total of
// p[lane & (N-1)].  N a power of two, 1 <= N <= 32.
template <int N>
__device__ __forceinline__ float transpose_reduce(float (&p)[N], int lane)
{
#pragma unroll
    for (int off = N / 2; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < off; ++k) {
            const float send = up ? p[k] : p[k + off];
            const float keep = up ? p[k + off] : p[k];
            p[k] = keep + __shfl_xor_sync(kFull, send, off);
        }
    }
    float v = p[0];
#pragma unroll
    for (int off = N; off < 32; off <<= 1) v += __shfl_xor_sync(kFull, v, off);
    return v;
}

__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory state of one problem (arrays sized for RMAX = 32*CG ranks).
template <int NW, int CG>
struct TileSmem {
    static constexpr int RMAX = 32 * CG;
    double alpha[RMAX], beta[RMAX], phin[RMAX], red[64];
    float st[RMAX], dd[RMAX], sv[RMAX], dv[RMAX], vs[RMAX];
    float part[NW > 1 ? NW * RMAX : 1];
    float errw[32];
    int32_t hot[RMAX], cold[RMAX], hpos[RMAX], cpos[RMAX], wcnt[32];
    int flags[4];                    // [parity]: some u~, v~ of this iteration left [e^-40, e^40]
    double sum[2];
};

// The iteration proper, for a tile of RPW rows per warp.  Returns false if the problem must be handed back.
template <int NW, int RPW, int CG>
__device__ __forceinline__ bool tile_solve(const SinkArgs& a, TileSmem<NW, CG>& sm, int Hn, int Cn, double sum_st,
                                           int info, float* out, int64_t b)
{
    constexpr int RMAX = 32 * CG, NT = NW * 32;
    const int R = a.R, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const double tol_abs = (double)a.tol * sum_st;

    const int row0 = warp * RPW;
    const int rowl = row0 + (lane & (RPW - 1));       // the row whose sum this lane ends up holding
    const bool row_ok = rowl < Hn;
    const bool row_owner = row_ok && lane < RPW;
    const float st_l = row_ok ? sm.st[rowl] : 1.0f;
    float K[RPW][CG];
    float ddg[CG], vreg[CG];
    bool col_ok[CG];
#pragma unroll
    for (int g = 0; g < CG; ++g) {
        const int col = lane + 32 * g;
        col_ok[g] = col < Cn;
        ddg[g] = col_ok[g] ? sm.dd[col] : 1.0f;
        vreg[g] = 1.0f;
    }
    auto build_tile = [&]() {
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            const int row = row0 + aa;
#pragma unroll
            for (int g = 0; g < CG; ++g) {
                const int col = lane + 32 * g;
                float v = 0.0f;
                if (row < Hn && col < Cn) {
                    const double c = (double)a.C[(int64_t)sm.hot[row] * R + sm.cold[col]] * a.inv_eps;
                    v = exp_split(sm.alpha[row] + sm.beta[col] - c);
                }
                K[aa][g] = v;
            }
        }
    };
    build_tile();
    float uo = 1.0f;                 // committed u~ of row `rowl`
    int t = 1;
    int until_check = a.check_every; // iterations until the next tolerance test (tested when it reaches 1)
    float err_out = 0.0f;
    const float tol_abs_f = (float)tol_abs;
    // u~ and v~ must stay inside [e^-40, e^40]; for positive floats that is one unsigned compare on the bits
    // (negative, NaN and infinite values fall outside too)
    const uint32_t lo_bits = __float_as_uint(kDriftLo), span_bits = __float_as_uint(kDriftHi) - lo_bits;

    for (;;) {
        const int par = t & 1;
        // ================= half-step 1: r = K~ v~ (row sums of iterate t), u' = s~ / r
        float p[RPW];
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            float acc = K[aa][0] * vreg[0];
#pragma unroll
            for (int g = 1; g < CG; ++g) acc = fmaf(K[aa][g], vreg[g], acc);
            p[aa] = acc;
        }
        const float r = transpose_reduce<RPW>(p, lane);
        const float un = row_ok ? st_l * rcp_fast(r) : 1.0f;
        bool odd = (__float_as_uint(un) - lo_bits) > span_bits;       // out of range: fold, or hand back
        // ================= half-step 2 (speculative until the stop test): c = K~^T u', v' = d / c
        float cp[CG];
#pragma unroll
        for (int g = 0; g < CG; ++g) cp[g] = 0.0f;
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) {
            const float ua = __shfl_sync(kFull, un, aa);
#pragma unroll
            for (int g = 0; g < CG; ++g) cp[g] = fmaf(K[aa][g], ua, cp[g]);
        }
        // ---- the row sums belong to iterate t: is this where the solve stops?
        const bool last = t >= a.max_iters;
        const bool check = a.tol > 0.0f && until_check == 1;
        float err = 0.0f;
        if (last || check) {                                             // uniform over the block
            float e = row_owner ? fabsf(fmaf(uo, r, -st_l)) : 0.0f;
            for (int o = 16; o > 0; o >>= 1) e += __shfl_xor_sync(kFull, e, o);
            err = e;
        }
        float vnew[CG];
        if (NW == 1) {
#pragma unroll
            for (int g = 0; g < CG; ++g) {
                const float vn = col_ok[g] ? ddg[g] * rcp_fast(cp[g]) : 1.0f;
                odd |= (__float_as_uint(vn) - lo_bits) > span_bits;
                vnew[g] = vn;
            }
            odd = __any_sync(kFull, odd);
        } else {
#pragma unroll
            for (int g = 0; g < CG; ++g) sm.part[warp * RMAX + lane + 32 * g] = cp[g];
            if ((last || check) && lane == 0) sm.errw[warp] = err;
            if (odd) sm.flags[par] = 1;
            __syncthreads();
            if (last || check) {
                err = 0.0f;
#pragma unroll
                for (int w = 0; w < NW; ++w) err += sm.errw[w];
            }
            if (tid == 0) sm.flags[par ^ 1] = 0;
        }
        if (last || (check && err <= tol_abs_f)) {
            // a row sum outside the safe range makes this row error meaningless: let the other kernel redo it
            const bool bad_r = row_ok && !(r > kSumLo && r < kSumHi);
            if (NW == 1 ? __any_sync(kFull, bad_r) : __syncthreads_or(bad_r)) return false;
            err_out = (float)((double)err / sum_st);
            if (a.tol > 0.0f && !(err <= tol_abs_f)) info |= TAOT_INFO_SINKHORN_CAP;
            break;
        }
        if (NW > 1) {
            for (int j = tid; j < Cn; j += NT) {
                float c = 0.0f;
#pragma unroll
                for (int w = 0; w < NW; ++w) c += sm.part[w * RMAX + j];
                const float vn = sm.dd[j] * rcp_fast(c);
                if ((__float_as_uint(vn) - lo_bits) > span_bits) sm.flags[par] = 1;
                sm.vs[j] = vn;
            }
            __syncthreads();
            odd = sm.flags[par] != 0;
#pragma unroll
            for (int g = 0; g < CG; ++g) vnew[g] = col_ok[g] ? sm.vs[lane + 32 * g] : 1.0f;
        }
        if (odd) {
            // rare: either u~, v~ merely drifted (fold them into the potentials) or a sum left the range in which
            // fp32 products are trustworthy (hand the problem back).  Decide from the sums themselves.
            bool bad = row_ok && !(r > kSumLo && r < kSumHi);
            if (NW == 1) {
#pragma unroll
                for (int g = 0; g < CG; ++g) bad |= col_ok[g] && !(cp[g] > kSumLo && cp[g] < kSumHi);
                bad = __any_sync(kFull, bad);
            } else {
                for (int j = tid; j < Cn; j += NT) {
                    float c = 0.0f;
#pragma unroll
                    for (int w = 0; w < NW; ++w) c += sm.part[w * RMAX + j];
                    bad |= !(c > kSumLo && c < kSumHi);
                }
                bad = __syncthreads_or(bad);
            }
            if (bad) return false;
        }
        // ---- commit iteration t+1
        uo = un;
#pragma unroll
        for (int g = 0; g < CG; ++g) vreg[g] = vnew[g];
        ++t;
        until_check = until_check == 1 ? a.check_every : until_check - 1;
        if (odd) {
            // fold u~, v~ into the fp64 potentials and rebuild the tile around them
            if (row_owner) sm.alpha[rowl] += log((double)uo);
            if (NW == 1) {
#pragma unroll
                for (int g = 0; g < CG; ++g)
                    if (col_ok[g]) sm.beta[lane + 32 * g] += log((double)vreg[g]);
                __syncwarp();
            } else {
                for (int j = tid; j < Cn; j += NT) sm.beta[j] += log((double)sm.vs[j]);
                __syncthreads();
            }
            uo = 1.0f;
#pragma unroll
            for (int g = 0; g < CG; ++g) vreg[g] = 1.0f;
            build_tile();
            if (NW > 1) __syncthreads();
        }
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
    if (NW > 1) __syncthreads();
    if (row_owner) sm.alpha[rowl] += log((double)uo);
    if (warp == 0) {
#pragma unroll
        for (int g = 0; g < CG; ++g)
            if (col_ok[g]) sm.beta[lane + 32 * g] += log((double)vreg[g]);     // every warp holds the same v~
    }
    __syncthreads();
    build_tile();
    float cs[CG];
#pragma unroll
    for (int g = 0; g < CG; ++g) {
        float acc = 0.0f;
#pragma unroll
        for (int aa = 0; aa < RPW; ++aa) acc += K[aa][g];
        cs[g] = acc;
    }
    float fg[CG];
    if (NW == 1) {
#pragma unroll
        for (int g = 0; g < CG; ++g)
            fg[g] = col_ok[g] ? (float)fmin(1.0, (double)ddg[g] / ((double)cs[g] + (double)a.eps0)) : 0.0f;
    } else {
#pragma unroll
        for (int g = 0; g < CG; ++g) sm.part[warp * RMAX + lane + 32 * g] = cs[g];
        __syncthreads();
        for (int j = tid; j < Cn; j += NT) {
            double c = 0.0;
#pragma unroll
            for (int w = 0; w < NW; ++w) c += (double)sm.part[w * RMAX + j];
            sm.vs[j] = (float)fmin(1.0, (double)sm.dd[j] / (c + (double)a.eps0));
        }
        __syncthreads();
#pragma unroll
        for (int g = 0; g < CG; ++g) fg[g] = col_ok[g] ? sm.vs[lane + 32 * g] : 0.0f;
    }
    // zero the R x R block, then scatter the hot x cold entries
    for (int q = tid; q < R * R; q += NT) out[q] = 0.0f;
    __syncthreads();
    int nonfinite = 0;
#pragma unroll
    for (int aa = 0; aa < RPW; ++aa) {
        const int row = row0 + aa;
        if (row >= Hn) continue;
        float* orow = out + (int64_t)sm.hot[row] * R;
#pragma unroll
        for (int g = 0; g < CG; ++g) {
            if (!col_ok[g]) continue;
            const float val = K[aa][g] * fg[g];
            if (!isfinite(val)) nonfinite = 1;
            orow[sm.cold[lane + 32 * g]] = val;
        }
    }
    nonfinite = __syncthreads_or(nonfinite);
    if (nonfinite) info |= TAOT_INFO_NONFINITE;
    if (tid == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
    return true;
}

// One-warp variant with a two-dimensional lane grid: lane = (lr, lc) with 4 row lanes x 8 column lanes; the lane
// holds K~[ra][cg] for rows ra*4 + lr (ra < NRA) and columns cg*8 + lc (cg < NCG).  Row sums reduce over the 8
// column lanes (3 butterfly shuffles per ra), column sums over the 4 row lanes (2 shuffles per cg); after a
// butterfly every lane of the group holds the same bits, so u~ and v~ are computed redundantly where they are
// needed and nothing is broadcast.  For the small problems of the planner (a few supply ranks, tens of demand
// ranks) this is a much shorter dependent chain per iteration than one row set per lane.
template <int NRA, int NCG, int CG, bool TOL>
__device__ __forceinline__ bool grid_solve(const SinkArgs& a, TileSmem<1, CG>& sm, int Hn, int Cn, double sum_st,
                                           int info, float* out, int64_t b)
{
    constexpr int RL = 4, CL = 8;
    const int R = a.R, lane = threadIdx.x & 31;
    const int lr = lane >> 3, lc = lane & 7;
    const double tol_abs = (double)a.tol * sum_st;

    float K[NRA][NCG];
    float stl[NRA], uo[NRA], ddg[NCG], vreg[NCG];
    bool row_ok[NRA], col_ok[NCG];
#pragma unroll
    for (int ra = 0; ra < NRA; ++ra) {
        const int row = ra * RL + lr;
        row_ok[ra] = row < Hn;
        stl[ra] = row_ok[ra] ? sm.st[row] : 1.0f;
        uo[ra] = 1.0f;
    }
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) {
        const int col = cg * CL + lc;
        col_ok[cg] = col < Cn;
        ddg[cg] = col_ok[cg] ? sm.dd[col] : 1.0f;
        vreg[cg] = 1.0f;
    }
    // Tolerance mode builds the tile in straight-line code: entries off the problem's block are computed from clamped
    // indices and then zeroed, so that the independent exponentials of a lane overlap instead of running one after
    // another behind a branch each (config 3: a build of the tile 15 k -> 9 k cycles).  The fixed-count builds keep
    // the branchy form: the straight-line one costs 30-45 registers, which slowed their loops by 3-5 %.
    auto build_tile = [&]() {
        if (TOL) {
            double al[NRA], be[NCG];
            const float* crow[NRA];
            int ccol[NCG];
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) {
                const int row = ra * RL + lr, rc = row < Hn ? row : Hn - 1;
                al[ra] = sm.alpha[rc];
                crow[ra] = a.C + (int64_t)sm.hot[rc] * R;
            }
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg) {
                const int col = cg * CL + lc, cc = col < Cn ? col : Cn - 1;
                be[cg] = sm.beta[cc];
                ccol[cg] = sm.cold[cc];
            }
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) {
#pragma unroll
                for (int cg = 0; cg < NCG; ++cg) {
                    const double c = (double)crow[ra][ccol[cg]] * a.inv_eps;
                    const float v = exp_split(al[ra] + be[cg] - c);
                    K[ra][cg] = (row_ok[ra] && col_ok[cg]) ? v : 0.0f;
                }
            }
        } else {
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) {
                const int row = ra * RL + lr;
#pragma unroll
                for (int cg = 0; cg < NCG; ++cg) {
                    const int col = cg * CL + lc;
                    float v = 0.0f;
                    if (row < Hn && col < Cn) {
                        const double c = (double)a.C[(int64_t)sm.hot[row] * R + sm.cold[col]] * a.inv_eps;
                        v = exp_split(sm.alpha[row] + sm.beta[col] - c);
                    }
                    K[ra][cg] = v;
                }
            }
        }
    };
    build_tile();
    int t = 1;
    int until_check = a.check_every;
    float err_out = 0.0f;
    const float tol_abs_f = (float)tol_abs;
    const uint32_t lo_bits = __float_as_uint(kDriftLo), span_bits = __float_as_uint(kDriftHi) - lo_bits;
    float usave[NRA], vsave[NCG];    // tolerance mode: the iterate whose error is still to be tested
    bool pend = false, near_pend = false;
    float e_pend = 0.0f;
#pragma unroll
    for (int ra = 0; ra < NRA; ++ra) usave[ra] = 1.0f;
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) vsave[cg] = 1.0f;

    for (;;) {
        // Drift test on the u~, v~ this iteration STARTS from; the vote is issued here and consumed at the end of
        // the iteration, so neither it nor the branch it feeds sits on the dependent chain.  Acting one update
        // late is safe: a value that left [e^-40, e^40] is still far inside the fp32 range, and should an update
        // jump past that range after all, its sums leave (kSumLo, kSumHi) and the problem is handed back.
        bool odd = false;
#pragma unroll
        for (int ra = 0; ra < NRA; ++ra) odd |= (__float_as_uint(uo[ra]) - lo_bits) > span_bits;
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) odd |= (__float_as_uint(vreg[cg]) - lo_bits) > span_bits;
        // (tolerance mode up to 32 ranks: this vote is taken further down, in one ballot with the error shares)
        if (!(TOL && CG == 1)) odd = __any_sync(kFull, odd);
        // ================= half-step 1: r = K~ v~, u' = s~ / r
        float r[NRA], un[NRA];
        auto row_sums = [&]() {
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) {
                float acc = K[ra][0] * vreg[0];
#pragma unroll
                for (int cg = 1; cg < NCG; ++cg) acc = fmaf(K[ra][cg], vreg[cg], acc);
                r[ra] = acc;
            }
#pragma unroll
            for (int off = 1; off < CL; off <<= 1) {
#pragma unroll
                for (int ra = 0; ra < NRA; ++ra) r[ra] += __shfl_xor_sync(kFull, r[ra], off);
            }
        };
        row_sums();
#pragma unroll
        for (int ra = 0; ra < NRA; ++ra) un[ra] = row_ok[ra] ? stl[ra] * rcp_fast(r[ra]) : 1.0f;
        // ================= half-step 2 (speculative until the stop test): c = K~^T u', v' = d / c
        float cp[NCG], vnew[NCG];
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) {
            float acc = K[0][cg] * un[0];
#pragma unroll
            for (int ra = 1; ra < NRA; ++ra) acc = fmaf(K[ra][cg], un[ra], acc);
            cp[cg] = acc;
        }
        // tolerance mode: this lane's share of the error of iterate t (from the row sums just formed).  Up to 32
        // ranks (VOTE) the shares are not summed here: as long as one of them alone exceeds the tolerance the sum does
        // too (they are non-negative), and that is settled by one vote; the sum is formed only when no share does
        // (see below).  Beyond 32 ranks the sum is formed in the shuffle levels of the column sums (measured: the
        // vote costs the larger tiles more than it saves).
        constexpr bool VOTE = CG == 1;
        float e_loc = 0.0f;
        bool near_now = true;
        if (TOL) {
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) e_loc += row_ok[ra] ? fabsf(fmaf(uo[ra], r[ra], -stl[ra])) : 0.0f;
            if (VOTE) {
                // One ballot carries both votes: u~ is the same in the 8 column lanes of a row lane, v~ in the 4 row
                // lanes of a column lane and the error share in the 8 column lanes, so the lanes with lr + lc even
                // (every lr and every lc occurs among them) vote on the drift and the others on the error share.
                constexpr unsigned kDriftLanes = 0xAA55AA55u;
                const bool drift_lane = (kDriftLanes >> lane) & 1u;
                const unsigned votes = __ballot_sync(kFull, drift_lane ? odd : (e_loc > tol_abs_f));
                odd = (votes & kDriftLanes) != 0u;
                near_now = (votes & ~kDriftLanes) == 0u;
            }
        }
#pragma unroll
        for (int off = CL; off < 32; off <<= 1) {
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg) cp[cg] += __shfl_xor_sync(kFull, cp[cg], off);
            if (TOL && !VOTE) e_loc += __shfl_xor_sync(kFull, e_loc, off);
        }
        auto over_row_lanes = [&](float e) {
#pragma unroll
            for (int off = CL; off < 32; off <<= 1) e += __shfl_xor_sync(kFull, e, off);
            return e;                                                    // the same bits in every lane
        };
        // ---- the row sums belong to iterate t: is this where the solve stops?  The loop body is kept free of
        // branches (a lone warp pays dearly for each one) and the one branch it has never waits for this iteration's
        // error: in tolerance mode the error of iterate t is computed every iteration but TESTED one iteration later,
        // when it has long arrived; the iterate it belongs to is kept in registers and restored if the test passes.
        auto row_error = [&]() {
            float e = 0.0f;
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) e += row_ok[ra] ? fabsf(fmaf(uo[ra], r[ra], -stl[ra])) : 0.0f;
#pragma unroll
            for (int off = CL; off < 32; off <<= 1) e += __shfl_xor_sync(kFull, e, off);
            return e;                                                    // the same bits in every lane
        };
        auto rows_bad = [&]() {
            bool bad_r = false;
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) bad_r |= row_ok[ra] && !(r[ra] > kSumLo && r[ra] < kSumHi);
            return __any_sync(kFull, bad_r) != 0;
        };
        bool check_now = false;
        if (TOL) {
            check_now = until_check == 1;
            until_check = check_now ? a.check_every : until_check - 1;
        }
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) vnew[cg] = col_ok[cg] ? ddg[cg] * rcp_fast(cp[cg]) : 1.0f;
        // VOTE: no share of iterate t-1's error exceeded the tolerance; else: its error, already summed, met it
        const bool stop_maybe = TOL && pend && (VOTE ? near_pend : e_pend <= tol_abs_f);
        const bool last = t >= a.max_iters;
        if (stop_maybe | last | odd) {
            const bool stop_prev = stop_maybe && (VOTE ? over_row_lanes(e_pend) : e_pend) <= tol_abs_f;
            const float err_now = TOL ? (VOTE ? over_row_lanes(e_loc) : e_loc) : 0.0f;
            if (stop_prev) {
                // iterate t-1 met the tolerance: go back to it (its row sums are recomputed for the range check)
#pragma unroll
                for (int ra = 0; ra < NRA; ++ra) uo[ra] = usave[ra];
#pragma unroll
                for (int cg = 0; cg < NCG; ++cg) vreg[cg] = vsave[cg];
                --t;
                row_sums();
                const float err = row_error();
                if (rows_bad()) return false;
                err_out = (float)((double)err / sum_st);
                break;
            }
            if (last || (check_now && err_now <= tol_abs_f)) {
                // the iteration cap, or (only reached together with a drift event) a test that is due right now
                const float err = TOL ? err_now : row_error();
                if (rows_bad()) return false;
                err_out = (float)((double)err / sum_st);
                if (TOL && !(err <= tol_abs_f)) info |= TAOT_INFO_SINKHORN_CAP;
                break;
            }
            if (odd) {
            // rare: either u~, v~ merely drifted (fold them into the potentials) or a sum of this update left the
            // range in which fp32 products are trustworthy (hand the problem back)
            bool bad = false;
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) bad |= row_ok[ra] && !(r[ra] > kSumLo && r[ra] < kSumHi);
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg) bad |= col_ok[cg] && !(cp[cg] > kSumLo && cp[cg] < kSumHi);
            if (__any_sync(kFull, bad)) return false;
            // commit iteration t+1, fold u~, v~ into the fp64 potentials (one lane per row / column), rebuild the tile
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra)
                if (row_ok[ra] && lc == 0) sm.alpha[ra * RL + lr] += log((double)un[ra]);
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg)
                if (col_ok[cg] && lr == 0) sm.beta[cg * CL + lc] += log((double)vnew[cg]);
            __syncwarp();
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) uo[ra] = 1.0f;
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg) vreg[cg] = 1.0f;
            build_tile();
            pend = false;                        // the test of iterate t was settled above
            ++t;
            continue;
            }
            // neither: the shares of iterate t-1 were all small but their sum was not; carry on
        }
        // ---- commit iteration t+1; iterate t stays behind until its error has been tested
        if (TOL) {
            pend = check_now;
            near_pend = near_now;
            e_pend = e_loc;
#pragma unroll
            for (int ra = 0; ra < NRA; ++ra) usave[ra] = uo[ra];
#pragma unroll
            for (int cg = 0; cg < NCG; ++cg) vsave[cg] = vreg[cg];
        }
#pragma unroll
        for (int ra = 0; ra < NRA; ++ra) uo[ra] = un[ra];
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) vreg[cg] = vnew[cg];
        ++t;
    }

    // ---- T = diag(u) M diag(v) from the total potentials, then the column cap
#pragma unroll
    for (int ra = 0; ra < NRA; ++ra)
        if (row_ok[ra] && lc == 0) sm.alpha[ra * RL + lr] += log((double)uo[ra]);
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg)
        if (col_ok[cg] && lr == 0) sm.beta[cg * CL + lc] += log((double)vreg[cg]);
    __syncwarp();
    build_tile();
    float fg[NCG];
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) {
        float acc = 0.0f;
#pragma unroll
        for (int ra = 0; ra < NRA; ++ra) acc += K[ra][cg];
#pragma unroll
        for (int off = CL; off < 32; off <<= 1) acc += __shfl_xor_sync(kFull, acc, off);
        fg[cg] = col_ok[cg] ? (float)fmin(1.0, (double)ddg[cg] / ((double)acc + (double)a.eps0)) : 0.0f;
    }
    for (int q = lane; q < R * R; q += 32) out[q] = 0.0f;
    __syncwarp();
    int nonfinite = 0;
#pragma unroll
    for (int ra = 0; ra < NRA; ++ra) {
        if (!row_ok[ra]) continue;
        float* orow = out + (int64_t)sm.hot[ra * RL + lr] * R;
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) {
            if (!col_ok[cg]) continue;
            const float val = K[ra][cg] * fg[cg];
            if (!isfinite(val)) nonfinite = 1;
            orow[sm.cold[cg * CL + lc]] = val;
        }
    }
    if (__any_sync(kFull, nonfinite != 0)) info |= TAOT_INFO_NONFINITE;
    if (lane == 0) {
        a.iters[b] = t;
        a.row_err[b] = err_out;
        if (info) atomicOr(a.info + b, info);
    }
    return true;
}

// Picks the smallest lane-grid tile that holds the problem (one warp); false: hand the problem back.
template <int CG, bool TOL>
__device__ __forceinline__ bool grid_dispatch(const SinkArgs& a, TileSmem<1, CG>& sm, int Hn, int Cn, double sum_st,
                                              int info, float* out, int64_t b)
{
#define TAOT_GRID(NRA, NCG) grid_solve<NRA, NCG, CG, TOL>(a, sm, Hn, Cn, sum_st, info, out, b)
    if (CG == 1) {                     // up to 32 ranks
        if (Cn <= 16) {
            if (Hn <= 4) return TAOT_GRID(1, 2);
            if (Hn <= 8) return TAOT_GRID(2, 2);
            if (Hn <= 16) return TAOT_GRID(4, 2);
            return TAOT_GRID(8, 2);
        }
        if (Hn <= 4) return TAOT_GRID(1, 4);
        if (Hn <= 8) return TAOT_GRID(2, 4);
        if (Hn <= 16) return TAOT_GRID(4, 4);
        return TAOT_GRID(8, 4);
    } else {                           // up to 64 ranks: rows in steps of 4 (NRA), columns in steps of 16 (NCG = 4, 6, 8)
#define TAOT_GRID_ROWS(NCG)                                  \
        if (Hn <= 8) return TAOT_GRID(2, NCG);              \
        if (Hn <= 12) return TAOT_GRID(3, NCG);             \
        if (Hn <= 16) return TAOT_GRID(4, NCG);             \
        if (Hn <= 20) return TAOT_GRID(5, NCG);             \
        if (Hn <= 24) return TAOT_GRID(6, NCG);             \
        return TAOT_GRID(8, NCG);
        if (Cn <= 32) { TAOT_GRID_ROWS(4) }
        if (Cn <= 48) { TAOT_GRID_ROWS(6) }
        TAOT_GRID_ROWS(8)
#undef TAOT_GRID_ROWS
    }
#undef TAOT_GRID
}

// RP0 < RP1 < RP2: rows-per-warp variants; the smallest that holds the problem's supply ranks runs.
// MINB: CTAs per SM the compiler must make room for (register cap); 1 = no cap.  The capped builds serve large
// batches of small problems, where more resident warps matter more than the rarely used large tiles.
// TOLK (one-warp kernels): the kernel is built for tolerance mode or for a fixed iteration count, not both, so
// that neither loop carries the other's registers.
template <int NW, int CG, int RP0, int RP1, int RP2, bool TOLK>
__device__ __forceinline__ void tile_problem(const SinkArgs& a, TileSmem<NW, CG>& sm, const int64_t b)
{
    constexpr int NT = NW * 32;
    const int R = a.R, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (a.skip_solved && a.iters[b] != kHandBack) return;      // chained launch: only what an earlier kernel left

    // ---- supply scaling gamma = min(1, sum d / max(sum s, eps0)), compaction of supply / demand ranks
    {
        double ps = 0.0, pd = 0.0;
        for (int i = tid; i < R; i += NT) {
            const float sv = a.s[b * R + i], dv = a.d[b * R + i];
            ps += sv > 0.0f ? (double)sv : 0.0;
            pd += dv > 0.0f ? (double)dv : 0.0;
        }
        for (int o = 16; o > 0; o >>= 1) {
            ps += __shfl_xor_sync(kFull, ps, o);
            pd += __shfl_xor_sync(kFull, pd, o);
        }
        if (lane == 0) { sm.red[warp] = ps; sm.red[32 + warp] = pd; }
        if (tid < 4) sm.flags[tid] = 0;
        __syncthreads();
        if (tid == 0) {
            double S = 0.0, D = 0.0;
            for (int w = 0; w < NW; ++w) { S += sm.red[w]; D += sm.red[32 + w]; }
            sm.sum[0] = S; sm.sum[1] = D;
        }
        __syncthreads();
    }
    const double sum_s = sm.sum[0], sum_d = sm.sum[1];
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, (double)a.eps0));
    for (int i = tid; i < R; i += NT) {
        const float sv = a.s[b * R + i], dv = a.d[b * R + i];
        sm.sv[i] = sv > 0.0f ? (float)(gamma * (double)sv) : 0.0f;
        sm.dv[i] = dv > 0.0f ? dv : 0.0f;
    }
    __syncthreads();
    const int Hn = compact_positive(sm.sv, R, sm.hot, sm.hpos, sm.wcnt);
    const int Cn = compact_positive(sm.dv, R, sm.cold, sm.cpos, sm.wcnt);
    if (Hn > (NW == 1 ? 32 : NW * RP2)) {    // does not fit any tile: another kernel takes it
        if (tid == 0) a.iters[b] = kHandBack;
        return;
    }
    for (int i = tid; i < Hn; i += NT) sm.st[i] = sm.sv[sm.hot[i]];
    for (int j = tid; j < Cn; j += NT) sm.dd[j] = sm.dv[sm.cold[j]];
    __syncthreads();

    int info = 0;
    if (sum_s > sum_d) info |= TAOT_INFO_SUPPLY_SCALED;
    float* out = a.plan + b * (int64_t)R * R;
    if (Hn == 0 || Cn == 0) {
        for (int q = tid; q < R * R; q += NT) out[q] = 0.0f;
        if (tid == 0) {
            a.iters[b] = 0;
            a.row_err[b] = 0.0f;
            if (info) atomicOr(a.info + b, info);
        }
        return;
    }
    double sum_st = 0.0;
    for (int i = 0; i < Hn; ++i) sum_st += (double)sm.st[i];          // same order in every thread

    // ---- iteration 1 in the log domain (v = 1 on every rank): phi = log s~ - LSE_j(-C_ij/eps) over all j,
    //      psi_j = log d_j - LSE_i(phi_i - C_ij/eps)
    for (int i = tid; i < Hn; i += NT) sm.phin[i] = log((double)sm.st[i]) - a.rowlse0[sm.hot[i]];
    __syncthreads();
    for (int j = tid; j < Cn; j += NT) {
        const int cj = sm.cold[j];
        double mx = -INFINITY;
        for (int i = 0; i < Hn; ++i) {
            const double x = sm.phin[i] - (double)a.C[(int64_t)sm.hot[i] * R + cj] * a.inv_eps;
            mx = x > mx ? x : mx;
        }
        double acc = 0.0;
        for (int i = 0; i < Hn; ++i)
            acc += (double)exp_split(sm.phin[i] - (double)a.C[(int64_t)sm.hot[i] * R + cj] * a.inv_eps - mx);
        sm.beta[j] = log((double)sm.dd[j]) - (mx + log(acc));
    }
    for (int i = tid; i < Hn; i += NT) sm.alpha[i] = sm.phin[i];
    __syncthreads();

    bool done;
    if constexpr (NW == 1) {
        done = grid_dispatch<CG, TOLK>(a, sm, Hn, Cn, sum_st, info, out, b);
    }
    else if (Hn <= NW * RP0) done = tile_solve<NW, RP0, CG>(a, sm, Hn, Cn, sum_st, info, out, b);
    else if (Hn <= NW * RP1) done = tile_solve<NW, RP1, CG>(a, sm, Hn, Cn, sum_st, info, out, b);
    else done = tile_solve<NW, RP2, CG>(a, sm, Hn, Cn, sum_st, info, out, b);
    if (!done && tid == 0) a.iters[b] = kHandBack;
}

template <int NW, int CG, int RP0, int RP1, int RP2, int MINB, bool TOLK = false>
__global__ void __launch_bounds__(NW * 32, MINB)
sinkhorn_tile_kernel(SinkArgs a, int64_t nprob)
{
    __shared__ TileSmem<NW, CG> sm;
    // one problem per CTA (a stride loop over the problems with a grid sized to the SMs was measured slower: the
    // set-up and write-out of one problem no longer overlap the iterations of the CTAs next to it)
    if ((int64_t)blockIdx.x < nprob) tile_problem<NW, CG, RP0, RP1, RP2, TOLK>(a, sm, (int64_t)blockIdx.x);
}

}  // namespace
