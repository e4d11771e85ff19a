/*
 * TAOT replica-placement planner -- CPU ORACLE.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the planner computes, written from the
 * paper's definitions and algorithms so that a reader can check it against them by eye.  It
 * shares no code with the CUDA library: no common header, helper, table or constant.  Only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it; the product path
 * never does.
 *
 * Floating point: the Sinkhorn solve is fp64 throughout.  The Phase-2 and Phase-3 scores,
 * which decide integer outcomes, are fp32 with one IEEE operation per line (compile with
 * -ffp-contract=off) so that a GPU evaluating the same expression gets the same bits.
 *
 * Notation (Method, Problem Formulation / Appendix A.1): R ranks, E experts, home(e) = e2r[e],
 * K guest slots per rank, S = R*K slots with slot s = r*K + kappa living on rank r = s / K,
 * T tokens per layer laid out so that source rank src(t) = t / (T/R), router top-k = k.
 *
 * Pinning status: every function below is pinned by tests/test_oracle_*.py against something
 * other than itself (closed forms, invariants, library routines, brute force, a hand trace).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Load collection (Appendix A.1, the definitions of n_re and l_r):
 *   n[l][r][e]        = number of (token, choice) pairs of source rank r routed to expert e
 *   expert_load[l][e] = sum_r n[l][r][e]
 *   rank_load[l][r]   = sum over experts homed on r of expert_load
 * An index outside [0, E) is counted in bad[l] and otherwise ignored.
 */
void oracle_histogram(const int32_t* topk, int32_t L, int64_t T, int32_t k, int32_t R, int32_t E,
                      const int32_t* e2r, int32_t* n, int32_t* expert_load, int32_t* rank_load,
                      int64_t* bad)
{
    const int64_t tpr = T / R;
    memset(n, 0, sizeof(int32_t) * (size_t)L * R * E);
    memset(expert_load, 0, sizeof(int32_t) * (size_t)L * E);
    memset(rank_load, 0, sizeof(int32_t) * (size_t)L * R);
    for (int32_t l = 0; l < L; ++l) {
        bad[l] = 0;
        for (int64_t t = 0; t < T; ++t) {
            const int64_t r = t / tpr;
            for (int32_t j = 0; j < k; ++j) {
                const int32_t e = topk[((int64_t)l * T + t) * k + j];
                if (e < 0 || e >= E) { bad[l]++; continue; }
                n[((int64_t)l * R + r) * E + e]++;
            }
        }
        for (int32_t e = 0; e < E; ++e) {
            int32_t tot = 0;
            for (int32_t r = 0; r < R; ++r) tot += n[((int64_t)l * R + r) * E + e];
            expert_load[(int64_t)l * E + e] = tot;
            rank_load[(int64_t)l * R + e2r[e]] += tot;
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Excess / spare against the mean load (Appendix A.1).  The mean is the INTEGER mean
 * floor(sum_r l_r / R): the paper's supply-scaling safeguard exists because of "integer mean
 * loads", so sum(excess) - sum(spare) = (sum l) mod R >= 0.
 */
void oracle_excess_spare(const int32_t* rank_load, int32_t L, int32_t R,
                         int64_t* mean, int32_t* excess, int32_t* spare)
{
    for (int32_t l = 0; l < L; ++l) {
        int64_t tot = 0;
        for (int32_t r = 0; r < R; ++r) tot += rank_load[(int64_t)l * R + r];
        const int64_t m = tot / R;
        mean[l] = m;
        for (int32_t r = 0; r < R; ++r) {
            const int64_t lr = rank_load[(int64_t)l * R + r];
            excess[(int64_t)l * R + r] = (int32_t)(lr > m ? lr - m : 0);
            spare[(int64_t)l * R + r] = (int32_t)(m > lr ? m - lr : 0);
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Phase 1: entropic OT by Sinkhorn-Knopp (Appendix A.2).
 *
 * The paper iterates u = s~/(M v), v = d/(M^T u) with M = exp(-W/eps) and T = diag(u) M diag(v).
 * Here the same iterates are carried as logarithms, phi = log u, psi = log v:
 *     phi_i = log s~_i - LSE_j(psi_j - W_ij/eps),   psi_j = log d_j - LSE_i(phi_i - W_ij/eps)
 * which is the identical sequence in exact arithmetic and cannot under- or overflow.
 * Start: v = 1 on every rank (psi = 0), u updated first.  A rank with s~_i = 0 has u_i = 0
 * (phi_i = -inf); a rank with d_j = 0 has v_j = 0 from its first update on.
 * s, d, C and eps arrive as fp32 (the library's interface types) and are promoted exactly.
 */
static double lse_skip_inf(const double* x, int32_t n)
{
    double mx = -INFINITY;
    for (int32_t i = 0; i < n; ++i) if (x[i] > mx) mx = x[i];
    if (mx == -INFINITY) return -INFINITY;
    double acc = 0.0;
    for (int32_t i = 0; i < n; ++i) if (x[i] != -INFINITY) acc += exp(x[i] - mx);
    return mx + log(acc);
}

/* Row-marginal violation of the current plan, relative to total (scaled) supply. */
static double row_violation(const double* phi, const double* psi, const double* Chat,
                            const double* st, double sum_st, int32_t R)
{
    double err = 0.0;
    for (int32_t i = 0; i < R; ++i) {
        double rs = 0.0;
        if (phi[i] != -INFINITY)
            for (int32_t j = 0; j < R; ++j)
                if (psi[j] != -INFINITY) rs += exp(phi[i] + psi[j] - Chat[(int64_t)i * R + j]);
        err += fabs(rs - st[i]);
    }
    return err / sum_st;
}

/*
 * max_iters iterations if tol <= 0; otherwise stop after the first iteration t (t a multiple
 * of check_every) whose row violation is <= tol, or at max_iters.  err_hist (nullable, length
 * max_iters) receives the row violation after every iteration.  The column-cap safeguard
 * T_ij *= min(1, d_j / (sum_i T_ij + eps0)) is applied to the returned plan.
 * Returns 0, or 1 if the cap was reached above tol in tolerance mode.
 */
int32_t oracle_sinkhorn(const float* s32, const float* d32, int32_t R, const float* C32, float eps32,
                        float eps0_32, int32_t max_iters, double tol, int32_t check_every,
                        double* plan, int32_t* n_iter, double* row_err, double* err_hist)
{
    const double eps = (double)eps32, eps0 = (double)eps0_32;
    double* Chat = (double*)malloc(sizeof(double) * (size_t)R * R);
    double* st = (double*)malloc(sizeof(double) * R);
    double* d = (double*)malloc(sizeof(double) * R);
    double* lst = (double*)malloc(sizeof(double) * R);
    double* ld = (double*)malloc(sizeof(double) * R);
    double* phi = (double*)malloc(sizeof(double) * R);
    double* psi = (double*)malloc(sizeof(double) * R);
    double* tmp = (double*)malloc(sizeof(double) * R);
    int32_t status = 0;

    for (int64_t q = 0; q < (int64_t)R * R; ++q) Chat[q] = (double)C32[q] / eps;

    /* supply scaling gamma = min(1, sum d / max(sum s, eps0)) */
    double sum_s = 0.0, sum_d = 0.0;
    for (int32_t i = 0; i < R; ++i) { sum_s += (double)s32[i]; sum_d += (double)d32[i]; }
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, eps0));
    double sum_st = 0.0;
    for (int32_t i = 0; i < R; ++i) {
        st[i] = gamma * (double)s32[i];
        d[i] = (double)d32[i];
        sum_st += st[i];
        lst[i] = st[i] > 0.0 ? log(st[i]) : -INFINITY;
        ld[i] = d[i] > 0.0 ? log(d[i]) : -INFINITY;
    }
    memset(plan, 0, sizeof(double) * (size_t)R * R);
    *n_iter = 0;
    *row_err = 0.0;
    if (!(sum_st > 0.0) || !(sum_d > 0.0)) goto done;   /* nothing to move */

    for (int32_t j = 0; j < R; ++j) psi[j] = 0.0;        /* v = 1 */
    for (int32_t i = 0; i < R; ++i) phi[i] = -INFINITY;
    int32_t t = 0;
    double err = INFINITY;
    while (t < max_iters) {
        ++t;
        for (int32_t i = 0; i < R; ++i) {                /* u = s~ / (M v) */
            if (lst[i] == -INFINITY) { phi[i] = -INFINITY; continue; }
            for (int32_t j = 0; j < R; ++j)
                tmp[j] = psi[j] == -INFINITY ? -INFINITY : psi[j] - Chat[(int64_t)i * R + j];
            phi[i] = lst[i] - lse_skip_inf(tmp, R);
        }
        for (int32_t j = 0; j < R; ++j) {                /* v = d / (M^T u) */
            if (ld[j] == -INFINITY) { psi[j] = -INFINITY; continue; }
            for (int32_t i = 0; i < R; ++i)
                tmp[i] = phi[i] == -INFINITY ? -INFINITY : phi[i] - Chat[(int64_t)i * R + j];
            psi[j] = ld[j] - lse_skip_inf(tmp, R);
        }
        const int check = tol > 0.0 && (t % check_every == 0);
        if (check || err_hist != NULL || t == max_iters)
            err = row_violation(phi, psi, Chat, st, sum_st, R);
        if (err_hist) err_hist[t - 1] = err;
        if (check && err <= tol) break;
    }
    /* the loop leaves either at a check or at t == max_iters: err belongs to iteration t */
    *n_iter = t;
    *row_err = (t > 0) ? err : 0.0;
    if (tol > 0.0 && err > tol) status = 1;

    /* T = diag(u) M diag(v), then the column cap */
    for (int32_t i = 0; i < R; ++i)
        for (int32_t j = 0; j < R; ++j)
            if (phi[i] != -INFINITY && psi[j] != -INFINITY)
                plan[(int64_t)i * R + j] = exp(phi[i] + psi[j] - Chat[(int64_t)i * R + j]);
    for (int32_t j = 0; j < R; ++j) {
        double cs = 0.0;
        for (int32_t i = 0; i < R; ++i) cs += plan[(int64_t)i * R + j];
        const double f = fmin(1.0, d[j] / (cs + eps0));
        for (int32_t i = 0; i < R; ++i) plan[(int64_t)i * R + j] *= f;
    }
done:
    free(Chat); free(st); free(d); free(lst); free(ld); free(phi); free(psi); free(tmp);
    return status;
}

/*
 * The same solve written exactly as the paper prints it: Gibbs kernel M and scaling vectors
 * (u, v) in fp64, an iteration count given in advance, no logarithms.  Valid only while exp(-W/eps)
 * does not underflow; used to cross-check the log-domain routine above.
 */
void oracle_sinkhorn_gibbs(const float* s32, const float* d32, int32_t R, const float* C32,
                           float eps32, float eps0_32, int32_t iters, double* plan)
{
    const double eps = (double)eps32, eps0 = (double)eps0_32;
    double* M = (double*)malloc(sizeof(double) * (size_t)R * R);
    double* u = (double*)calloc(R, sizeof(double));
    double* v = (double*)malloc(sizeof(double) * R);
    double sum_s = 0.0, sum_d = 0.0;
    for (int64_t q = 0; q < (int64_t)R * R; ++q) M[q] = exp(-(double)C32[q] / eps);
    for (int32_t i = 0; i < R; ++i) { sum_s += (double)s32[i]; sum_d += (double)d32[i]; }
    const double gamma = fmin(1.0, sum_d / fmax(sum_s, eps0));
    memset(plan, 0, sizeof(double) * (size_t)R * R);
    if (sum_s > 0.0 && sum_d > 0.0) {
        for (int32_t j = 0; j < R; ++j) v[j] = 1.0;
        for (int32_t t = 0; t < iters; ++t) {
            for (int32_t i = 0; i < R; ++i) {
                double mv = 0.0;
                for (int32_t j = 0; j < R; ++j) mv += M[(int64_t)i * R + j] * v[j];
                const double si = gamma * (double)s32[i];
                u[i] = si > 0.0 ? si / mv : 0.0;
            }
            for (int32_t j = 0; j < R; ++j) {
                double mu = 0.0;
                for (int32_t i = 0; i < R; ++i) mu += M[(int64_t)i * R + j] * u[i];
                v[j] = (double)d32[j] > 0.0 ? (double)d32[j] / mu : 0.0;
            }
        }
        if (iters > 0)
            for (int32_t i = 0; i < R; ++i)
                for (int32_t j = 0; j < R; ++j)
                    plan[(int64_t)i * R + j] = u[i] * M[(int64_t)i * R + j] * v[j];
        for (int32_t j = 0; j < R; ++j) {
            double cs = 0.0;
            for (int32_t i = 0; i < R; ++i) cs += plan[(int64_t)i * R + j];
            const double f = fmin(1.0, (double)d32[j] / (cs + eps0));
            for (int32_t i = 0; i < R; ++i) plan[(int64_t)i * R + j] *= f;
        }
    }
    free(M); free(u); free(v);
}

/* ------------------------------------------------------------------------------------------
 * Topology preference derived from the cost matrix when the caller supplies none
 * (Appendix A.3: 1 intra-node, w_inter < 1 inter-node, 0 for the home rank):
 *   B_ii = 0;  B_ij = min(1, c_min / C_ij) with c_min the smallest positive off-diagonal cost
 * (fp32 divide), and 1 where C_ij <= 0.
 */
void oracle_default_preference(const float* C, int32_t R, float* B)
{
    float cmin = INFINITY;
    for (int32_t i = 0; i < R; ++i)
        for (int32_t j = 0; j < R; ++j)
            if (i != j && C[(int64_t)i * R + j] > 0.0f && C[(int64_t)i * R + j] < cmin)
                cmin = C[(int64_t)i * R + j];
    for (int32_t i = 0; i < R; ++i)
        for (int32_t j = 0; j < R; ++j) {
            const float c = C[(int64_t)i * R + j];
            float b;
            if (i == j) b = 0.0f;
            else if (!(c > 0.0f) || cmin == INFINITY) b = 1.0f;
            else { b = cmin / c; if (b > 1.0f) b = 1.0f; }
            B[(int64_t)i * R + j] = b;
        }
}

/* ------------------------------------------------------------------------------------------
 * Spill by cumulative-excess differencing (Appendix A.3, the two equations before the score):
 * within each rank sort its experts ascending by (load, index); sigma_k = max(cum_k - mean, 0);
 * spill of the k-th = sigma_k - sigma_{k-1}.
 */
void oracle_spill(const int32_t* expert_load, const int32_t* e2r, int32_t R, int32_t E,
                  int64_t mean, int32_t* spill)
{
    int32_t* mine = (int32_t*)malloc(sizeof(int32_t) * E);
    for (int32_t e = 0; e < E; ++e) spill[e] = 0;
    for (int32_t r = 0; r < R; ++r) {
        int32_t cnt = 0;
        for (int32_t e = 0; e < E; ++e) if (e2r[e] == r) mine[cnt++] = e;
        /* insertion sort, ascending by (load, index); 'mine' starts index-ascending so it is stable */
        for (int32_t a = 1; a < cnt; ++a) {
            const int32_t x = mine[a];
            int32_t b = a - 1;
            while (b >= 0 && expert_load[mine[b]] > expert_load[x]) { mine[b + 1] = mine[b]; --b; }
            mine[b + 1] = x;
        }
        int64_t cum = 0, sigma_prev = 0;
        for (int32_t a = 0; a < cnt; ++a) {
            cum += expert_load[mine[a]];
            const int64_t sigma = cum > mean ? cum - mean : 0;
            spill[mine[a]] = (int32_t)(sigma - sigma_prev);
            sigma_prev = sigma;
        }
    }
    free(mine);
}

/* ------------------------------------------------------------------------------------------
 * Phase 2: column-priority iterative matching (Appendix A.3, Algorithm 2), one layer.
 *
 * score_er = min(spill_e, spare_r) + alpha * B[home(e)][r] + 0.1 alpha * T[home(e)][r] / max(excess_home(e), eps0)
 * with alpha = mean * R / E, all in fp32, one rounding per operation, in exactly this order.
 * A pair is a candidate unless r is e's home, e already sits on r, r was matched in this outer
 * round, spare_r <= 0 or spill_e <= 0.  Every rank with a candidate takes its best expert
 * (ties: lowest e); every expert chosen by several ranks keeps the best of them (ties: lowest
 * r); winners are applied together.  The inner loop ends when no candidate is left, which is
 * what the paper's fixed |C| inner rounds reach as well (later rounds would change nothing).
 * Output: slot_expert[r*K+kappa] (-1 = empty), slot_tokens[r*K+kappa]; spill/spare are updated
 * in place to their residuals.
 */
void oracle_match(int32_t R, int32_t E, int32_t K, const int32_t* e2r, int64_t mean,
                  const int32_t* excess, int32_t* spill, int32_t* spare, const float* B,
                  const float* plan, float eps0, int32_t* slot_expert, int32_t* slot_tokens,
                  int32_t* inner_rounds)
{
    const float alpha = (float)(mean * (int64_t)R) / (float)E;
    const float beta = 0.1f * alpha;
    uint8_t* U = (uint8_t*)calloc((size_t)E * R, 1);
    uint8_t* matched = (uint8_t*)malloc(R);
    int32_t* estar = (int32_t*)malloc(sizeof(int32_t) * R);
    float* best = (float*)malloc(sizeof(float) * R);
    int32_t* rstar = (int32_t*)malloc(sizeof(int32_t) * E);
    int32_t rounds = 0;
    for (int32_t s = 0; s < R * K; ++s) { slot_expert[s] = -1; slot_tokens[s] = 0; }

    for (int32_t kappa = 0; kappa < K; ++kappa) {
        memset(matched, 0, R);
        for (;;) {
            /* Steps 1-2: every rank's best candidate expert */
            int any = 0;
            for (int32_t r = 0; r < R; ++r) {
                estar[r] = -1;
                best[r] = 0.0f;
                if (matched[r] || spare[r] <= 0) continue;
                for (int32_t e = 0; e < E; ++e) {
                    const int32_t h = e2r[e];
                    if (h == r || U[(int64_t)e * R + r] || spill[e] <= 0) continue;
                    const int32_t gain = spill[e] < spare[r] ? spill[e] : spare[r];
                    float ex = (float)excess[h];
                    if (ex < eps0) ex = eps0;
                    const float tn = plan[(int64_t)h * R + r] / ex;
                    const float t1 = alpha * B[(int64_t)h * R + r];
                    const float t2 = beta * tn;
                    float sc = (float)gain + t1;
                    sc = sc + t2;
                    if (estar[r] < 0 || sc > best[r]) { estar[r] = e; best[r] = sc; }
                }
                if (estar[r] >= 0) any = 1;
            }
            if (!any) break;
            ++rounds;
            /* Step 3: arbitration, best rank per chosen expert */
            for (int32_t e = 0; e < E; ++e) rstar[e] = -1;
            for (int32_t r = 0; r < R; ++r) {
                const int32_t e = estar[r];
                if (e < 0) continue;
                if (rstar[e] < 0 || best[r] > best[rstar[e]]) rstar[e] = r;
            }
            /* Step 4: apply all winners */
            for (int32_t e = 0; e < E; ++e) {
                const int32_t r = rstar[e];
                if (r < 0) continue;
                const int32_t g = spill[e] < spare[r] ? spill[e] : spare[r];
                spill[e] -= g;
                spare[r] -= g;
                U[(int64_t)e * R + r] = 1;
                matched[r] = 1;
                slot_expert[r * K + kappa] = e;
                slot_tokens[r * K + kappa] = g;
            }
        }
    }
    if (inner_rounds) *inner_rounds = rounds;
    free(U); free(matched); free(estar); free(best); free(rstar);
}

/* ------------------------------------------------------------------------------------------
 * Phase 3: Lagrangian auction (Appendix A.4, Algorithm 3), one layer.
 *
 * Each round: every slot with tokens still to collect bids for the source rank r that still
 * holds tokens of its expert and maximises B3[r][rank(slot)] - price_r (ties: lowest r); every
 * rank that received bids serves the best one (ties: lowest slot) with
 * x = min(n_r,e, A_slot); a rank that served x > 0 gets dearer by one price step.
 * B3 is the topology bonus: B off the diagonal, 1 on it (a source rank is intra-node with
 * itself).  price_r is kept as price_step * wins_r, a single fp32 product.
 * max_rounds <= 0 runs to completion (at most R*S + S rounds are ever productive).
 * X[r*S + s] receives the tokens rank r sends to slot s.  Returns the residual sum of A.
 */
int64_t oracle_auction(int32_t R, int32_t E, int32_t K, const int32_t* n /*[R,E]*/,
                       const int32_t* slot_expert, const int32_t* slot_tokens, const float* B,
                       float price_step, int32_t max_rounds, int32_t* X, int32_t* rounds_out)
{
    const int32_t S = R * K;
    int32_t* nrem = (int32_t*)malloc(sizeof(int32_t) * (size_t)R * E);
    int32_t* A = (int32_t*)malloc(sizeof(int32_t) * S);
    int32_t* wins = (int32_t*)calloc(R, sizeof(int32_t));
    int32_t* rstar = (int32_t*)malloc(sizeof(int32_t) * S);
    float* bid = (float*)malloc(sizeof(float) * S);
    int32_t* sstar = (int32_t*)malloc(sizeof(int32_t) * R);
    memcpy(nrem, n, sizeof(int32_t) * (size_t)R * E);
    memcpy(A, slot_tokens, sizeof(int32_t) * S);
    memset(X, 0, sizeof(int32_t) * (size_t)R * S);
    const int64_t cap = (int64_t)R * S + S;
    int32_t rounds = 0;
    for (;;) {
        if (max_rounds > 0 && rounds >= max_rounds) break;
        if ((int64_t)rounds >= cap) break;
        /* Step 1: slots bid */
        int any = 0;
        for (int32_t s = 0; s < S; ++s) {
            rstar[s] = -1;
            bid[s] = 0.0f;
            const int32_t e = slot_expert[s];
            if (e < 0 || A[s] <= 0) continue;
            const int32_t host = s / K;
            for (int32_t r = 0; r < R; ++r) {
                if (nrem[(int64_t)r * E + e] <= 0) continue;
                const float b3 = (r == host) ? 1.0f : B[(int64_t)r * R + host];
                const float price = price_step * (float)wins[r];
                const float sc = b3 - price;
                if (rstar[s] < 0 || sc > bid[s]) { rstar[s] = r; bid[s] = sc; }
            }
            if (rstar[s] >= 0) any = 1;
        }
        if (!any) break;
        ++rounds;
        /* Step 2: ranks serve their best bidder */
        for (int32_t r = 0; r < R; ++r) sstar[r] = -1;
        for (int32_t s = 0; s < S; ++s) {
            const int32_t r = rstar[s];
            if (r < 0) continue;
            if (sstar[r] < 0 || bid[s] > bid[sstar[r]]) sstar[r] = s;
        }
        /* Steps 3-4: allocate and update */
        for (int32_t r = 0; r < R; ++r) {
            const int32_t s = sstar[r];
            if (s < 0) continue;
            const int32_t e = slot_expert[s];
            const int32_t have = nrem[(int64_t)r * E + e];
            const int32_t x = have < A[s] ? have : A[s];
            X[(int64_t)r * S + s] += x;
            nrem[(int64_t)r * E + e] -= x;
            A[s] -= x;
            if (x > 0) wins[r]++;
        }
    }
    int64_t residual = 0;
    for (int32_t s = 0; s < S; ++s) if (slot_expert[s] >= 0) residual += A[s];
    if (rounds_out) *rounds_out = rounds;
    free(nrem); free(A); free(wins); free(rstar); free(bid); free(sstar);
    return residual;
}

/* ------------------------------------------------------------------------------------------
 * Token reassignment given the schedule (Problem Formulation: the paper gives the counts X and
 * no per-token rule; the rule here is: earliest tokens move first, lowest slot fills first).
 * Walk one layer's routing table in flat order q = t*k + j.  For source rank r = src(t) and
 * expert e = topk[q], let ord be the number of earlier entries of the same (r, e).  The slots
 * holding e, in ascending slot order s_1 < s_2 < ..., take the first X[r][s_1] such entries,
 * the next X[r][s_2], and so on; an entry beyond them keeps e.  A moved entry is rewritten
 * to E + s.  Out-of-range indices are copied unchanged.
 */
void oracle_assign(const int32_t* topk, int64_t T, int32_t k, int32_t R, int32_t E, int32_t K,
                   const int32_t* slot_expert, const int32_t* X, int32_t* new_idx)
{
    const int32_t S = R * K;
    const int64_t tpr = T / R;
    int64_t* ord = (int64_t*)malloc(sizeof(int64_t) * E);
    for (int32_t r = 0; r < R; ++r) {
        for (int32_t e = 0; e < E; ++e) ord[e] = 0;
        for (int64_t t = (int64_t)r * tpr; t < (int64_t)(r + 1) * tpr; ++t) {
            for (int32_t j = 0; j < k; ++j) {
                const int64_t q = t * k + j;
                const int32_t e = topk[q];
                if (e < 0 || e >= E) { new_idx[q] = e; continue; }
                const int64_t o = ord[e]++;
                int64_t cum = 0;
                int32_t target = e;
                for (int32_t s = 0; s < S; ++s) {
                    if (slot_expert[s] != e) continue;
                    cum += X[(int64_t)r * S + s];
                    if (o < cum) { target = E + s; break; }
                }
                new_idx[q] = target;
            }
        }
    }
    free(ord);
}

/* ------------------------------------------------------------------------------------------
 * Dispatch report of one layer (Appendix B.3, the four-part per-layer diagnostics; Evaluation,
 * the metric definitions: imbalance, intra-/inter-node transfers, weighted cost at 1 : lambda).
 *
 *   part 1  loads before: rank_load, expert_load; hot ranks (l_r above the mean), hot experts
 *           (positive spill, i.e. the experts Phase 2 may clone); spill is returned per expert
 *   part 2  cloning plan: per slot the tokens rerouted to it (column sum of X) and the kind of
 *           copy, from the home rank of its expert to the rank of the slot:
 *             0 empty, 1 intra-node (B[home][host] >= 1), 2 inter-node, 3 home rank itself;
 *           counts of each kind; weighted cost intra + lambda * inter, and sum of C[home][host]
 *   part 3  projected load: l'_r = l_r - tokens leaving r's home experts + tokens entering r's slots
 *   part 4  rho = (max_r l_r - mean) / mean with mean = total / R (Problem Formulation), before
 *           and after; largest absolute deviation from the mean as a fraction, before and after;
 *           peak-load reduction (max before - max after) / max before; fraction rerouted.
 * Ratios are fp64, one IEEE operation each; a zero denominator gives 0.
 *
 * ints[14]: total, rerouted, floor mean, max before, min before, max after, min after, hot ranks,
 *           cold ranks, hot experts, clones, intra, inter, same-rank
 * reals[8]: rho before, rho after, deviation before, deviation after, peak reduction,
 *           fraction rerouted, cost at 1:lambda, cost by C
 */
void oracle_report(int32_t R, int32_t E, int32_t K, const int32_t* e2r, const float* C, const float* B,
                   const int32_t* expert_load, const int32_t* rank_load, const int32_t* slot_expert,
                   const int32_t* X, double lambda, int32_t* spill, int32_t* load_after,
                   int32_t* slot_moved, int32_t* slot_kind, int64_t* ints, double* reals)
{
    const int32_t S = R * K;
    int64_t total = 0;
    for (int32_t r = 0; r < R; ++r) total += rank_load[r];
    const int64_t mfloor = total / R;
    const double mean = (double)total / (double)R;

    /* part 1 */
    oracle_spill(expert_load, e2r, R, E, mfloor, spill);
    int64_t hot_ranks = 0, cold_ranks = 0, hot_experts = 0;
    int64_t max_b = rank_load[0], min_b = rank_load[0];
    for (int32_t r = 0; r < R; ++r) {
        if (rank_load[r] > mfloor) ++hot_ranks;
        if (rank_load[r] < mfloor) ++cold_ranks;
        if (rank_load[r] > max_b) max_b = rank_load[r];
        if (rank_load[r] < min_b) min_b = rank_load[r];
    }
    for (int32_t e = 0; e < E; ++e) if (spill[e] > 0) ++hot_experts;

    /* part 2 */
    int64_t rerouted = 0, clones = 0, intra = 0, inter = 0, same = 0;
    double cost_C = 0.0;
    for (int32_t s = 0; s < S; ++s) {
        int64_t moved = 0;
        for (int32_t r = 0; r < R; ++r) moved += X[(int64_t)r * S + s];
        slot_moved[s] = (int32_t)moved;
        rerouted += moved;
        const int32_t e = slot_expert[s];
        if (e < 0) { slot_kind[s] = 0; continue; }
        const int32_t home = e2r[e], host = s / K;
        ++clones;
        if (home == host) { slot_kind[s] = 3; ++same; }
        else if (B[(int64_t)home * R + host] >= 1.0f) { slot_kind[s] = 1; ++intra; }
        else { slot_kind[s] = 2; ++inter; }
        cost_C = cost_C + (double)C[(int64_t)home * R + host];
    }
    const double linter = lambda * (double)inter;
    const double cost_ratio = (double)intra + linter;

    /* part 3 */
    for (int32_t r = 0; r < R; ++r) load_after[r] = rank_load[r];
    for (int32_t s = 0; s < S; ++s) {
        const int32_t e = slot_expert[s];
        if (e < 0) continue;
        load_after[e2r[e]] -= slot_moved[s];
        load_after[s / K] += slot_moved[s];
    }
    int64_t max_a = load_after[0], min_a = load_after[0];
    for (int32_t r = 0; r < R; ++r) {
        if (load_after[r] > max_a) max_a = load_after[r];
        if (load_after[r] < min_a) min_a = load_after[r];
    }

    /* part 4 */
    double rho_b = 0.0, rho_a = 0.0, dev_b = 0.0, dev_a = 0.0, peak = 0.0, frac = 0.0;
    if (mean > 0.0) {
        const double up_b = (double)max_b - mean, dn_b = mean - (double)min_b;
        const double up_a = (double)max_a - mean, dn_a = mean - (double)min_a;
        rho_b = up_b / mean;
        rho_a = up_a / mean;
        dev_b = (up_b > dn_b ? up_b : dn_b) / mean;
        dev_a = (up_a > dn_a ? up_a : dn_a) / mean;
    }
    if (max_b > 0) peak = (double)(max_b - max_a) / (double)max_b;
    if (total > 0) frac = (double)rerouted / (double)total;

    ints[0] = total; ints[1] = rerouted; ints[2] = mfloor; ints[3] = max_b; ints[4] = min_b;
    ints[5] = max_a; ints[6] = min_a; ints[7] = hot_ranks; ints[8] = cold_ranks; ints[9] = hot_experts;
    ints[10] = clones; ints[11] = intra; ints[12] = inter; ints[13] = same;
    reals[0] = rho_b; reals[1] = rho_a; reals[2] = dev_b; reals[3] = dev_a; reals[4] = peak;
    reals[5] = frac; reals[6] = cost_ratio; reals[7] = cost_C;
}
