// Phase 2 (Appendix A.3, Algorithm 2: column-priority iterative matching) and Phase 3
// (Appendix A.4, Algorithm 3: Lagrangian auction), one CTA per layer, all state in shared memory.
//
// Both phases are chains of short dependent rounds; a round is "every rank (slot) takes an
// argmax, conflicts are arbitrated by a second argmax, winners are applied".  The argmaxes are
// taken over packed 64-bit keys (score bits high, inverted index low) so that a single integer
// max gives "highest score, lowest index on ties", independent of thread order.  Scores are fp32
// with one rounding per operation (__fmul_rn / __fadd_rn / __fdiv_rn: no FMA contraction), which
// keeps every integer decision reproducible bit for bit on a CPU.
#include "taot_internal.cuh"

namespace {

typedef unsigned long long u64;

struct MatchArgs {
    const int32_t* n;            // [L,R,E]
    const int32_t* expert_load;  // [L,E]
    const int32_t* rank_load;    // [L,R]
    const float* plan;           // [L,R,R]
    const int32_t* e2r;          // [E]
    const float* B;              // [R,R]
    const int32_t* rank_off;     // [R+1]
    const int32_t* rank_list;    // [E]
    int32_t* slot_expert;        // [L,R,K]
    int32_t* slot_tokens;        // [L,R,K]
    int32_t* X;                  // [L,R,S]
    int32_t* rounds;             // [L,2] or null
    int32_t* info;               // [L]
    int32_t* nrem_g;             // [L, dmax, R] global fallback for the remaining counts
    int32_t R, E, K, dmax;
    float eps0, price_step;
    int32_t auction_max_rounds;
    int32_t nrem_in_smem;
};

__device__ __forceinline__ uint32_t ordered_bits(float f)
{
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ u64 warp_max_u64(u64 k)
{
    for (int o = 16; o > 0; o >>= 1) {
        const u64 other = __shfl_xor_sync(0xffffffffu, k, o);
        k = other > k ? other : k;
    }
    return k;
}

__global__ void match_kernel(MatchArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int R = a.R, E = a.E, K = a.K, S = R * K;
    const int NT = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NW = NT >> 5;
    const int64_t l = blockIdx.x;

    // ---- carve shared memory
    u64* arb_e = reinterpret_cast<u64*>(smem_raw);            // [E]  Phase 2 arbitration per expert
    u64* arb_r = arb_e + E;                                    // [R]  Phase 3 arbitration per rank
    int32_t* spill = reinterpret_cast<int32_t*>(arb_r + R);    // [E]
    int32_t* hotlist = spill + E;                              // [E]
    int32_t* dcol = hotlist + E;                               // [E]  expert -> column of nrem, or -1
    int32_t* spare = dcol + E;                                 // [R]
    int32_t* excess = spare + R;                               // [R]
    int32_t* matched = excess + R;                             // [R]
    int32_t* estar = matched + R;                              // [R]
    int32_t* wins = estar + R;                                 // [R]
    int32_t* slot_e = wins + R;                                // [S]
    int32_t* slot_a0 = slot_e + S;                             // [S]  planned tokens (Phase 2 result)
    int32_t* slot_a = slot_a0 + S;                             // [S]  still to collect (Phase 3)
    int32_t* nrem_s = slot_a + S;                              // [dmax*R] if it fits
    __shared__ long long s_tot;
    __shared__ int s_cnt, s_any;

    const int32_t* n = a.n + l * (int64_t)R * E;
    const int32_t* el = a.expert_load + l * E;
    const int32_t* rl = a.rank_load + l * R;
    const float* plan = a.plan + l * (int64_t)R * R;
    int32_t* nrem = a.nrem_in_smem ? nrem_s : a.nrem_g + l * (int64_t)a.dmax * R;

    // ---- integer mean, excess, spare (Appendix A.1)
    if (tid == 0) s_tot = 0;
    __syncthreads();
    {
        long long part = 0;
        for (int r = tid; r < R; r += NT) part += rl[r];
        if (part) atomicAdd(reinterpret_cast<u64*>(&s_tot), (u64)part);
    }
    __syncthreads();
    const long long mean = s_tot / R;
    for (int r = tid; r < R; r += NT) {
        const long long lr = rl[r];
        excess[r] = (int32_t)(lr > mean ? lr - mean : 0);
        spare[r] = (int32_t)(mean > lr ? mean - lr : 0);
        wins[r] = 0;
        arb_r[r] = 0;
    }
    // ---- spill by cumulative-excess differencing: position of e in its rank's (load, index) order
    for (int e = tid; e < E; e += NT) {
        const int r = a.e2r[e];
        const int32_t mine = el[e];
        long long cum = 0;
        for (int q = a.rank_off[r]; q < a.rank_off[r + 1]; ++q) {
            const int e2 = a.rank_list[q];
            const int32_t v = el[e2];
            if (v < mine || (v == mine && e2 <= e)) cum += v;
        }
        const long long hi = cum - mean, lo = cum - mine - mean;
        spill[e] = (int32_t)((hi > 0 ? hi : 0) - (lo > 0 ? lo : 0));
        arb_e[e] = 0;
    }
    for (int s = tid; s < S; s += NT) { slot_e[s] = -1; slot_a0[s] = 0; }
    __syncthreads();

    const float alpha = __fdiv_rn((float)(mean * (long long)R), (float)E);
    const float beta = __fmul_rn(0.1f, alpha);

    // =========================================================== Phase 2
    int rounds2 = 0;
    for (int kappa = 0; kappa < K; ++kappa) {
        for (int r = tid; r < R; r += NT) matched[r] = 0;
        for (;;) {
            if (tid == 0) { s_cnt = 0; s_any = 0; }
            __syncthreads();
            for (int e = tid; e < E; e += NT)
                if (spill[e] > 0) hotlist[atomicAdd(&s_cnt, 1)] = e;
            __syncthreads();
            const int nhot = s_cnt;
            if (nhot == 0) break;
            // Steps 1-2: every unmatched cold rank takes its best candidate expert
            for (int r = warp; r < R; r += NW) {
                if (matched[r] || spare[r] <= 0) { if (lane == 0) estar[r] = -1; continue; }
                const int32_t sp = spare[r];
                u64 key = 0;
                for (int q = lane; q < nhot; q += 32) {
                    const int e = hotlist[q];
                    const int hr = a.e2r[e];
                    if (hr == r) continue;
                    bool placed = false;
                    for (int kk = 0; kk < kappa; ++kk) placed |= (slot_e[r * K + kk] == e);
                    if (placed) continue;
                    const int32_t gain = spill[e] < sp ? spill[e] : sp;
                    const float ex = fmaxf((float)excess[hr], a.eps0);
                    const float tn = __fdiv_rn(plan[(int64_t)hr * R + r], ex);
                    const float t1 = __fmul_rn(alpha, a.B[(int64_t)hr * R + r]);
                    const float t2 = __fmul_rn(beta, tn);
                    const float sc = __fadd_rn(__fadd_rn((float)gain, t1), t2);
                    const u64 k64 = ((u64)__float_as_uint(sc) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)e);
                    key = k64 > key ? k64 : key;
                }
                key = warp_max_u64(key);
                if (lane == 0) {
                    if (key == 0) estar[r] = -1;
                    else {
                        const int e = (int)(0xFFFFFFFFu - (uint32_t)key);
                        estar[r] = e;
                        // Step 3: arbitration, best rank per expert (ties: lowest rank)
                        atomicMax(arb_e + e, (key & 0xFFFFFFFF00000000ull) | (u64)(0xFFFFFFFFu - (uint32_t)r));
                        s_any = 1;
                    }
                }
            }
            __syncthreads();
            if (!s_any) break;
            // Step 4: winners take min(spill, spare)
            for (int r = tid; r < R; r += NT) {
                const int e = estar[r];
                if (e >= 0 && (uint32_t)arb_e[e] == 0xFFFFFFFFu - (uint32_t)r) {
                    const int32_t g = spill[e] < spare[r] ? spill[e] : spare[r];
                    spill[e] -= g;
                    spare[r] -= g;
                    matched[r] = 1;
                    slot_e[r * K + kappa] = e;
                    slot_a0[r * K + kappa] = g;
                }
            }
            __syncthreads();
            for (int q = tid; q < nhot; q += NT) arb_e[hotlist[q]] = 0;
            ++rounds2;
            __syncthreads();
        }
        __syncthreads();
    }

    // =========================================================== Phase 3
    // compact the experts that sit in some slot; keep their per-rank remaining counts transposed [col][r]
    for (int e = tid; e < E; e += NT) dcol[e] = -1;
    if (tid == 0) s_cnt = 0;
    __syncthreads();
    for (int s = tid; s < S; s += NT) {
        slot_a[s] = slot_a0[s];
        if (slot_e[s] >= 0) dcol[slot_e[s]] = -2;
    }
    __syncthreads();
    for (int e = tid; e < E; e += NT)
        if (dcol[e] == -2) dcol[e] = atomicAdd(&s_cnt, 1);
    __syncthreads();
    const int D = s_cnt;
    for (int e = 0; e < E; ++e) {
        const int col = dcol[e];
        if (col < 0) continue;
        for (int r = tid; r < R; r += NT) nrem[col * R + r] = n[(int64_t)r * E + e];
    }
    int32_t* Xl = a.X + l * (int64_t)R * S;
    for (int64_t q = tid; q < (int64_t)R * S; q += NT) Xl[q] = 0;
    __syncthreads();

    int rounds3 = 0;
    const long long cap = (long long)R * S + S;
    for (;;) {
        if (a.auction_max_rounds > 0 && rounds3 >= a.auction_max_rounds) break;
        if (rounds3 >= cap || D == 0) break;
        if (tid == 0) s_any = 0;
        __syncthreads();
        // Step 1: every unfinished slot bids for the source rank with the best bonus minus price
        for (int s = warp; s < S; s += NW) {
            const int e = slot_e[s];
            if (e < 0 || slot_a[s] <= 0) continue;
            const int host = s / K;
            const int32_t* col = nrem + dcol[e] * R;
            u64 key = 0;
            for (int r = lane; r < R; r += 32) {
                if (col[r] <= 0) continue;
                const float b3 = (r == host) ? 1.0f : a.B[(int64_t)r * R + host];
                const float price = __fmul_rn(a.price_step, (float)wins[r]);
                const float sc = __fsub_rn(b3, price);
                const u64 k64 = ((u64)ordered_bits(sc) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)r);
                key = k64 > key ? k64 : key;
            }
            key = warp_max_u64(key);
            if (lane == 0 && key != 0) {
                const int r = (int)(0xFFFFFFFFu - (uint32_t)key);
                // Step 2: the rank keeps its best bidder (ties: lowest slot)
                atomicMax(arb_r + r, (key & 0xFFFFFFFF00000000ull) | (u64)(0xFFFFFFFFu - (uint32_t)s));
                s_any = 1;
            }
        }
        __syncthreads();
        if (!s_any) break;
        // Steps 3-4: allocate, update holdings, plan and price
        for (int r = tid; r < R; r += NT) {
            const u64 k64 = arb_r[r];
            if (k64 == 0) continue;
            arb_r[r] = 0;
            const int s = (int)(0xFFFFFFFFu - (uint32_t)k64);
            const int e = slot_e[s];
            int32_t* cell = nrem + dcol[e] * R + r;
            const int32_t x = *cell < slot_a[s] ? *cell : slot_a[s];
            Xl[(int64_t)r * S + s] += x;
            *cell -= x;
            slot_a[s] -= x;
            if (x > 0) wins[r]++;
        }
        ++rounds3;
        __syncthreads();
    }

    // ---- outputs
    int residual = 0;
    for (int s = tid; s < S; s += NT) {
        a.slot_expert[l * S + s] = slot_e[s];
        a.slot_tokens[l * S + s] = slot_a0[s];
        if (slot_e[s] >= 0 && slot_a[s] > 0) residual = 1;
    }
    residual = __syncthreads_or(residual);
    if (tid == 0) {
        if (a.rounds) { a.rounds[l * 2] = rounds2; a.rounds[l * 2 + 1] = rounds3; }
        if (residual) atomicOr(a.info + l, TAOT_INFO_AUCTION_RESIDUAL);
    }
}

size_t match_smem_fixed(int R, int E, int K)
{
    const int S = R * K;
    return sizeof(u64) * (E + R) + sizeof(int32_t) * (3 * (size_t)E + 5 * (size_t)R + 3 * (size_t)S);
}

}  // namespace

int taot_launch_match(taot_handle_t h, const int32_t* d_n, const int32_t* d_expert_load,
                      const int32_t* d_rank_load, const float* d_plan, int32_t* d_slot_expert,
                      int32_t* d_slot_tokens, int32_t* d_X, int32_t* d_rounds, int32_t* d_info,
                      int32_t* d_nrem, cudaStream_t st)
{
    const taot_params& p = h->p;
    MatchArgs a;
    a.n = d_n; a.expert_load = d_expert_load; a.rank_load = d_rank_load; a.plan = d_plan;
    a.e2r = h->d_e2r; a.B = h->d_B; a.rank_off = h->d_rank_off; a.rank_list = h->d_rank_list;
    a.slot_expert = d_slot_expert; a.slot_tokens = d_slot_tokens; a.X = d_X; a.rounds = d_rounds;
    a.info = d_info; a.nrem_g = d_nrem;
    a.R = p.R; a.E = p.E; a.K = p.K;
    a.dmax = p.E < p.R * p.K ? p.E : p.R * p.K;
    a.eps0 = p.eps0; a.price_step = p.price_step; a.auction_max_rounds = p.auction_max_rounds;
    size_t smem = match_smem_fixed(p.R, p.E, p.K);
    const size_t nrem_bytes = sizeof(int32_t) * (size_t)a.dmax * p.R;
    a.nrem_in_smem = (smem + nrem_bytes <= 200 * 1024) ? 1 : 0;
    if (a.nrem_in_smem) smem += nrem_bytes;
    const int NT = p.R <= 32 ? 128 : (p.R <= 64 ? 256 : (p.R <= 128 ? 512 : 1024));
    TAOT_CUDA_OK(cudaFuncSetAttribute(match_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    match_kernel<<<p.L, NT, smem, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
