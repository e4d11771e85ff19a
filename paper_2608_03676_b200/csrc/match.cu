// Phase 2 (Appendix A.3, Algorithm 2: column-priority iterative matching) and Phase 3
// (Appendix A.4, Algorithm 3: Lagrangian auction), one CTA per layer, all round state in shared
// memory.
//
// Both phases are chains of short dependent rounds; a round is "every rank (slot) takes an
// argmax, conflicts are arbitrated by a second argmax, winners are applied".  The argmaxes are
// taken over packed 64-bit keys (score bits high, inverted index low) so that a single integer
// max gives "highest score, lowest index on ties", independent of thread order.  Scores are fp32
// with one rounding per operation (__fmul_rn / __fadd_rn / __fsub_rn / __fdiv_rn: no FMA
// contraction), which keeps every integer decision reproducible bit for bit on a CPU.
//
// Phase 2: the two score terms that do not change between rounds (alpha*B and 0.1*alpha*T_norm)
// are computed once per layer for the experts that spill; a round is then one thread per rank
// scanning those experts with coalesced reads.
//
// Phase 3: the bonus matrix of a real topology has a handful of distinct values (tiers).  Within
// a tier a slot's score  B3 - step*wins[r]  depends on r only through wins[r], so every score a bid
// can take is one of (tier, win count) pairs, and those are listed once per handle in order of
// decreasing fp32 score (equal scores grouped).  Ranks are kept as bit sets (per tier and host, per
// win count, per expert availability); a slot walks the list with a cursor that never moves back
// and a probe is a few word-wide ANDs instead of a scan over all R ranks.  The exact fp32 score is
// what orders the list, so win counts or tiers whose scores round to the same float compete on the
// rank index alone, as in a dense scan.  A bonus matrix with more than kMaxTiers distinct values (or
// a price step that is not positive) takes the dense scan instead.
// A round of the bit-set auction is a chain of a few dozen dependent instructions between two plain barriers, so its
// cost is the instructions on that chain: every lane, whatever its slot's state, runs the same straight code (a slot
// that is done has an empty mask and sends its key to a word nobody reads), shared memory is addressed by 32-bit
// shared addresses, the end of the auction is read from a counter of live slots instead of a reducing barrier, and
// only the two rare events -- a cursor that has to move, a win -- branch off.
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
    const uint32_t* tiermask;    // [ntiers][W][R hosts] bit r of word w: B3[32w + r][host] == tierval[t]
    const float* tierval;        // [ntiers] descending
    const uint32_t* bidlist;     // [nbid] (tier, win count) pairs by decreasing score: w << 8 | t, bit 31: next has the same score
    int32_t* slot_expert;        // [L,R,K]
    int32_t* slot_tokens;        // [L,R,K]
    int32_t* X;                  // [L,R,S]
    int32_t* rounds;             // [L,2] or null
    int32_t* info;               // [L]
    int32_t* nrem_g;             // [L, dmax, R] global fallback for the remaining counts
    float* t12;                  // [L, E, 2, R] scratch: alpha*B and beta*T_norm rows of the spilling experts
    int32_t R, E, K, dmax, ntiers, W, nbid;
    float eps0, price_step;
    int32_t auction_max_rounds;
    int32_t ablation;            // TAOT_ABLATE_* bits: a term switched off is an exact zero in the score
    int32_t nrem_in_smem;
    int32_t tm_in_smem;
    int32_t big_floats;          // 4-byte words of the shared block that holds the Phase-2 score rows, then nrem
    long long* cyc;              // [L][16] SM cycles per part of the kernel as thread 0 sees them, or null (profiling aid):
                                 // 0 set-up, 1 Phase 2, 2 Phase-3 set-up, 3 Phase-3 bids (to the first barrier of a round),
                                 // 4 Phase-3 updates (to the second barrier), 5 whole kernel, 6 / 7 the busiest thread's own
                                 // probe and arbitration time in Phase 3, 8-11 Phase-2 split, 12 the Phase-3 loop as a whole.
                                 // A barrier does not hold a warp up until its next shared-memory access, so the wait at
                                 // the first barrier is counted under 4 and the wait at the second under 3 of the next round.
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

// Barrier over the first `nthreads` threads of the CTA only (a multiple of 32), on hardware barrier 1: the auction's
// rounds involve the warps that hold slots, the others wait at the CTA-wide barrier that follows the auction.  The
// aligned form: every lane of a warp that takes part reaches it together (the loop's conditions are the same for all
// lanes of a warp and the branches inside a round close before it).
__device__ __forceinline__ void bar_part(int nthreads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// Shared-memory accesses of the auction's rounds by 32-bit shared address: one instruction each, no 64-bit address
// arithmetic and no address-space conversion on the chain of a round.
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void red_max_u32(uint32_t addr, uint32_t v) { asm volatile("red.shared.max.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void red_and_u32(uint32_t addr, uint32_t v) { asm volatile("red.shared.and.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void red_add_u32(uint32_t addr, uint32_t v) { asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void red_or_u32(uint32_t addr, uint32_t v) { asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }

constexpr int kMaxW = 8;          // words of a rank bit set: R <= 256
constexpr size_t kSmemBudget = 224 * 1024;   // dynamic shared memory the kernel plans with (227 KB per CTA less the static part)

// Lowest set bit over kMaxW words (bit index = 32*w + bit), or -1: independent ANDs and a select tree
// instead of a word-by-word scan, so that a lone warp is not held up by a long dependency chain.
__device__ __forceinline__ int first_hit(const uint32_t (&cand)[8], const uint32_t* lv, int stride, int W)
{
    uint32_t h[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) h[w] = (w < W) ? (cand[w] & lv[w * stride]) : 0u;
    // pairwise: keep the lower word if it is nonzero
    const uint32_t a0 = h[0] ? h[0] : h[1]; const int i0 = h[0] ? 0 : 1;
    const uint32_t a1 = h[2] ? h[2] : h[3]; const int i1 = h[2] ? 2 : 3;
    const uint32_t a2 = h[4] ? h[4] : h[5]; const int i2 = h[4] ? 4 : 5;
    const uint32_t a3 = h[6] ? h[6] : h[7]; const int i3 = h[6] ? 6 : 7;
    const uint32_t b0 = a0 ? a0 : a1; const int j0 = a0 ? i0 : i1;
    const uint32_t b1 = a2 ? a2 : a3; const int j1 = a2 ? i2 : i3;
    const uint32_t c = b0 ? b0 : b1; const int k = b0 ? j0 : j1;
    return c ? (k << 5) + __ffs(c) - 1 : -1;
}

// Arbitration "best bidder per target" for one warp's worth of bids.  Many bidders often pick the
// same target (all slots of a tier chase the cheapest rank), so the lanes that bid for the same
// target first agree on their best key with warp-wide reductions and only one of them touches the
// shared-memory arbiter.  key = (score bits << 32) | inverted bidder index; valid bids have key != 0.
__device__ __forceinline__ void arbitrate(u64* arb, int target, u64 key)
{
    // (a hardware match-any on the target was measured several times slower than this loop over distinct targets)
    unsigned todo = __ballot_sync(0xffffffffu, key != 0);
    const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
    const int lane = threadIdx.x & 31;
    while (todo) {                                   // one pass per distinct target among this warp's bids
        const int leader = __ffs(todo) - 1;
        const int tgt = __shfl_sync(0xffffffffu, target, leader);
        const bool mine = key != 0 && target == tgt;
        const unsigned group = __ballot_sync(0xffffffffu, mine);
        const uint32_t hi_max = __reduce_max_sync(0xffffffffu, mine ? hi : 0u);
        const uint32_t lo_max = __reduce_max_sync(0xffffffffu, (mine && hi == hi_max) ? lo : 0u);
        if (lane == leader) atomicMax(arb + tgt, ((u64)hi_max << 32) | (u64)lo_max);
        todo &= ~group;
    }
}

template <bool TIMED>
__global__ void __launch_bounds__(1024)
match_kernel(MatchArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int R = a.R, E = a.E, K = a.K, S = R * K, W = a.W;
    const int NT = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NW = NT >> 5;
    const int64_t l = blockIdx.x;

    // ---- carve shared memory
    u64* arb_e = reinterpret_cast<u64*>(smem_raw);            // [E]  Phase 2 arbitration per expert
    u64* arb_r = arb_e + E;                                    // [2][R]  Phase 3 arbitration per rank, ping-pong by round
    int32_t* spill = reinterpret_cast<int32_t*>(arb_r + 2 * R); // [E]
    int32_t* hot0 = spill + E;                                 // [E]  experts that spill at the start of Phase 2
    int32_t* hot_home = hot0 + E;                              // [E]  their home ranks
    int32_t* dcol = hot_home + E;                              // [E]  expert -> column of nrem, or -1
    int32_t* spare = dcol + E;                                 // [R]
    int32_t* excess = spare + R;                               // [R]
    int32_t* matched = excess + R;                             // [R]
    int32_t* estar = matched + R;                              // [R]
    int32_t* wins = estar + R;                                 // [R]
    int32_t* slot_e = wins + R;                                // [S]
    int32_t* slot_a0 = slot_e + S;                             // [S]  planned tokens (Phase 2 result)
    int32_t* slot_a = slot_a0 + S;                             // [S]  still to collect (Phase 3)
    uint32_t* avail = reinterpret_cast<uint32_t*>(slot_a + S); // [W][dmax]  ranks still holding tokens of the expert (word-major: no bank conflicts across slots)
    uint32_t* lvl = avail + a.dmax * W;                        // [W][S+1]   ranks by win count (word-major)
    uint32_t* tm_s = lvl + (S + 1) * W;                                // [ntiers][W][S] tier masks by slot, if they fit
    uint32_t* bid_s = tm_s + (a.tm_in_smem ? a.ntiers * W * S : 0);    // [nbid] (tier, win count) pairs, best score first
    int32_t* tw_word = reinterpret_cast<int32_t*>(bid_s + a.nbid);     // [ntiers][S] word holding the whole tier for the slot's host, or -1
    uint32_t* tw_mask = reinterpret_cast<uint32_t*>(tw_word + (a.nbid ? a.ntiers * S : 0));   // [ntiers][S] that word's mask
    int32_t* nrem_s = reinterpret_cast<int32_t*>(tw_mask + (a.nbid ? a.ntiers * S : 0));      // [dmax*R] if it fits
    __shared__ long long s_tot;
    __shared__ int s_cnt, s_any, s_ns;
    __shared__ uint32_t s_live3, s_lastwin;      // Phase 3: slots that can still bid; 1 + the last round somebody won
    __shared__ int s_wcnt[32];

    const int32_t* n = a.n + l * (int64_t)R * E;
    const int32_t* el = a.expert_load + l * E;
    const int32_t* rl = a.rank_load + l * R;
    const float* plan = a.plan + l * (int64_t)R * R;
    int32_t* nrem = a.nrem_in_smem ? nrem_s : a.nrem_g + l * (int64_t)a.dmax * R;
    float* t12 = a.t12 + l * (int64_t)E * 2 * R;      // global scratch; replaced by shared memory below if the rows fit

    const bool timed = TIMED && tid == 0;
    const long long c_start = timed ? clock64() : 0;
    long long c_bid = 0, c_upd = 0, c_probe = 0, c_atom = 0, c_scan = 0, c_win = 0, c_row = 0, c_build = 0;
    // ---- integer mean, excess, spare (Appendix A.1)
    if (tid == 0) { s_tot = 0; s_cnt = 0; }
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
        arb_r[R + r] = 0;
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
        const int32_t sp = (int32_t)((hi > 0 ? hi : 0) - (lo > 0 ? lo : 0));
        spill[e] = sp;
        arb_e[e] = 0;
    }
    for (int s = tid; s < S; s += NT) { slot_e[s] = -1; slot_a0[s] = 0; }
    __syncthreads();
    // the experts that spill, in ascending index order (position q in this list orders them as the index does, so
    // "lowest expert on ties" is "lowest position on ties")
    int nhot0 = 0;
    for (int base = 0; base < E; base += NT) {
        const int e = base + tid;
        const bool hot = e < E && spill[e] > 0;
        const unsigned bal = __ballot_sync(0xffffffffu, hot);
        if (lane == 0) s_wcnt[warp] = __popc(bal);
        __syncthreads();
        int off = nhot0, tot = 0;
        for (int w = 0; w < NW; ++w) { const int c = s_wcnt[w]; if (w < warp) off += c; tot += c; }
        if (hot) {
            const int q = off + __popc(bal & ((1u << lane) - 1u));
            hot0[q] = e;
            hot_home[q] = a.e2r[e];
        }
        nhot0 += tot;
        __syncthreads();
    }

    const float alpha = __fdiv_rn((float)(mean * (long long)R), (float)E);
    const float beta = __fmul_rn(0.1f, alpha);
    // Phase 2 keeps the current score of every (rank, spilling expert) pair as an integer key, row stride odd so that
    // neither a rank's scan nor an expert's update meets bank conflicts; the keys and the round-invariant rows below
    // are only used in Phase 2 and the remaining counts only exist in Phase 3: they share one block
    const int NHs = nhot0 | 1;
    const bool keyed = nhot0 > 0 && (int64_t)NHs * R <= (int64_t)a.big_floats;
    uint32_t* keyM = reinterpret_cast<uint32_t*>(nrem_s);                       // [R][NHs]
    const int64_t key_words = keyed ? (int64_t)NHs * R : 0;
    if (key_words + (int64_t)nhot0 * 2 * R <= (int64_t)a.big_floats) t12 = reinterpret_cast<float*>(nrem_s) + key_words;

    // ---- round-invariant score terms of the spilling experts: t1 = alpha*B, t2 = beta*T/max(excess, eps0)
#pragma unroll 4
    for (int64_t idx = tid; idx < (int64_t)nhot0 * R; idx += NT) {
        const int q = (int)(idx / R), r = (int)(idx - (int64_t)q * R);
        const int hr = hot_home[q];
        const float ex = fmaxf((float)excess[hr], a.eps0);
        const float tn = (a.ablation & TAOT_ABLATE_HINT) ? 0.0f : __fdiv_rn(plan[(int64_t)hr * R + r], ex);
        const float bp = (a.ablation & TAOT_ABLATE_TOPOLOGY) ? 0.0f : a.B[(int64_t)hr * R + r];
        t12[((int64_t)q * 2) * R + r] = __fmul_rn(alpha, bp);
        t12[((int64_t)q * 2 + 1) * R + r] = __fmul_rn(beta, tn);
    }
    __syncthreads();

    // =========================================================== Phase 2
    const long long c_p2 = timed ? clock64() : 0;
    int rounds2 = 0;
    int qsh = 0;                                  // lanes per rank in the scan: QS = 2^qsh, the largest power of two <= min(32, NT / R)
    while ((2 << qsh) <= 32 && (2 << qsh) * R <= NT) ++qsh;
    const int QS = 1 << qsh;
    const int qs = tid & (QS - 1);
    // score of expert position q on rank r as an ordered integer key, 0 if the pair is no candidate (Algorithm 2's mask:
    // the expert still spills, r is not its home, it is not on r already); the rank-side conditions (unmatched, spare
    // left) are tested by the rank's scan
    auto pair_key = [&](int q, int r, int kappa) -> uint32_t {
        const int e = hot0[q];
        const int32_t se = spill[e];
        bool ok = se > 0 && hot_home[q] != r;
        for (int kk = 0; kk < kappa; ++kk) ok = ok && (slot_e[r * K + kk] != e);
        const int32_t sp = spare[r];
        const int32_t gain = se < sp ? se : sp;
        const float sc = __fadd_rn(__fadd_rn((float)gain, t12[((int64_t)q * 2) * R + r]), t12[((int64_t)q * 2 + 1) * R + r]);
        return ok ? ordered_bits(sc) : 0u;
    };
    int32_t* served = dcol;                       // [E] positions of the experts served in a round (dcol is Phase 3's)
    for (int kappa = 0; keyed && kappa < K; ++kappa) {
        // Between rounds a pair's score changes only when its expert was served (its spill shrank): a rank's spare
        // changes only when it is matched, and then it is out for this slot index.  So all keys are formed once per
        // slot index and a round re-forms the rows of the experts it served; a rank's arg-max is one load and one
        // compare per spilling expert.
        const long long c_b0 = timed ? clock64() : 0;
        // arbitration state per expert: best score among this round's bidders, then the lowest rank that has it
        uint32_t* arb_hi = reinterpret_cast<uint32_t*>(arb_e);
        uint32_t* arb_lo = arb_hi + E;
        int smax = 0;                              // largest spare of this slot index: a row changes only below it
        for (int r = tid; r < R; r += NT) { matched[r] = 0; smax = spare[r] > smax ? spare[r] : smax; }
        for (int e = tid; e < E; e += NT) { arb_hi[e] = 0u; arb_lo[e] = 0xFFFFFFFFu; }
        smax = __reduce_max_sync(0xffffffffu, smax);
        if (tid == 0) s_cnt = 0;
        __syncthreads();
        if (lane == 0) atomicMax(&s_cnt, smax);
        for (int64_t idx = tid; idx < (int64_t)nhot0 * R; idx += NT) {
            const int q = (int)(idx / R), r = (int)(idx - (int64_t)q * R);
            keyM[r * NHs + q] = pair_key(q, r, kappa);
        }
        __syncthreads();
        const int32_t spare_cap = s_cnt;
        if (timed) c_build += clock64() - c_b0;
        for (;;) {
            const long long c_s0 = timed ? clock64() : 0;
            // Steps 1-2: every unmatched cold rank takes its best candidate expert (ties: lowest position = lowest index)
            // (QS lanes per rank with QS * R <= NT: one pass covers every rank)
            const int r = tid >> qsh;
            uint32_t my_bk = 0u;                   // this thread's bid, if it is the lead lane of a bidding rank
            int my_q = -1;
            {
                u64 key = 0;
                if (r < R && !matched[r] && spare[r] > 0) {
                    const uint32_t* row = keyM + r * NHs;
                    uint32_t bk = 0u;
                    int bq = 0;
#pragma unroll 4
                    for (int q = qs; q < nhot0; q += QS) {      // ascending positions: a strict compare keeps the lowest
                        const uint32_t k32 = row[q];
                        if (k32 > bk) { bk = k32; bq = q; }
                    }
                    if (bk != 0u) key = ((u64)bk << 32) | (u64)(0xFFFFFFFFu - (uint32_t)bq);
                }
                for (int o = 1; o < QS; o <<= 1) {
                    const u64 other = __shfl_xor_sync(0xffffffffu, key, o);
                    key = other > key ? other : key;
                }
                if (qs == 0 && r < R && key != 0) {
                    my_bk = (uint32_t)(key >> 32);
                    my_q = (int)(0xFFFFFFFFu - (uint32_t)key);
                }
            }
            const int my_e = my_q >= 0 ? hot0[my_q] : 0;
            // Step 3, first half: the best score any rank offers the expert (native 32-bit shared-memory atomics; agreeing
            // inside the warp first on the expert most lanes want was measured and cost more than the conflicts it saves)
            if (my_q >= 0) atomicMax(&arb_hi[my_e], my_bk);
            if (!__syncthreads_or(my_q >= 0)) break;
            if (tid == 0) s_ns = 0;
            // Step 3, second half: among the ranks that offer it, the lowest
            if (my_q >= 0 && arb_hi[my_e] == my_bk) atomicMin(&arb_lo[my_e], (uint32_t)r);
            __syncthreads();
            const long long c_s1 = timed ? clock64() : 0;
            if (timed) c_scan += c_s1 - c_s0;
            // Step 4: winners take min(spill, spare), and put the arbitration entries back.  A row of keys changes only
            // where min(spill, spare_r) does, i.e. for ranks with more spare than the expert now spills: rows whose
            // expert still spills at least the largest spare of this slot index are left as they are.
            if (my_q >= 0 && arb_lo[my_e] == (uint32_t)r) {
                const int32_t g = spill[my_e] < spare[r] ? spill[my_e] : spare[r];
                spill[my_e] -= g;
                spare[r] -= g;
                matched[r] = 1;
                slot_e[r * K + kappa] = my_e;
                slot_a0[r * K + kappa] = g;
                arb_hi[my_e] = 0u;                 // (a loser compares arb_lo with its own rank: the reset value is nobody's)
                arb_lo[my_e] = 0xFFFFFFFFu;
                if (spill[my_e] < spare_cap) served[atomicAdd(&s_ns, 1)] = my_q;
            }
            __syncthreads();
            const long long c_s2 = timed ? clock64() : 0;
            const int ns = s_ns;
            if (ns > 0) {                          // uniform over the CTA
                for (int idx = tid; idx < ns * R; idx += NT) {
                    const int i = idx / R, r = idx - i * R;
                    const int q = served[i];
                    keyM[r * NHs + q] = pair_key(q, r, kappa);
                }
                __syncthreads();
            }
            ++rounds2;
            if (timed) { const long long c_s3 = clock64(); c_win += c_s2 - c_s1; c_row += c_s3 - c_s2; }
        }
        __syncthreads();
    }
    for (int kappa = 0; !keyed && kappa < K; ++kappa) {
        for (int r = tid; r < R; r += NT) matched[r] = 0;
        for (;;) {
            if (tid == 0) s_any = 0;
            __syncthreads();
            // Steps 1-2: every unmatched cold rank takes its best candidate expert.  QS adjacent lanes share one rank
            // and split the list of spilling experts between them; their best keys meet by xor-shuffles.
            for (int rb = 0; rb < R; rb += NT >> qsh) {
                const int r = rb + (tid >> qsh);                  // whole warps stay in the loop for the warp-wide steps
                int best_e = -1;
                u64 key = 0;
                const int32_t sp = r < R ? spare[r] : 0;
                if (r < R && !matched[r] && sp > 0) {
                    for (int q = qs; q < nhot0; q += QS) {
                        const int e = hot0[q];
                        const int32_t se = spill[e];
                        if (se <= 0 || hot_home[q] == r) continue;
                        bool placed = false;
                        for (int kk = 0; kk < kappa; ++kk) placed |= (slot_e[r * K + kk] == e);
                        if (placed) continue;
                        const int32_t gain = se < sp ? se : sp;
                        const float t1 = t12[((int64_t)q * 2) * R + r];
                        const float t2 = t12[((int64_t)q * 2 + 1) * R + r];
                        const float sc = __fadd_rn(__fadd_rn((float)gain, t1), t2);
                        const u64 k64 = ((u64)ordered_bits(sc) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)e);   // ordered: a negative preference may give a negative score
                        key = k64 > key ? k64 : key;
                    }
                }
                for (int o = 1; o < QS; o <<= 1) {
                    const u64 other = __shfl_xor_sync(0xffffffffu, key, o);
                    key = other > key ? other : key;
                }
                if (key != 0) best_e = (int)(0xFFFFFFFFu - (uint32_t)key);
                const bool lead = qs == 0 && r < R;
                if (lead) {
                    estar[r] = best_e;
                    if (key != 0) s_any = 1;
                }
                // Step 3: arbitration, best rank per expert (ties: lowest rank)
                arbitrate(arb_e, best_e, (key == 0 || !lead) ? 0ull : ((key & 0xFFFFFFFF00000000ull) | (u64)(0xFFFFFFFFu - (uint32_t)r)));
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
            for (int q = tid; q < nhot0; q += NT) arb_e[hot0[q]] = 0;
            ++rounds2;
        }
        __syncthreads();
    }

    // =========================================================== Phase 3
    const long long c_p3 = timed ? clock64() : 0;
    long long c_p3loop = c_p3, c_p3end = c_p3;
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
    for (int i = tid; i < a.dmax * W; i += NT) avail[i] = 0u;
    for (int i = tid; i < (S + 1) * W; i += NT) lvl[i] = 0u;
    __syncthreads();
    const int D = s_cnt;
    for (int e = tid; e < E; e += NT)
        if (dcol[e] >= 0) hot0[dcol[e]] = e;                   // column -> expert (the Phase-2 list is no longer needed)
    __syncthreads();
#pragma unroll 4
    for (int q = tid; q < D * R; q += NT) {
        const int col = q / R, r = q - col * R;
        const int32_t v = n[(int64_t)r * E + hot0[col]];
        nrem[q] = v;
        if (v > 0) atomicOr(avail + (r >> 5) * a.dmax + col, 1u << (r & 31));
    }
    for (int r = tid; r < R; r += NT) atomicOr(lvl + (r >> 5) * (S + 1), 1u << (r & 31));      // every rank starts with 0 wins
    int32_t* Xl = a.X + l * (int64_t)R * S;
    for (int64_t q = tid; q < (int64_t)R * S; q += NT) Xl[q] = 0;
    __syncthreads();

    int rounds3 = 0;
    const long long cap = (long long)R * S + S;
    const bool tiered = a.nbid > 0 && S <= NT;
    if (tiered && D > 0) {
        // ---- bit-set auction: thread s is slot s for the whole auction and keeps the slot's state in registers.
        // A bid walks the list of all (tier, win count) pairs in order of decreasing score: the first pair that still
        // has a candidate rank (in the tier for this slot's host, holding tokens of the slot's expert, with that win
        // count) is the bid; pairs of equal score are scanned together and the lowest rank wins.  Win counts only grow
        // and holdings only shrink, so no pair before the cursor can ever regain a candidate: the cursor never moves
        // back and a round costs one or two probes per slot.
        const int s = tid;
        bool live = s < S && slot_e[s] >= 0 && slot_a[s] > 0;
        const int e = live ? slot_e[s] : 0;
        const int col = live ? dcol[e] : 0;
        const int host = s < S ? s / K : 0;
        int32_t A = live ? slot_a[s] : 0;
        const uint32_t* av = avail + col;                          // word w at av[w * dmax]
        // this slot's tier masks: tier t, word w at tm[(t * W + w) * tms]; a shared-memory copy when it fits
        const uint32_t* tm = a.tiermask + host;
        int tms = R;
        if (a.tm_in_smem) {
            for (int q = tid; q < a.ntiers * W * S; q += NT) {
                const int ss = q % S, tw = q / S;
                tm_s[q] = a.tiermask[(int64_t)tw * R + ss / K];
            }
            tm = tm_s + (s < S ? s : 0);
            tms = S;
        }
        for (int q = tid; q < a.nbid; q += NT) bid_s[q] = a.bidlist[q];
        for (int q = tid; q < 2 * R; q += NT) reinterpret_cast<uint32_t*>(arb_r)[q] = 0u;     // the two arbiter sets
        __syncthreads();
        const int LS = S + 1;                                      // lvl: word w of level wl at lvl[w * LS + wl]
        // a tier whose ranks (for this slot's host) all sit in one 32-bit word is probed with that word alone
        if (s < S) {
            for (int t = 0; t < a.ntiers; ++t) {
                int nz = 0, wd = 0;
                uint32_t val = 0u;
                for (int w = 0; w < W; ++w) {
                    const uint32_t mk = tm[(t * W + w) * tms];
                    if (mk) { ++nz; wd = w; val = mk; }
                }
                tw_word[t * S + s] = nz <= 1 ? wd : -1;
                tw_mask[t * S + s] = nz <= 1 ? val : tm[(t * W) * tms];      // several words: the mask of word 0
            }
        }
        // Per-slot state of the walk, all in registers: the cursor, and the entry under it decoded once per cursor
        // position into exactly what a probe needs -- this slot's tier mask for the word it looks at, the addresses of
        // that word in the expert's availability set and in the win-count set, and the arbitration key of the entry.
        int cur = 0;                             // list entry (start of a group of equal scores) that may still hit
        int pw = 0;                              // word the probe looks at
        uint32_t e_pr = 0u;                      // the list word under the cursor
        uint32_t e_mk = 0u;                      // tier mask for word pw; 0 for a group of tied entries (generic probe)
        int e_wd = -1;                           // the tier's only word, or -1 if it spans several
        const uint32_t* p_av = av;               // &avail[pw][col]
        uint32_t* p_lv = lvl;                    // &lvl[pw][win count of the entry]
        uint32_t keyb = 0u;                      // (list position, slot) packed for the arbiter
        auto load_entry = [&]() {
            if (cur >= a.nbid) { live = false; e_mk = 0u; return; }     // nothing left this slot could ever bid for
            e_pr = bid_s[cur];
            const int t = (int)(e_pr & 0xFFu), wl = (int)((e_pr >> 8) & 0xFFFFu);
            e_wd = tw_word[t * S + s];
            pw = e_wd >= 0 ? e_wd : 0;
            e_mk = (e_pr & 0x80000000u) ? 0u : tw_mask[t * S + s];      // several words: the mask of word 0
            p_av = av + pw * a.dmax;
            p_lv = lvl + pw * LS + wl;
            keyb = ((uint32_t)(a.nbid - cur) << 16) | (uint32_t)(0xFFFF - s);
        };
        if (live) load_entry();
        // The rounds end when no slot can bid any more.  A count of the slots that still can, kept in shared memory,
        // tells: it is only ever changed between the two barriers of a round and only read between the second barrier
        // of one round and the first of the next, so every thread sees the same value and no round needs a barrier that
        // also reduces a predicate (about 150 cycles more than a plain one after a shared-memory atomic).
        if (tid == 0) { s_live3 = 0u; s_lastwin = 0u; }
        __syncthreads();
        if (live) atomicAdd(&s_live3, 1u);
        __syncthreads();
        uint32_t* const arb = reinterpret_cast<uint32_t*>(arb_r);     // [R] best bid per rank; the winner clears its entry
        long long limit = cap;
        if (a.auction_max_rounds > 0 && a.auction_max_rounds < limit) limit = a.auction_max_rounds;
        const int round_limit = (int)(limit < 0x7fffffffLL ? limit : 0x7fffffffLL);
        if (timed) c_p3loop = clock64();
        const int NP = ((S + 31) >> 5) << 5;      // threads that take part in the rounds: the warps holding slots
        const uint32_t a_arb = smem_u32(arb), a_avc = smem_u32(av);
        const uint32_t a_live = smem_u32(&s_live3), a_lastwin = smem_u32(&s_lastwin);
        // a slot that does not bid sends its key to a word of its own behind the R arbiters (the block holds 4R words):
        // the bid is one instruction for every lane, whatever the slot's state
        const uint32_t a_idle = a_arb + 4u * (uint32_t)(R + tid % (3 * R));
        const uint32_t dmax4 = (uint32_t)a.dmax * 4u;
        uint32_t a_av = smem_u32(p_av), a_lv = smem_u32(p_lv);       // the two words a probe reads
        const bool nrem_smem = a.nrem_in_smem != 0;
        int32_t* const nrem_col = nrem + col * R;                    // this slot's expert: what each rank still holds
        const uint32_t a_cell0 = nrem_smem ? smem_u32(nrem_col) : 0u;
        int32_t* const Xs = Xl + s;                                   // column s of the plan
        bool dying = false;                       // the cursor ran off the list: leave the count after the next barrier
        while (tid < NP && rounds3 < round_limit) {
            const long long c_r0 = TIMED ? clock64() : 0;
            // Step 1: bid for the source rank with the best bonus minus price.
            // An entry whose score no other entry shares: while the cursor rests on it its candidate set (tier for this
            // host AND holding the expert AND this win count) can only shrink -- a rank enters this win count from the
            // one below, and the entry of the same tier with that lower count comes earlier in the list, so it was found
            // empty for good before the cursor got here.  Words found empty therefore stay empty: the probe is one word
            // (the tier's only word, or the word of the last hit), two loads and two ANDs, the same for every lane; a
            // slot that is done keeps a zero mask.  Only a probe that comes back empty leaves this path.
            const uint32_t nlive = lds_u32(a_live);
            uint32_t hit = e_mk & lds_u32(a_av) & lds_u32(a_lv);
            uint32_t a_sel = a_lv;               // win-count word of the rank bid for (the tied groups set their own)
            int r_best = (pw << 5) + __ffs(hit) - 1;
            bool bids = hit != 0u;
            if (hit == 0u && live) {
                uint32_t* p_sel = p_lv;
                r_best = -1;
                for (;;) {
                    hit = e_mk & *p_av & *p_lv;
                    if (hit) { r_best = (pw << 5) + __ffs(hit) - 1; p_sel = p_lv; break; }
                    if (!(e_pr & 0x80000000u)) { // an empty word: the tier's next word, or the next entry
                        if (e_wd < 0 && pw + 1 < W) {
                            ++pw;
                            e_mk = tm[((int)(e_pr & 0xFFu) * W + pw) * tms];
                            p_av += a.dmax;
                            p_lv += LS;
                        } else {
                            ++cur;
                            load_entry();
                        }
                    } else {
                        // a group of entries with one and the same fp32 score: probe every entry, the lowest rank wins
                        int g = cur;
                        uint32_t pr;
                        do {
                            pr = bid_s[g++];
                            const int t = (int)(pr & 0xFFu), wl = (int)((pr >> 8) & 0xFFFFu);
                            const int wd = tw_word[t * S + s];
                            int r;
                            if (wd >= 0) {
                                const uint32_t h1 = tw_mask[t * S + s] & av[wd * a.dmax] & lvl[wd * LS + wl];
                                r = h1 ? (wd << 5) + __ffs(h1) - 1 : -1;
                            } else {
                                uint32_t cand[kMaxW];
#pragma unroll
                                for (int w = 0; w < kMaxW; ++w) cand[w] = (w < W) ? (tm[(t * W + w) * tms] & av[w * a.dmax]) : 0u;
                                r = first_hit(cand, lvl + wl, LS, W);
                            }
                            if (r >= 0 && (r_best < 0 || r < r_best)) { r_best = r; p_sel = lvl + (r >> 5) * LS + wl; }
                        } while (pr & 0x80000000u);
                        if (r_best >= 0) break;
                        cur = g;                 // the whole group is empty for good
                        load_entry();
                    }
                    if (!live) break;
                }
                a_av = smem_u32(p_av);
                a_lv = smem_u32(p_lv);
                a_sel = smem_u32(p_sel);
                bids = r_best >= 0;
                dying = !live;
            }
            // Step 2: the rank keeps its best bidder (ties: lowest slot).  The position of a score in the list orders
            // scores exactly as their fp32 values do, so (list position, slot) packs into one 32-bit key and a single
            // native shared-memory max arbitrates: smaller position = higher score, then the lower slot.
            const uint32_t a_mine = bids ? a_arb + ((uint32_t)r_best << 2) : a_idle;
            const long long c_rp = TIMED ? clock64() : 0;
            red_max_u32(a_mine, keyb);
            if (TIMED) { const long long c_ra = clock64(); c_probe += c_rp - c_r0; c_atom += c_ra - c_rp; }
            bar_part(NP);
            const long long c_r1 = TIMED ? clock64() : 0;
            // Steps 3-4: the winning slot of each rank collects x = min(n, A); holdings, plan and price follow.  The
            // rank bid for holds tokens of the expert (its availability bit was set) and the slot still wants some, so
            // x > 0 and the rank's win count goes from the entry's to the next: its bit moves one word up in lvl.
            const bool won = (lds_u32(a_mine) == keyb) & bids;
            if (dying) { red_add_u32(a_live, 0xFFFFFFFFu); dying = false; }
            if (won) {
                const uint32_t bit = 1u << (r_best & 31);
                red_and_u32(a_sel, ~bit);
                red_or_u32(a_sel + 4u, bit);
                sts_u32(a_mine, 0u);             // losers of this round compare against their own key: 0 is nobody's
                sts_u32(a_lastwin, (uint32_t)rounds3 + 1u);
                int32_t have;
                if (nrem_smem) have = (int32_t)lds_u32(a_cell0 + ((uint32_t)r_best << 2));
                else have = nrem_col[r_best];
                const int32_t x = have < A ? have : A;
                if (nrem_smem) sts_u32(a_cell0 + ((uint32_t)r_best << 2), (uint32_t)(have - x));
                else nrem_col[r_best] = have - x;
                A -= x;
                if (have == x) red_and_u32(a_avc + (uint32_t)(r_best >> 5) * dmax4, ~bit);
                if (A <= 0) { live = false; e_mk = 0u; red_add_u32(a_live, 0xFFFFFFFFu); }
                Xs[(int64_t)r_best * S] = x;     // a (rank, slot) pair is served at most once
            }
            // nobody was left before this round (the same answer in every thread): one more round, empty, ends the loop
            rounds3 = nlive ? rounds3 + 1 : round_limit;
            bar_part(NP);
            if (TIMED && timed) { const long long c_r2 = clock64(); c_bid += c_r1 - c_r0; c_upd += c_r2 - c_r1; }
        }
        if (timed) c_p3end = clock64();
        if (s < S) slot_a[s] = A;
        __syncthreads();
        rounds3 = (int)s_lastwin;                 // rounds in which somebody bid
    } else {
        for (;;) {
            if (a.auction_max_rounds > 0 && rounds3 >= a.auction_max_rounds) break;
            if (rounds3 >= cap || D == 0) break;
            if (tid == 0) s_any = 0;
            __syncthreads();
            // Step 1: every unfinished slot bids for the source rank with the best bonus minus price (dense scan)
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
                const int col = dcol[slot_e[s]];
                int32_t* cell = nrem + col * R + r;
                const int32_t have = *cell;
                const int32_t x = have < slot_a[s] ? have : slot_a[s];
                Xl[(int64_t)r * S + s] = x;          // a (rank, slot) pair is served at most once
                *cell = have - x;
                slot_a[s] -= x;
                if (x > 0) wins[r]++;
            }
            ++rounds3;
            __syncthreads();
        }
    }

    // ---- outputs
    int residual = 0;
    for (int s = tid; s < S; s += NT) {
        a.slot_expert[l * S + s] = slot_e[s];
        a.slot_tokens[l * S + s] = slot_a0[s];
        if (slot_e[s] >= 0 && slot_a[s] > 0) residual = 1;
    }
    residual = __syncthreads_or(residual);
    if (TIMED) {                                  // the busiest thread's own probe and arbitration time
        __shared__ unsigned long long s_mx[2];
        if (tid == 0) { s_mx[0] = 0; s_mx[1] = 0; }
        __syncthreads();
        unsigned long long mp = (unsigned long long)c_probe, ma = (unsigned long long)c_atom;
        for (int o = 16; o > 0; o >>= 1) {        // one atomic per warp: 64-bit shared-memory atomics from every thread
            const unsigned long long op = __shfl_xor_sync(0xffffffffu, mp, o), oa = __shfl_xor_sync(0xffffffffu, ma, o);
            mp = op > mp ? op : mp;               // would cost more than the rounds they report on
            ma = oa > ma ? oa : ma;
        }
        if ((tid & 31) == 0) { atomicMax(&s_mx[0], mp); atomicMax(&s_mx[1], ma); }
        __syncthreads();
        c_probe = (long long)s_mx[0]; c_atom = (long long)s_mx[1];
    }
    if (tid == 0) {
        if (a.rounds) { a.rounds[l * 2] = rounds2; a.rounds[l * 2 + 1] = rounds3; }
        if (residual) atomicOr(a.info + l, TAOT_INFO_AUCTION_RESIDUAL);
        if (timed) {
            long long* c = a.cyc + l * 16;
            c[0] = c_p2 - c_start; c[1] = c_p3 - c_p2; c[2] = c_p3loop - c_p3; c[3] = c_bid; c[4] = c_upd;
            c[5] = clock64() - c_start; c[6] = c_probe; c[7] = c_atom;
            c[8] = c_scan; c[9] = c_win; c[10] = c_row; c[11] = c_build;
            c[12] = c_p3end - c_p3loop;
            for (int i = 13; i < 16; ++i) c[i] = 0;
        }
    }
}

size_t match_smem_fixed(int R, int E, int K, int dmax, int W, int ntiers)
{
    const size_t S = (size_t)R * K;
    return sizeof(u64) * (E + 2 * (size_t)R) + sizeof(int32_t) * (4 * (size_t)E + 5 * (size_t)R + 3 * S) +
           sizeof(uint32_t) * ((size_t)dmax * W + (S + 1) * W);
}

}  // namespace

int taot_launch_match(taot_handle_t h, const int32_t* d_n, const int32_t* d_expert_load,
                      const int32_t* d_rank_load, const float* d_plan, int32_t* d_slot_expert,
                      int32_t* d_slot_tokens, int32_t* d_X, int32_t* d_rounds, int32_t* d_info,
                      int32_t* d_nrem, float* d_t12, cudaStream_t st, long long* d_cyc)
{
    const taot_params& p = h->p;
    MatchArgs a;
    a.cyc = d_cyc;
    a.n = d_n; a.expert_load = d_expert_load; a.rank_load = d_rank_load; a.plan = d_plan;
    a.e2r = h->d_e2r; a.B = h->d_B; a.rank_off = h->d_rank_off; a.rank_list = h->d_rank_list;
    a.tiermask = h->d_tiermask; a.tierval = h->d_tierval; a.bidlist = h->d_bidlist;
    a.slot_expert = d_slot_expert; a.slot_tokens = d_slot_tokens; a.X = d_X; a.rounds = d_rounds;
    a.info = d_info; a.nrem_g = d_nrem; a.t12 = d_t12;
    a.R = p.R; a.E = p.E; a.K = p.K;
    a.dmax = p.E < p.R * p.K ? p.E : p.R * p.K;
    a.W = (p.R + 31) / 32;
    a.nbid = (h->ntiers > 0 && h->nbid > 0 && a.W <= kMaxW && p.R * p.K <= 1024) ? h->nbid : 0;
    a.ntiers = a.nbid > 0 ? h->ntiers : 0;
    a.eps0 = p.eps0; a.price_step = p.price_step; a.auction_max_rounds = p.auction_max_rounds;
    a.ablation = p.ablation;
    size_t smem = match_smem_fixed(p.R, p.E, p.K, a.dmax, a.W, a.ntiers);
    if (a.nbid > 0) smem += sizeof(uint32_t) * ((size_t)a.nbid + 2 * (size_t)a.ntiers * p.R * p.K);
    const size_t nrem_bytes = sizeof(int32_t) * (size_t)a.dmax * p.R;
    const size_t tm_bytes = sizeof(uint32_t) * (size_t)a.ntiers * a.W * p.R * p.K;
    a.tm_in_smem = (a.ntiers > 0 && smem + tm_bytes <= 96 * 1024) ? 1 : 0;
    if (a.tm_in_smem) smem += tm_bytes;
    a.nrem_in_smem = (smem + nrem_bytes <= kSmemBudget) ? 1 : 0;
    // one block for Phase 2 (per spilling expert R keys and 2 * R floats of round-invariant score rows) and then the
    // remaining counts: as large as the counts need if those live in shared memory, and as much of what Phase 2 could
    // use as there is room for
    size_t big = a.nrem_in_smem ? nrem_bytes : 0;
    const size_t want = sizeof(float) * ((size_t)p.R * ((size_t)p.E | 1) + 2 * (size_t)p.R * (size_t)p.E);
    const size_t room = kSmemBudget > smem ? kSmemBudget - smem : 0;
    if (big < want) big = want < room ? want : (room > big ? room : big);
    a.big_floats = (int32_t)(big / 4);
    smem += big;
    if (smem > 227 * 1024) return TAOT_ERR_UNSUPPORTED;
    TAOT_CUDA_OK(cudaFuncSetAttribute(match_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (d_cyc) TAOT_CUDA_OK(cudaFuncSetAttribute(match_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int need = p.R * p.K > p.R ? p.R * p.K : p.R;
    // two threads per slot (or rank): Phase 2 splits each rank's scan over more lanes, and the extra warps cost the
    // auction's barriers less than that saves (measured: 256 threads for 16 and 64 ranks, 512 for 256 ranks x 1 slot)
    int NT = 2 * (((need + 31) / 32) * 32);
    NT = NT < 256 ? 256 : (NT > 1024 ? 1024 : NT);
    if (d_cyc) match_kernel<true><<<p.L, NT, smem, st>>>(a);
    else match_kernel<false><<<p.L, NT, smem, st>>>(a);
    TAOT_CUDA_OK(cudaGetLastError());
    return 1;
}
