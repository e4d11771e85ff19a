// C ABI of libtaot: handle management, argument validation, workspace carve-up and the
// stage chaining of taot_plan / taot_plan_host.  No arithmetic of the method lives here except
// the two topology tables derived once per handle (the preference matrix B when the caller
// gives none, and the first-iteration row normaliser of the Sinkhorn solve).
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "taot_internal.cuh"

namespace {

bool valid_params(const taot_params* p)
{
    if (p->struct_size != (int32_t)sizeof(taot_params)) return false;
    if (p->L < 1 || p->R < 1 || p->E < 1 || p->K < 1 || p->k < 1) return false;
    if (p->T < p->R || p->T % p->R != 0) return false;
    if (p->T * (int64_t)p->k >= ((int64_t)1 << 31)) return false;
    if (!(p->eps > 0.0f) || !std::isfinite(p->eps)) return false;
    if (p->max_iters < 1) return false;
    if (!(p->eps0 >= 0.0f) || !std::isfinite(p->eps0)) return false;
    if (!std::isfinite(p->price_step) || !std::isfinite(p->tol)) return false;
    if (p->ablation & ~(TAOT_ABLATE_HINT | TAOT_ABLATE_TOPOLOGY)) return false;
    return true;
}

bool supported_params(const taot_params* p)
{
    return p->R <= 1024 && p->E <= 1024 && p->K <= 8 && p->k <= 64 &&
           (int64_t)p->L * p->R * ((p->T / p->R * p->k + TAOT_CHUNK - 1) / TAOT_CHUNK) < ((int64_t)1 << 31);
}

template <typename T>
int upload(T** dst, const T* src, size_t count)
{
    if (cudaMalloc(reinterpret_cast<void**>(dst), sizeof(T) * count) != cudaSuccess) return TAOT_ERR_CUDA;
    if (cudaMemcpy(*dst, src, sizeof(T) * count, cudaMemcpyHostToDevice) != cudaSuccess) return TAOT_ERR_CUDA;
    return TAOT_OK;
}

void layout(taot_handle_t h)
{
    const taot_params& p = h->p;
    h->seg = p.T / p.R * p.k;
    h->nc = (int32_t)((h->seg + TAOT_CHUNK - 1) / TAOT_CHUNK);
    const int64_t r2 = (int64_t)p.R * p.R;
    int64_t cap = r2 / 4 > 12288 ? r2 / 4 : 12288;
    h->kcap = (int32_t)(cap < r2 ? cap : r2);
    h->kcap_global = 0;
    if (p.R > 256) {                      // beyond shared memory: the kernel matrix lives in workspace
        h->kcap = 0;
        h->kcap_global = r2 / 4;          // |hot| * |cold| <= R^2/4 whenever supply and demand ranks are disjoint
    }
    const size_t LR = (size_t)p.L * p.R;
    const int dmax = p.E < p.R * p.K ? p.E : p.R * p.K;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off = taot_align_up(off + bytes, 256); return o; };
    const size_t path = p.R <= 256 ? 1 : 0;       // beyond 256 ranks only Phase 1 runs: no schedule buffers
    h->off_cc = take(path * sizeof(int32_t) * LR * h->nc * p.E);
    h->off_excess = take(sizeof(int32_t) * LR);
    h->off_spare = take(sizeof(int32_t) * LR);
    h->off_s = take(sizeof(float) * LR);
    h->off_d = take(sizeof(float) * LR);
    h->off_nrem = take(path * sizeof(int32_t) * (size_t)p.L * dmax * p.R);
    h->off_t12 = take(path * sizeof(float) * (size_t)p.L * p.E * 2 * p.R);
    h->off_kt = take(sizeof(float) * (size_t)p.L * (size_t)h->kcap_global);
    h->off_dc = take(path * sizeof(int32_t) * LR * h->nc * ((size_t)p.E + (size_t)p.R * p.K + 1));
    h->off_cyc = take(path * sizeof(long long) * (size_t)p.L * 16);
    h->off_tc = take((p.R > 256 && p.R % 128 == 0) ? sizeof(float) * taot_sinkhorn_tc_ws_floats(p.R, p.L) : 0);
    h->tb_ok = (path && p.E <= 256 && h->seg % 16 == 0) ? 1 : 0;
    h->off_tb = take(h->tb_ok ? (size_t)p.L * (size_t)p.T * p.k : 0);
    h->off_tbflag = take(h->tb_ok ? sizeof(int32_t) * LR * h->nc : 0);
    h->ws_bytes = off;

    const size_t S = (size_t)p.R * p.K;
    off = 0;
    h->hoff_topk = take(sizeof(int32_t) * (size_t)p.L * p.T * p.k);
    h->hoff_new = take(sizeof(int32_t) * (size_t)p.L * p.T * p.k);
    h->hoff_n = take(sizeof(int32_t) * LR * p.E);
    h->hoff_el = take(sizeof(int32_t) * (size_t)p.L * p.E);
    h->hoff_rl = take(sizeof(int32_t) * LR);
    h->hoff_ex = take(sizeof(int32_t) * LR);
    h->hoff_sp = take(sizeof(int32_t) * LR);
    h->hoff_plan = take(sizeof(float) * LR * p.R);
    h->hoff_it = take(sizeof(int32_t) * p.L);
    h->hoff_err = take(sizeof(float) * p.L);
    h->hoff_se = take(sizeof(int32_t) * p.L * S);
    h->hoff_st = take(sizeof(int32_t) * p.L * S);
    h->hoff_X = take(sizeof(int32_t) * LR * S);
    h->hoff_rounds = take(sizeof(int32_t) * p.L * 2);
    h->hoff_info = take(sizeof(int32_t) * p.L);
    h->hoff_ws = take(h->ws_bytes);
    h->host_ws_bytes = off;
}

inline char* at(void* base, size_t off) { return static_cast<char*>(base) + off; }

// View of handle h on layers [l0, l0 + Lg): every per-layer array of the workspace starts at the group's first layer.
taot_handle_s* make_view(const taot_handle_s* h, int g, int l0, int Lg)
{
    taot_handle_s* v = new taot_handle_s(*h);
    const taot_params& p = h->p;
    v->is_view = 1;
    v->ngroups = 0;
    v->p.L = Lg;
    const size_t R = p.R, E = p.E, S = (size_t)p.R * p.K, nc = h->nc, l = (size_t)l0;
    const size_t dmax = E < S ? E : S;
    v->off_cc += 4 * l * R * nc * E;
    v->off_excess += 4 * l * R;
    v->off_spare += 4 * l * R;
    v->off_s += 4 * l * R;
    v->off_d += 4 * l * R;
    v->off_nrem += 4 * l * dmax * R;
    v->off_t12 += 4 * l * E * 2 * R;
    v->off_dc += 4 * l * R * nc * (E + S + 1);
    v->off_cyc += 8 * l * 16;
    v->off_tb += l * (size_t)p.T * p.k;
    v->off_tbflag += 4 * l * R * nc;
    if (v->d_merge_part) v->d_merge_part += l * TAOT_MERGE_PARTS * E;
    if (v->d_merge_cnt) v->d_merge_cnt += l;
    return v;
}

}  // namespace

extern "C" {

const char* taot_status_string(int status)
{
    switch (status) {
        case TAOT_OK: return "ok";
        case TAOT_ERR_NULL: return "a required pointer is NULL";
        case TAOT_ERR_PARAM: return "a parameter is out of range";
        case TAOT_ERR_UNSUPPORTED: return "size not supported by this build";
        case TAOT_ERR_CUDA: return "a CUDA runtime call failed";
        case TAOT_ERR_ALIGN: return "a device pointer is misaligned";
        case TAOT_ERR_STATIC_CAPACITY:
            return "taot_histogram_static: L*R*chunks*E*4 bytes of per-chunk counts exceed the built-in "
                   "scratch (TAOT_STATIC_SCRATCH_BYTES); use taot_histogram with a workspace";
        default: return "unknown status";
    }
}

int taot_create(taot_handle_t* out, const taot_params* params, const int32_t* h_e2r, const float* h_C,
                const float* h_B)
{
    if (out) *out = nullptr;
    if (!out || !params || !h_e2r || !h_C) return TAOT_ERR_NULL;
    if (!valid_params(params)) return TAOT_ERR_PARAM;
    if (!supported_params(params)) return TAOT_ERR_UNSUPPORTED;
    const int R = params->R, E = params->E;
    for (int e = 0; e < E; ++e)
        if (h_e2r[e] < 0 || h_e2r[e] >= R) return TAOT_ERR_PARAM;
    for (int64_t q = 0; q < (int64_t)R * R; ++q)
        if (!std::isfinite(h_C[q]) || h_C[q] < 0.0f) return TAOT_ERR_PARAM;
    if (h_B)
        for (int64_t q = 0; q < (int64_t)R * R; ++q)
            if (!std::isfinite(h_B[q])) return TAOT_ERR_PARAM;

    taot_handle_s* h = new (std::nothrow) taot_handle_s();
    if (!h) return TAOT_ERR_CUDA;
    std::memset(h, 0, sizeof(*h));
    h->p = *params;
    if (h->p.check_every < 1) h->p.check_every = 1;
    if (cudaGetDevice(&h->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess) {
        delete h;
        return TAOT_ERR_CUDA;
    }
    layout(h);

    // topology preference: given, or derived from the cost tiers (1 at the cheapest off-diagonal
    // cost, c_min / C elsewhere, 0 on the diagonal)
    std::vector<float> B((size_t)R * R);
    if (h_B) {
        std::memcpy(B.data(), h_B, sizeof(float) * (size_t)R * R);
    } else {
        float cmin = INFINITY;
        for (int i = 0; i < R; ++i)
            for (int j = 0; j < R; ++j) {
                const float c = h_C[(size_t)i * R + j];
                if (i != j && c > 0.0f && c < cmin) cmin = c;
            }
        for (int i = 0; i < R; ++i)
            for (int j = 0; j < R; ++j) {
                const float c = h_C[(size_t)i * R + j];
                float b = 1.0f;
                if (i == j) b = 0.0f;
                else if (c > 0.0f && std::isfinite(cmin)) { b = cmin / c; if (b > 1.0f) b = 1.0f; }
                B[(size_t)i * R + j] = b;
            }
    }
    // distinct values of the auction bonus (B off the diagonal, 1 on it) and, per host and value,
    // the set of source ranks that have it
    std::vector<float> tierval;
    std::vector<uint32_t> tiermask;
    {
        std::vector<float> vals;
        for (int i = 0; i < R && (int)vals.size() <= TAOT_MAX_TIERS; ++i)
            for (int j = 0; j < R && (int)vals.size() <= TAOT_MAX_TIERS; ++j) {
                const float b3 = (i == j) ? 1.0f : B[(size_t)i * R + j];
                bool seen = false;
                for (float v : vals) seen |= (v == b3);
                if (!seen) vals.push_back(b3);
            }
        if ((int)vals.size() <= TAOT_MAX_TIERS) {
            for (size_t x = 0; x < vals.size(); ++x)
                for (size_t y = x + 1; y < vals.size(); ++y)
                    if (vals[y] > vals[x]) std::swap(vals[x], vals[y]);
            tierval = vals;
            const int W = (R + 31) / 32, Tn = (int)vals.size();
            tiermask.assign((size_t)R * Tn * W, 0u);
            for (int host = 0; host < R; ++host)
                for (int r = 0; r < R; ++r) {
                    const float b3 = (r == host) ? 1.0f : B[(size_t)r * R + host];
                    for (int t = 0; t < Tn; ++t)
                        if (vals[t] == b3) tiermask[((size_t)t * W + (r >> 5)) * R + host] |= 1u << (r & 31);
                }
        }
    }
    h->ntiers = (int32_t)tierval.size();
    // Every score a bid of the tiered auction can take is  tierval[t] - price_step * w  for a tier t and a win count
    // w in [0, S].  All (t, w) pairs are listed once, best score first (evaluated with the same two fp32 operations
    // the kernel uses), so that a slot walks the list instead of comparing tiers; pairs with the same score form a
    // group (bit 31 = "the next entry has the same score").  Entry: w << 8 | t.
    std::vector<uint32_t> bidlist;
    if (h->ntiers > 0 && params->price_step > 0.0f && R <= 256) {
        const int S = R * params->K;
        struct Pair { float sc; int t, w; };
        std::vector<Pair> pairs;
        pairs.reserve((size_t)h->ntiers * (S + 1));
        for (int t = 0; t < h->ntiers; ++t)
            for (int w = 0; w <= S; ++w) {
                volatile float price = params->price_step * (float)w;     // one rounding per operation
                volatile float sc = tierval[t] - price;
                pairs.push_back(Pair{sc, t, w});
            }
        std::stable_sort(pairs.begin(), pairs.end(), [](const Pair& x, const Pair& y) { return x.sc > y.sc; });
        bidlist.resize(pairs.size());
        for (size_t i = 0; i < pairs.size(); ++i) {
            const bool tie_next = i + 1 < pairs.size() && pairs[i + 1].sc == pairs[i].sc;
            bidlist[i] = ((uint32_t)pairs[i].w << 8) | (uint32_t)pairs[i].t | (tie_next ? 0x80000000u : 0u);
        }
    }
    h->nbid = (int32_t)bidlist.size();
    // a cost that depends only on "same node of 8 ranks / same rail group of 32 ranks / neither" lets the Sinkhorn
    // sums be taken tier by tier (sinkhorn_tiered.cu)
    h->tier_ok = 0;
    if (R == 256 || R == 512 || R == 1024) {
        // The block sizes are read off the first row: a node is the run of ranks at rank 0's cheapest off-diagonal
        // cost, a rail group the run up to the next change (a cost with two values only has no group tier: any group
        // size then gives the same sums, 32 is taken).  The whole matrix is then checked against that structure.
        const int shapes[4][2] = {{8, 32}, {4, 16}, {4, 32}, {16, 32}};
        int node = 1;
        while (node < R && h_C[node] == h_C[1]) ++node;
        int group = node;
        while (group < R && h_C[group] == h_C[node < R ? node : R - 1]) ++group;
        if (group >= R) group = 32 > node ? 32 : 2 * node;             // two tiers only
        for (int k = 0; k < 4 && !h->tier_ok; ++k) {
            if (shapes[k][0] != node || shapes[k][1] != group || R % group != 0) continue;
            const float c1 = h_C[1], c2 = h_C[node], c3 = h_C[group < R ? group : R - 1];
            bool ok = std::isfinite(c1) && std::isfinite(c2) && std::isfinite(c3);
            for (int i = 0; i < R && ok; ++i)
                for (int j = 0; j < R && ok; ++j) {
                    if (i == j) continue;
                    const float want = (i / node == j / node) ? c1 : ((i / group == j / group) ? c2 : c3);
                    ok = h_C[(size_t)i * R + j] == want;
                }
            if (ok) {
                h->tier_ok = 1;
                h->tier_node = node; h->tier_group = group;
                h->tier_cost[0] = c1; h->tier_cost[1] = c2; h->tier_cost[2] = c3;
            }
        }
    }
    // first Sinkhorn row update with v = 1 on every rank: log-sum-exp of -C_ij/eps over all j
    std::vector<double> lse0(R);
    for (int i = 0; i < R; ++i) {
        double mx = -INFINITY;
        for (int j = 0; j < R; ++j) {
            const double x = -(double)h_C[(size_t)i * R + j] / (double)params->eps;
            if (x > mx) mx = x;
        }
        double acc = 0.0;
        for (int j = 0; j < R; ++j) acc += std::exp(-(double)h_C[(size_t)i * R + j] / (double)params->eps - mx);
        lse0[i] = mx + std::log(acc);
    }
    // Gibbs kernel for the tensor-core solve (more than 256 ranks, no tier structure, exp(-C/eps) well inside fp32):
    // M and its transpose, each split into two TF32-exact parts (high: low 13 mantissa bits cleared; low: the rest,
    // again with 13 bits cleared)
    std::vector<float> gibbs;
    if (R > 256 && R % 128 == 0 && !h->tier_ok && !std::getenv("TAOT_NO_TENSOR_CORES")) {
        double worst = 0.0;
        for (size_t q = 0; q < (size_t)R * R; ++q) worst = std::max(worst, (double)h_C[q] / (double)params->eps);
        if (worst <= 20.0) {
            gibbs.resize(4 * (size_t)R * R);
            auto split = [](float x, float* hi, float* lo) {
                uint32_t b;
                std::memcpy(&b, &x, 4);
                b &= 0xFFFFE000u;
                std::memcpy(hi, &b, 4);
                float l = x - *hi;
                std::memcpy(&b, &l, 4);
                b &= 0xFFFFE000u;
                std::memcpy(lo, &b, 4);
            };
            for (int i = 0; i < R; ++i)
                for (int j = 0; j < R; ++j) {
                    const float m = (float)std::exp(-(double)h_C[(size_t)i * R + j] / (double)params->eps);
                    float hi, lo;
                    split(m, &hi, &lo);
                    gibbs[(size_t)i * R + j] = hi;
                    gibbs[(size_t)R * R + (size_t)i * R + j] = lo;
                    gibbs[2 * (size_t)R * R + (size_t)j * R + i] = hi;
                    gibbs[3 * (size_t)R * R + (size_t)j * R + i] = lo;
                }
        }
    }
    // experts by home rank (CSR), ascending expert index inside a rank
    std::vector<int32_t> off(R + 1, 0), list(E);
    for (int e = 0; e < E; ++e) off[h_e2r[e] + 1]++;
    for (int r = 0; r < R; ++r) off[r + 1] += off[r];
    {
        std::vector<int32_t> cur(off.begin(), off.end() - 1);
        for (int e = 0; e < E; ++e) list[cur[h_e2r[e]]++] = e;
    }
    int rc = TAOT_OK;
    if (rc == TAOT_OK) rc = upload(&h->d_e2r, h_e2r, (size_t)E);
    if (rc == TAOT_OK) rc = upload(&h->d_C, h_C, (size_t)R * R);
    if (rc == TAOT_OK) rc = upload(&h->d_B, B.data(), (size_t)R * R);
    if (rc == TAOT_OK) rc = upload(&h->d_rowlse0, lse0.data(), (size_t)R);
    if (rc == TAOT_OK && !gibbs.empty()) rc = upload(&h->d_gibbs, gibbs.data(), gibbs.size());
    if (rc == TAOT_OK) rc = upload(&h->d_rank_off, off.data(), (size_t)R + 1);
    if (rc == TAOT_OK) rc = upload(&h->d_rank_list, list.data(), (size_t)E);
    if (rc == TAOT_OK && h->ntiers > 0) rc = upload(&h->d_tierval, tierval.data(), tierval.size());
    if (rc == TAOT_OK && R <= 256) {
        // targets (experts, then guest slots) in the order of the send buffer: by destination rank, then by index
        const int K = params->K, NT = E + R * K;
        std::vector<int32_t> tdest(NT + 1), torder(NT + 1), tpos(NT + 1), fill(R + 1, 0);
        for (int t = 0; t < NT; ++t) tdest[t] = t < E ? h_e2r[t] : (t - E) / K;
        tdest[NT] = R;
        for (int t = 0; t <= NT; ++t) fill[tdest[t]]++;
        int32_t run = 0;
        for (int q = 0; q <= R; ++q) { const int32_t c = fill[q]; fill[q] = run; run += c; }
        for (int t = 0; t <= NT; ++t) { tpos[t] = fill[tdest[t]]++; torder[tpos[t]] = t; }   // ascending t inside a rank
        rc = upload(&h->d_tpos, tpos.data(), tpos.size());
        if (rc == TAOT_OK) rc = upload(&h->d_torder, torder.data(), torder.size());
        if (rc == TAOT_OK) rc = upload(&h->d_tdest, tdest.data(), tdest.size());
    }
    if (rc == TAOT_OK && h->ntiers > 0) rc = upload(&h->d_tiermask, tiermask.data(), tiermask.size());
    if (rc == TAOT_OK && h->nbid > 0) rc = upload(&h->d_bidlist, bidlist.data(), bidlist.size());
    // the merge of a layer's chunk counts is shared by several CTAs where a layer has enough of them (the kernel sits in
    // the chain of latency-bound stages): their partial expert loads and a counter of finished parts per layer
    if (rc == TAOT_OK && R % (32 * TAOT_MERGE_PARTS) == 0) {
        const size_t parts = (size_t)params->L * TAOT_MERGE_PARTS * E;
        if (cudaMalloc(reinterpret_cast<void**>(&h->d_merge_part), sizeof(int32_t) * parts) != cudaSuccess ||
            cudaMalloc(reinterpret_cast<void**>(&h->d_merge_cnt), sizeof(int32_t) * params->L) != cudaSuccess ||
            cudaMemset(h->d_merge_cnt, 0, sizeof(int32_t) * params->L) != cudaSuccess)
            rc = TAOT_ERR_CUDA;
    }
    for (int i = 0; i < 6 && rc == TAOT_OK; ++i)
        if (cudaEventCreate(&h->ev[i]) != cudaSuccess) rc = TAOT_ERR_CUDA;
    // Layer groups for taot_plan: only where every group's routing table still keeps the memory system busy (more
    // chunks than three waves of the per-chunk kernels), i.e. where there are bandwidth-bound stages to hide
    if (rc == TAOT_OK && R <= 256) {
        int G = TAOT_MAX_GROUPS;
        if (const char* env = std::getenv("TAOT_PLAN_GROUPS")) {      // tuning knob: cap on the number of groups (1 = never split)
            const int cap = std::atoi(env);
            if (cap >= 1 && cap < G) G = cap;
        }
        const int64_t chunks_per_layer = (int64_t)R * h->nc;
        while (G > 1 && (params->L < 2 * G || (params->L / G) * chunks_per_layer <= 3 * (int64_t)h->sm_count)) --G;
        if (G > 1) {
            if (cudaEventCreate(&h->ev_fork) != cudaSuccess) rc = TAOT_ERR_CUDA;      // timed: origin of the group trace
            // (only where a group's chain of latency-bound stages outlasts the copy of the whole table: 256 ranks)
            if (rc == TAOT_OK && h->tb_ok && R >= 256 && cudaStreamCreateWithFlags(&h->bstream, cudaStreamNonBlocking) != cudaSuccess) rc = TAOT_ERR_CUDA;
            // Group sizes grow: a group's chain of latency-bound stages takes about as long whatever its size, so a
            // group can only finish (and rewrite its part of the table) under the others' chains if it started
            // earlier by about the time its reassignment takes; the stagger of the starts is the histogram of the
            // group itself.  Measured on configs 3 and 4: 2 : 3 : 5 : 8 best with four groups, 2 : 3 : 4 : 6 : 9 with
            // five, 3 : 4 : 5 : 6 : 8 : 10 with six (and six about 2 % faster than four where the table is large enough
            // for six).  At 256 ranks the chain (a thousand Sinkhorn iterations, two thousand auction rounds) is several
            // times as long as all bandwidth-bound work together, and since the reassignment reads one byte per entry
            // it is short enough to fit behind the other groups' chains whatever the order: equal sizes, which keep
            // the last chain's own reassignment small, measured 1.88 ms against 1.95 ms with growing sizes at config 4
            // (config 3, 64 ranks: 0.82 ms growing, 0.84 ms equal).
            static const double kWeights[4][TAOT_MAX_GROUPS] = {
                {2.0, 3.0, 5.0, 8.0, 0.0, 0.0}, {2.0, 3.0, 4.0, 6.0, 9.0, 0.0}, {3.0, 4.0, 5.0, 6.0, 8.0, 10.0},
                {1.0, 1.0, 1.0, 1.0, 1.0, 1.0}};
            const double* wt = kWeights[G <= 4 ? 0 : ((G == 6 && R >= 256) ? 3 : G - 4)];
            double wsum = 0.0;
            for (int g = 0; g < G; ++g) wsum += wt[g];
            int l0 = 0;
            double acc = 0.0;
            for (int g = 0; g < G && rc == TAOT_OK; ++g) {
                acc += wt[g];
                int end = g + 1 == G ? params->L : (int)std::lround(params->L * acc / wsum);
                if (end < l0 + 1) end = l0 + 1;
                if (end > params->L - (G - 1 - g)) end = params->L - (G - 1 - g);
                const int Lg = end - l0;
                h->group_len[g] = Lg;
                h->group_l0[g] = l0;
                l0 += Lg;
                if (g > 0 && cudaStreamCreateWithFlags(&h->gstream[g], cudaStreamNonBlocking) != cudaSuccess) rc = TAOT_ERR_CUDA;
                if (rc == TAOT_OK && cudaEventCreateWithFlags(&h->ev_hist[g], cudaEventDisableTiming) != cudaSuccess) rc = TAOT_ERR_CUDA;
                if (rc == TAOT_OK && cudaEventCreateWithFlags(&h->ev_join[g], cudaEventDisableTiming) != cudaSuccess) rc = TAOT_ERR_CUDA;
                if (rc == TAOT_OK && cudaEventCreateWithFlags(&h->ev_bytes[g], cudaEventDisableTiming) != cudaSuccess) rc = TAOT_ERR_CUDA;
                h->ngroups = g + 1;
            }
        }
    }
    if (rc == TAOT_OK && cudaDeviceSynchronize() != cudaSuccess) rc = TAOT_ERR_CUDA;
    if (rc != TAOT_OK) {
        taot_destroy(h);
        return rc;
    }
    // the views copy the finished handle (every device pointer is in place by now)
    for (int g = 0; g < h->ngroups; ++g) {
        h->group[g] = make_view(h, g, h->group_l0[g], h->group_len[g]);
        for (int i = 0; i < 6; ++i) {          // the group's own stage events (profiling level 3)
            h->group[g]->ev[i] = nullptr;
            if (cudaEventCreate(&h->group[g]->ev[i]) != cudaSuccess) { taot_destroy(h); return TAOT_ERR_CUDA; }
        }
    }
    *out = h;
    return TAOT_OK;
}

int taot_destroy(taot_handle_t h)
{
    if (!h) return TAOT_OK;
    cudaDeviceSynchronize();
    for (int g = 0; g < TAOT_MAX_GROUPS; ++g) {
        if (h->group[g])
            for (int i = 0; i < 6; ++i)
                if (h->group[g]->ev[i]) cudaEventDestroy(h->group[g]->ev[i]);
        delete h->group[g];                    // a view owns nothing but its stage events
        if (h->gstream[g]) cudaStreamDestroy(h->gstream[g]);
        if (h->ev_hist[g]) cudaEventDestroy(h->ev_hist[g]);
        if (h->ev_join[g]) cudaEventDestroy(h->ev_join[g]);
        if (h->ev_bytes[g]) cudaEventDestroy(h->ev_bytes[g]);
    }
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->bstream) cudaStreamDestroy(h->bstream);
    cudaFree(h->d_e2r); cudaFree(h->d_C); cudaFree(h->d_B); cudaFree(h->d_rowlse0); cudaFree(h->d_gibbs);
    cudaFree(h->d_rank_off); cudaFree(h->d_rank_list); cudaFree(h->d_tierval); cudaFree(h->d_tiermask);
    cudaFree(h->d_tpos); cudaFree(h->d_torder); cudaFree(h->d_tdest); cudaFree(h->d_bidlist);
    cudaFree(h->d_merge_part); cudaFree(h->d_merge_cnt);
    for (int i = 0; i < 6; ++i)
        if (h->ev[i]) cudaEventDestroy(h->ev[i]);
    delete h;
    return TAOT_OK;
}

int taot_workspace_bytes(taot_handle_t h, size_t* bytes)
{
    if (!h || !bytes) return TAOT_ERR_NULL;
    *bytes = h->ws_bytes;
    return TAOT_OK;
}

int taot_host_workspace_bytes(taot_handle_t h, size_t* bytes)
{
    if (!h || !bytes) return TAOT_ERR_NULL;
    *bytes = h->host_ws_bytes;
    return TAOT_OK;
}

int taot_set_profiling(taot_handle_t h, int32_t on)
{
    if (!h) return TAOT_ERR_NULL;
    h->profiling = on < 0 ? 0 : (on > 3 ? 3 : on);
    return TAOT_OK;
}

int taot_get_stage_ms(taot_handle_t h, float* h_ms)
{
    if (!h || !h_ms) return TAOT_ERR_NULL;
    TAOT_CUDA_OK(cudaEventSynchronize(h->ev[5]));
    for (int i = 0; i < 5; ++i) TAOT_CUDA_OK(cudaEventElapsedTime(h_ms + i, h->ev[i], h->ev[i + 1]));
    return TAOT_OK;
}

int taot_get_match_cycles(taot_handle_t h, const void* ws, int64_t* h_cycles)
{
    if (!h || !ws || !h_cycles) return TAOT_ERR_NULL;
    if (h->p.R > 256) return TAOT_ERR_UNSUPPORTED;
    TAOT_CUDA_OK(cudaMemcpy(h_cycles, static_cast<const char*>(ws) + h->off_cyc, sizeof(int64_t) * (size_t)h->p.L * 16,
                            cudaMemcpyDeviceToHost));
    return TAOT_OK;
}

int taot_get_group_trace(taot_handle_t h, int32_t* groups, float* h_ms)
{
    if (!h || !groups || !h_ms) return TAOT_ERR_NULL;
    *groups = h->ngroups > 1 ? h->ngroups : 0;
    for (int g = 0; g < *groups; ++g) {
        TAOT_CUDA_OK(cudaEventSynchronize(h->group[g]->ev[5]));
        for (int i = 0; i < 6; ++i) TAOT_CUDA_OK(cudaEventElapsedTime(h_ms + g * 6 + i, h->ev_fork, h->group[g]->ev[i]));
    }
    return TAOT_OK;
}

int taot_tier_structure(taot_handle_t h, int32_t* node, int32_t* group)
{
    if (!h || !node || !group) return TAOT_ERR_NULL;
    *node = h->tier_ok ? h->tier_node : 0;
    *group = h->tier_ok ? h->tier_group : 0;
    return TAOT_OK;
}

int taot_last_launch_count(taot_handle_t h, int32_t* count)
{
    if (!h || !count) return TAOT_ERR_NULL;
    *count = h->last_launches;
    return TAOT_OK;
}

int taot_histogram(taot_handle_t h, const int32_t* d_topk, int32_t* d_n, int32_t* d_expert_load,
                   int32_t* d_rank_load, int32_t* d_info, void* ws, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;      // beyond 256 ranks only Phase 1 is built
    if (!h || !d_topk || !d_n || !d_expert_load || !d_rank_load || !d_info || !ws) return TAOT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(d_topk) & 3) || (reinterpret_cast<uintptr_t>(ws) & 255)) return TAOT_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* cc = reinterpret_cast<int32_t*>(at(ws, h->off_cc));
    int a = taot_launch_histogram(h, d_topk, cc, d_info, st, ws);
    if (a < 0) return a;
    int b = taot_launch_merge(h, cc, d_n, d_expert_load, d_rank_load, nullptr, nullptr, nullptr, nullptr, st);
    if (b < 0) return b;
    h->last_launches = a + b;
    return TAOT_OK;
}

int taot_excess_spare(taot_handle_t h, const int32_t* d_rank_load, int32_t B, int32_t* d_excess,
                      int32_t* d_spare, float* d_s, float* d_d, void* stream)
{
    if (!h || !d_rank_load) return TAOT_ERR_NULL;
    if (B < 1) return TAOT_ERR_PARAM;
    int a = taot_launch_excess_spare(h, d_rank_load, B, d_excess, d_spare, d_s, d_d, static_cast<cudaStream_t>(stream));
    if (a < 0) return a;
    h->last_launches = a;
    return TAOT_OK;
}

int taot_sinkhorn(taot_handle_t h, const float* d_s, const float* d_d, int32_t B, float* d_plan,
                  int32_t* d_iters, float* d_row_err, int32_t* d_info, void* ws, void* stream)
{
    if (!h || !d_s || !d_d || !d_plan || !d_iters || !d_row_err || !d_info) return TAOT_ERR_NULL;
    if (B < 1) return TAOT_ERR_PARAM;
    if (h->kcap_global > 0 && (!ws || (reinterpret_cast<uintptr_t>(ws) & 255))) return ws ? TAOT_ERR_ALIGN : TAOT_ERR_NULL;
    int a = taot_launch_sinkhorn(h, d_s, d_d, B, d_plan, d_iters, d_row_err, d_info,
                                 ws ? reinterpret_cast<float*>(at(ws, h->off_kt)) : nullptr,
                                 static_cast<cudaStream_t>(stream),
                                 ws ? reinterpret_cast<float*>(at(ws, h->off_tc)) : nullptr);
    if (a < 0) return a;
    // s and d are the caller's here: problems with a NaN or an infinity in them are closed out after the solve
    int g = taot_launch_sinkhorn_guard(h, d_s, d_d, B, d_plan, d_iters, d_row_err, d_info, static_cast<cudaStream_t>(stream));
    if (g < 0) return g;
    h->last_launches = a + g;
    return TAOT_OK;
}

int taot_match(taot_handle_t h, const int32_t* d_n, const int32_t* d_expert_load, const int32_t* d_rank_load,
               const float* d_plan, int32_t* d_slot_expert, int32_t* d_slot_tokens, int32_t* d_X,
               int32_t* d_rounds, int32_t* d_info, void* ws, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;      // beyond 256 ranks only Phase 1 is built
    if (!h || !d_n || !d_expert_load || !d_rank_load || !d_slot_expert || !d_slot_tokens || !d_X || !d_info || !ws)
        return TAOT_ERR_NULL;
    if (!d_plan && !(h->p.ablation & TAOT_ABLATE_HINT)) return TAOT_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return TAOT_ERR_ALIGN;
    int a = taot_launch_match(h, d_n, d_expert_load, d_rank_load, d_plan, d_slot_expert, d_slot_tokens, d_X,
                              d_rounds, d_info, reinterpret_cast<int32_t*>(at(ws, h->off_nrem)),
                              reinterpret_cast<float*>(at(ws, h->off_t12)), static_cast<cudaStream_t>(stream),
                              (h->profiling & 2) ? reinterpret_cast<long long*>(at(ws, h->off_cyc)) : nullptr);
    if (a < 0) return a;
    h->last_launches = a;
    return TAOT_OK;
}

int taot_dispatch(taot_handle_t h, const int32_t* d_new_idx, int32_t* d_send_counts, int32_t* d_target_counts,
                  int32_t* d_perm, int32_t* d_info, void* ws, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;
    if (!h || !d_new_idx || !d_send_counts || !d_perm || !d_info || !ws) return TAOT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(d_new_idx) & 3) || (reinterpret_cast<uintptr_t>(d_perm) & 3) ||
        (reinterpret_cast<uintptr_t>(ws) & 255))
        return TAOT_ERR_ALIGN;
    if (d_new_idx == d_perm) return TAOT_ERR_PARAM;
    int a = taot_launch_dispatch(h, d_new_idx, d_send_counts, d_target_counts, d_perm, d_info, ws,
                                 static_cast<cudaStream_t>(stream));
    if (a < 0) return a;
    h->last_launches = a;
    return TAOT_OK;
}

int taot_report(taot_handle_t h, const int32_t* d_expert_load, const int32_t* d_rank_load,
                const int32_t* d_slot_expert, const int32_t* d_X, double lambda, taot_report_row* d_rows,
                int32_t* d_spill, int32_t* d_load_after, int32_t* d_slot_moved, int32_t* d_slot_kind, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;
    if (!h || !d_expert_load || !d_rank_load || !d_slot_expert || !d_X || !d_rows) return TAOT_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_rows) & 7) return TAOT_ERR_ALIGN;
    if (!std::isfinite(lambda)) return TAOT_ERR_PARAM;
    int a = taot_launch_report(h, d_expert_load, d_rank_load, d_slot_expert, d_X, lambda, d_rows, d_spill,
                               d_load_after, d_slot_moved, d_slot_kind, static_cast<cudaStream_t>(stream));
    if (a < 0) return a;
    h->last_launches = a;
    return TAOT_OK;
}

int taot_assign(taot_handle_t h, const int32_t* d_topk, const int32_t* d_slot_expert, const int32_t* d_X,
                int32_t* d_new_idx, int32_t* d_info, void* ws, int32_t reuse_counts, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;      // beyond 256 ranks only Phase 1 is built
    if (!h || !d_topk || !d_slot_expert || !d_X || !d_new_idx || !d_info || !ws) return TAOT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(d_topk) & 3) || (reinterpret_cast<uintptr_t>(d_new_idx) & 3) ||
        (reinterpret_cast<uintptr_t>(ws) & 255))
        return TAOT_ERR_ALIGN;
    if (d_topk == d_new_idx) return TAOT_ERR_PARAM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* cc = reinterpret_cast<int32_t*>(at(ws, h->off_cc));
    int launches = 0;
    if (!reuse_counts) {
        int a = taot_launch_histogram(h, d_topk, cc, d_info, st, ws);
        if (a < 0) return a;
        launches += a;
    }
    int b = taot_launch_assign(h, d_topk, ws, d_slot_expert, d_X, d_new_idx, d_info, st);
    if (b < 0) return b;
    h->last_launches = launches + b;
    return TAOT_OK;
}

}  // extern "C"

namespace {

// The five stages for the layers of one handle (or of one view of it) on one stream.  `hist_after`, if set, is waited for
// before the chunk histogram starts and `hist_done`, if set, is recorded after it: consecutive layer groups start
// their bandwidth-bound first stage one after the other instead of sharing the memory system.
// `bytes_later`: the one-byte copy of the table is not made by the histogram pass and the reassignment is left out --
// the caller makes the copy elsewhere and then calls assign_stage.
int plan_stages(taot_handle_t h, const int32_t* d_topk, const taot_outputs* o, void* ws, cudaStream_t st, bool marks,
                cudaEvent_t hist_after, cudaEvent_t hist_done, int* launches, bool bytes_later = false)
{
    const taot_params& p = h->p;
    int32_t* cc = reinterpret_cast<int32_t*>(at(ws, h->off_cc));
    int32_t* excess = o->excess ? o->excess : reinterpret_cast<int32_t*>(at(ws, h->off_excess));
    int32_t* spare = o->spare ? o->spare : reinterpret_cast<int32_t*>(at(ws, h->off_spare));
    float* fs = reinterpret_cast<float*>(at(ws, h->off_s));
    float* fd = reinterpret_cast<float*>(at(ws, h->off_d));
    TAOT_CUDA_OK(cudaMemsetAsync(o->info, 0, sizeof(int32_t) * p.L, st));
    int total = 0, a;
#define TAOT_MARK(i) if (marks) TAOT_CUDA_OK(cudaEventRecord(h->ev[i], st))
    // NVTX ranges around the enqueue of each stage (header-only NVTX: free unless a profiler is attached)
    struct Range {
        explicit Range(const char* name) { nvtxRangePushA(name); }
        ~Range() { nvtxRangePop(); }
    };
    TAOT_MARK(0);
    if (hist_after) TAOT_CUDA_OK(cudaStreamWaitEvent(st, hist_after, 0));
    {
        Range r("taot:histogram");
        if ((a = taot_launch_histogram(h, d_topk, cc, o->info, st, ws, !bytes_later)) < 0) return a;
    }
    total += a;
    if (hist_done) TAOT_CUDA_OK(cudaEventRecord(hist_done, st));
    TAOT_MARK(1);
    {
        Range r("taot:merge+excess_spare");
        if ((a = taot_launch_merge(h, cc, o->n, o->expert_load, o->rank_load, excess, spare, fs, fd, st)) < 0) return a;
    }
    total += a;
    TAOT_MARK(2);
    nvtxRangePushA("taot:sinkhorn");
    if (p.ablation & TAOT_ABLATE_HINT) {       // Phase 1 switched off: no solve, a zero hint
        TAOT_CUDA_OK(cudaMemsetAsync(o->plan, 0, sizeof(float) * (size_t)p.L * p.R * p.R, st));
        TAOT_CUDA_OK(cudaMemsetAsync(o->sinkhorn_iters, 0, sizeof(int32_t) * p.L, st));
        TAOT_CUDA_OK(cudaMemsetAsync(o->row_err, 0, sizeof(float) * p.L, st));
        a = 0;
    } else if ((a = taot_launch_sinkhorn(h, fs, fd, p.L, o->plan, o->sinkhorn_iters, o->row_err, o->info,
                                         reinterpret_cast<float*>(at(ws, h->off_kt)), st)) < 0) {
        nvtxRangePop();
        return a;
    }
    nvtxRangePop();
    total += a;
    TAOT_MARK(3);
    nvtxRangePushA("taot:match+auction");
    if ((a = taot_launch_match(h, o->n, o->expert_load, o->rank_load, o->plan, o->slot_expert, o->slot_tokens,
                               o->X, o->rounds, o->info, reinterpret_cast<int32_t*>(at(ws, h->off_nrem)),
                               reinterpret_cast<float*>(at(ws, h->off_t12)), st,
                               (marks && (h->profiling & 2)) ? reinterpret_cast<long long*>(at(ws, h->off_cyc)) : nullptr)) < 0) {
        nvtxRangePop();
        return a;
    }
    nvtxRangePop();
    total += a;
    TAOT_MARK(4);
    if (!bytes_later) {
        Range r("taot:reassignment");
        if ((a = taot_launch_assign(h, d_topk, ws, o->slot_expert, o->X, o->new_idx, o->info, st)) < 0) return a;
        total += a;
        TAOT_MARK(5);
    }
#undef TAOT_MARK
    *launches += total;
    return TAOT_OK;
}

// The last stage on its own, for a call whose plan_stages left it out.
int assign_stage(taot_handle_t h, const int32_t* d_topk, const taot_outputs* o, void* ws, cudaStream_t st, bool marks,
                 int* launches)
{
    nvtxRangePushA("taot:reassignment");
    const int a = taot_launch_assign(h, d_topk, ws, o->slot_expert, o->X, o->new_idx, o->info, st);
    nvtxRangePop();
    if (a < 0) return a;
    if (marks) TAOT_CUDA_OK(cudaEventRecord(h->ev[5], st));
    *launches += a;
    return TAOT_OK;
}

// the outputs of layers [l0, ...) of a call
taot_outputs outputs_from_layer(const taot_params& p, const taot_outputs* o, int l0)
{
    const size_t l = (size_t)l0, R = p.R, E = p.E, S = (size_t)p.R * p.K;
    taot_outputs g = *o;
    g.n += l * R * E; g.expert_load += l * E; g.rank_load += l * R;
    if (g.excess) g.excess += l * R;
    if (g.spare) g.spare += l * R;
    g.plan += l * R * R; g.sinkhorn_iters += l; g.row_err += l;
    g.slot_expert += l * S; g.slot_tokens += l * S; g.X += l * R * S;
    if (g.rounds) g.rounds += l * 2;
    g.new_idx += l * (size_t)p.T * p.k; g.info += l;
    return g;
}

}  // namespace

extern "C" {

int taot_plan(taot_handle_t h, const int32_t* d_topk, const taot_outputs* o, void* ws, void* stream)
{
    if (h && h->p.R > 256) return TAOT_ERR_UNSUPPORTED;      // beyond 256 ranks only Phase 1 is built
    if (!h || !d_topk || !o || !ws) return TAOT_ERR_NULL;
    if (!o->n || !o->expert_load || !o->rank_load || !o->plan || !o->sinkhorn_iters || !o->row_err ||
        !o->slot_expert || !o->slot_tokens || !o->X || !o->new_idx || !o->info)
        return TAOT_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(d_topk) & 3) || (reinterpret_cast<uintptr_t>(o->new_idx) & 3) ||
        (reinterpret_cast<uintptr_t>(ws) & 255))
        return TAOT_ERR_ALIGN;
    if (d_topk == o->new_idx) return TAOT_ERR_PARAM;
    const taot_params& p = h->p;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int total = 0;
    if (h->ngroups <= 1 || (h->profiling && h->profiling != 3)) {
        // one group on the caller's stream (always when stage times are asked for: they are only defined here)
        const int rc = plan_stages(h, d_topk, o, ws, st, h->profiling != 0, nullptr, nullptr, &total);
        if (rc != TAOT_OK) return rc;
        h->last_launches = total;
        return TAOT_OK;
    }
    // Layer groups: group 0 on the caller's stream, the others on the handle's streams, forked from the caller's
    // stream by an event and joined back into it by one event each; no allocation, no synchronisation, and the fork /
    // join pattern is what stream capture expects.
    TAOT_CUDA_OK(cudaEventRecord(h->ev_fork, st));
    const bool side_bytes = h->bstream != nullptr && h->tb_ok && (reinterpret_cast<uintptr_t>(d_topk) & 15) == 0 &&
                            (reinterpret_cast<uintptr_t>(o->new_idx) & 15) == 0;
    for (int g = 0; g < h->ngroups; ++g) {
        taot_handle_s* v = h->group[g];
        const int l0 = h->group_l0[g];
        cudaStream_t gs = g == 0 ? st : h->gstream[g];
        if (g > 0) TAOT_CUDA_OK(cudaStreamWaitEvent(gs, h->ev_fork, 0));
        const taot_outputs go = outputs_from_layer(p, o, l0);
        const int rc = plan_stages(v, d_topk + (size_t)l0 * p.T * p.k, &go, ws, gs, h->profiling == 3,
                                   g > 0 ? h->ev_hist[g - 1] : nullptr,
                                   (g + 1 < h->ngroups || side_bytes) ? h->ev_hist[g] : nullptr, &total, side_bytes);
        if (rc != TAOT_OK) return rc;
        if (g > 0 && !side_bytes) TAOT_CUDA_OK(cudaEventRecord(h->ev_join[g], gs));
    }
    if (side_bytes) {
        // The one-byte copies the reassignment reads are made on a stream of their own once every histogram is done (the
        // memory system is idle from then until the first matching ends), by a grid too small to get in the way of the
        // chains; each group's reassignment waits for its copy.
        TAOT_CUDA_OK(cudaStreamWaitEvent(h->bstream, h->ev_hist[h->ngroups - 1], 0));
        for (int g = 0; g < h->ngroups; ++g) {
            const int a = taot_launch_table_bytes(h->group[g], d_topk + (size_t)h->group_l0[g] * p.T * p.k, ws, h->bstream);
            if (a < 0) return a;
            total += a;
            TAOT_CUDA_OK(cudaEventRecord(h->ev_bytes[g], h->bstream));
        }
        for (int g = 0; g < h->ngroups; ++g) {
            cudaStream_t gs = g == 0 ? st : h->gstream[g];
            const taot_outputs go = outputs_from_layer(p, o, h->group_l0[g]);
            TAOT_CUDA_OK(cudaStreamWaitEvent(gs, h->ev_bytes[g], 0));
            const int rc = assign_stage(h->group[g], d_topk + (size_t)h->group_l0[g] * p.T * p.k, &go, ws, gs,
                                        h->profiling == 3, &total);
            if (rc != TAOT_OK) return rc;
            if (g > 0) TAOT_CUDA_OK(cudaEventRecord(h->ev_join[g], gs));
        }
    }
    for (int g = 1; g < h->ngroups; ++g) TAOT_CUDA_OK(cudaStreamWaitEvent(st, h->ev_join[g], 0));
    h->last_launches = total;
    return TAOT_OK;
}

// H2D copy of the routing table, the whole path on device staging buffers; `d` receives the device pointers
static int plan_on_staging(taot_handle_t h, const int32_t* h_topk, void* d_ws, void* stream, taot_outputs* d)
{
    const taot_params& p = h->p;
    if (p.R > 256) return TAOT_ERR_UNSUPPORTED;      // what taot_plan would refuse is refused before the copy is queued
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t NE = (size_t)p.L * p.T * p.k;
    d->n = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_n));
    d->expert_load = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_el));
    d->rank_load = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_rl));
    d->excess = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_ex));
    d->spare = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_sp));
    d->plan = reinterpret_cast<float*>(at(d_ws, h->hoff_plan));
    d->sinkhorn_iters = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_it));
    d->row_err = reinterpret_cast<float*>(at(d_ws, h->hoff_err));
    d->slot_expert = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_se));
    d->slot_tokens = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_st));
    d->X = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_X));
    d->rounds = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_rounds));
    d->new_idx = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_new));
    d->info = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_info));
    int32_t* d_topk = reinterpret_cast<int32_t*>(at(d_ws, h->hoff_topk));
    TAOT_CUDA_OK(cudaMemcpyAsync(d_topk, h_topk, sizeof(int32_t) * NE, cudaMemcpyHostToDevice, st));
    return taot_plan(h, d_topk, d, at(d_ws, h->hoff_ws), stream);
}

int taot_plan_host(taot_handle_t h, const int32_t* h_topk, const taot_outputs* o, void* d_ws, void* stream)
{
    if (!h || !h_topk || !o || !d_ws) return TAOT_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_ws) & 255) return TAOT_ERR_ALIGN;
    const taot_params& p = h->p;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t LR = (size_t)p.L * p.R, S = (size_t)p.R * p.K, NE = (size_t)p.L * p.T * p.k;
    taot_outputs d;
    const int rc = plan_on_staging(h, h_topk, d_ws, stream, &d);
    if (rc != TAOT_OK) return rc;
#define TAOT_BACK(member, count, type)                                                                       \
    if (o->member)                                                                                           \
        TAOT_CUDA_OK(cudaMemcpyAsync(o->member, d.member, sizeof(type) * (count), cudaMemcpyDeviceToHost, st))
    TAOT_BACK(n, LR * p.E, int32_t);
    TAOT_BACK(expert_load, (size_t)p.L * p.E, int32_t);
    TAOT_BACK(rank_load, LR, int32_t);
    TAOT_BACK(excess, LR, int32_t);
    TAOT_BACK(spare, LR, int32_t);
    TAOT_BACK(plan, LR * p.R, float);
    TAOT_BACK(sinkhorn_iters, (size_t)p.L, int32_t);
    TAOT_BACK(row_err, (size_t)p.L, float);
    TAOT_BACK(slot_expert, p.L * S, int32_t);
    TAOT_BACK(slot_tokens, p.L * S, int32_t);
    TAOT_BACK(X, LR * S, int32_t);
    TAOT_BACK(rounds, (size_t)p.L * 2, int32_t);
    TAOT_BACK(new_idx, NE, int32_t);
    TAOT_BACK(info, (size_t)p.L, int32_t);
#undef TAOT_BACK
    return TAOT_OK;
}

int taot_host_block_layout(taot_handle_t h, size_t* offsets, size_t* bytes)
{
    if (!h || !offsets || !bytes) return TAOT_ERR_NULL;
    const size_t base = h->hoff_n;
    const size_t off[14] = {h->hoff_n, h->hoff_el, h->hoff_rl, h->hoff_ex, h->hoff_sp, h->hoff_plan, h->hoff_it,
                            h->hoff_err, h->hoff_se, h->hoff_st, h->hoff_X, h->hoff_rounds, 0, h->hoff_info};
    for (int i = 0; i < 14; ++i) offsets[i] = (i == 12) ? (size_t)-1 : off[i] - base;     // member 12 is new_idx
    *bytes = h->hoff_ws - base;
    return TAOT_OK;
}

int taot_plan_host_block(taot_handle_t h, const int32_t* h_topk, int32_t* h_new_idx, void* h_block, void* d_ws,
                         void* stream)
{
    if (!h || !h_topk || !h_new_idx || !h_block || !d_ws) return TAOT_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(d_ws) & 255) return TAOT_ERR_ALIGN;
    const taot_params& p = h->p;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t NE = (size_t)p.L * p.T * p.k;
    taot_outputs d;
    const int rc = plan_on_staging(h, h_topk, d_ws, stream, &d);
    if (rc != TAOT_OK) return rc;
    // the staging buffers of all outputs but the routing table are one contiguous range: one copy
    TAOT_CUDA_OK(cudaMemcpyAsync(h_block, at(d_ws, h->hoff_n), h->hoff_ws - h->hoff_n, cudaMemcpyDeviceToHost, st));
    TAOT_CUDA_OK(cudaMemcpyAsync(h_new_idx, d.new_idx, sizeof(int32_t) * NE, cudaMemcpyDeviceToHost, st));
    return TAOT_OK;
}

}  // extern "C"
