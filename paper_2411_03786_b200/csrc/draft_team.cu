// Context N-gram drafting for batches of short and medium histories: persistent CTAs whose warp teams pull
// sequences from a queue.
//
// A batch of many sequences is a throughput job, and what a one-CTA-per-sequence launch loses on it is not
// the scan but everything around it: table reset, grouping, ranking, mixing and the output are a chain of
// short phases separated by barriers and dependent loads, a few microseconds per sequence whatever its
// length, and the last wave of CTAs is ragged.  Here
//   - the grid is two CTAs per SM, launched once; each CTA is split into teams of T warps (T = 1, 2, 4, 8
//     or 16), every team owns a slice of shared memory with its own hash table and scratch, and
//     synchronises with a named barrier of its own (a team of one warp with __syncwarp), so the phases of
//     one sequence never stall another team;
//   - a team takes the next sequence from a global counter until none is left, so long and short sequences
//     balance and there is no ragged wave (the CTA that exits last re-arms the counter);
//   - the team first copies its sequence's history into its slice of shared memory (128-bit loads, all in
//     flight at once): the scan, the suffix and key comparisons of every match, the repeated passes of a
//     sequence with more groups than its table holds, and the candidate rows then read shared memory;
//   - T follows the batch and the history length: many short histories run one or two warps per sequence
//     (ten and more sequences in flight per SM), longer ones up to 16 warps;
//   - every group is ranked by counting, whatever the number of groups, and later passes rank their groups
//     together with the earlier winners the same way (see rank_pass).
// Semantics (matching, grouping, ranking, mixing, duplicates, model rows, status bits) are those of the
// latency kernel in draft.cu; results are bit-identical.
#include <stdlib.h>

#include "draft_common.cuh"

namespace ngs {

constexpr int TEAM_MAX_WARPS = 16;            // warps per CTA
constexpr int TEAM_SMEM_BUDGET = 112 * 1024;  // per CTA, so that two CTAs share an SM

// Byte offsets inside one team's slice of shared memory.
struct TeamLayout {
    int table;     // int rep[slots], cnt[slots], last[slots], grp_slot[max_groups]
    int gkey;      // u64 [gkey_cap]
    int rank;      // int [gkey_cap]
    int run_key;   // u64 [n_q][topk]
    int cand_rows; // int [n_cand_max][w]
    int cand;      // int cand_src | cand_cnt | cand_keep | dropped, each [n_cand_max]
    int row_of;    // int [B]
    int chain;     // int [k_tab][w] then chain_ok[k_tab]
    int queue;     // int [T][kMatchQueue]
    int misc;      // TeamMisc
    int hist;      // int [cap]: the sequence's history
    int bytes;     // size of the slice (multiple of 16)
    int n_cand_max;
    int gkey_cap;
    int teams;     // teams per CTA
};

struct TeamMisc {
    int seq;
    int n_groups;
    int overflow;
    int n_out;
    int n_run[kMaxNQ];
    int n_cnt[kMaxNQ];
    int tq[kMaxQ];
    int cand_off[kMaxNQ + 2];
    int n_surv;
    int reached;
    unsigned long long tau[kMaxNQ];
};

template <int T, bool PT>  // T warps per team; PT: SPEC_FLAG_PARTIAL_TAIL
__global__ void __launch_bounds__(TEAM_MAX_WARPS * 32, 2) draft_team_kernel(const DraftParams P, const TeamLayout Y, unsigned int* work) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int TT = T * 32;  // threads of a team
    // A team's warps are Y.teams apart: with four or eight teams per CTA they all sit on the same scheduler of
    // the SM and, running the same phase of the same sequence, share the instruction lines it has fetched.
    const int team = ((int)threadIdx.x >> 5) % Y.teams, warp = ((int)threadIdx.x >> 5) / Y.teams;
    const int lane = (int)threadIdx.x & 31, tid = warp * 32 + lane;
    unsigned char* base = smem_raw + (size_t)team * Y.bytes;
    TeamMisc* sm = reinterpret_cast<TeamMisc*>(base + Y.misc);
    DraftTable tab;
    tab.rep = reinterpret_cast<int*>(base + Y.table);
    tab.cnt = tab.rep + P.slots;
    tab.last = tab.cnt + P.slots;
    tab.grp_slot = tab.last + P.slots;
    tab.n_groups = &sm->n_groups;
    tab.overflow = &sm->overflow;
    DraftScratch X;
    X.gkey = reinterpret_cast<unsigned long long*>(base + Y.gkey);
    X.rank_acc = reinterpret_cast<int*>(base + Y.rank);
    X.run_key = reinterpret_cast<unsigned long long*>(base + Y.run_key);
    X.n_run = sm->n_run;
    X.n_cnt = sm->n_cnt;
    X.cand = reinterpret_cast<int32_t*>(base + Y.cand_rows);
    X.cand_src = reinterpret_cast<int*>(base + Y.cand);
    X.cand_cnt = X.cand_src + Y.n_cand_max;
    X.cand_keep = X.cand_cnt + Y.n_cand_max;
    X.dropped = X.cand_keep + Y.n_cand_max;
    X.row_of = reinterpret_cast<int*>(base + Y.row_of);
    X.chain = reinterpret_cast<int*>(base + Y.chain);
    X.chain_ok = X.chain + P.k_tab * P.w;
    X.cand_off = sm->cand_off;
    X.n_out = &sm->n_out;
    X.n_surv = &sm->n_surv;
    X.tau = sm->tau;
    int* wq = reinterpret_cast<int*>(base + Y.queue) + warp * kMatchQueue;  // this warp's queue of matches
    int32_t* hist_s = reinterpret_cast<int32_t*>(base + Y.hist);

    // barrier over the team: named barrier team + 1 (barrier 0 is the CTA's), or the warp's own
    auto team_sync = [&]() {
        if constexpr (T == 1) __syncwarp();
        else asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(TT) : "memory");
    };

    grid_launch_dependents();
    grid_dependency_wait();  // histories and lengths come from the previous step's commit; the counter from the previous batch

    for (;;) {
        if (tid == 0) sm->seq = (int)atomicAdd(&work[0], 1u);
        team_sync();
        const int s = *((volatile int*)&sm->seq);
        if (s >= P.S) break;
        const int32_t* __restrict__ hg = P.hist + (size_t)s * P.cap;
        int L = P.len[s];
        if (L < 0 || L > P.cap) {
            if (tid == 0) atomicOr(P.status, SPEC_STATUS_CAPACITY);
            L = 0;
        }
        {   // the history goes into shared memory: all of a thread's loads are issued before the first store
            const int4* g4 = reinterpret_cast<const int4*>(hg);
            int4* s4 = reinterpret_cast<int4*>(hist_s);
            const int n4 = (L + 3) >> 2;  // cap % 4 == 0 and L <= cap: the last vector stays inside the row
            for (int i0 = 0; i0 < n4; i0 += 8 * TT) {
                int4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TT + tid;
                    if (i < n4) v[u] = g4[i];
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int i = i0 + u * TT + tid;
                    if (i < n4) s4[i] = v[u];
                }
            }
        }
        team_sync();
        const int32_t* h = hist_s;
        if (tid < kMaxQ) sm->tq[tid] = (tid < L) ? h[L - 1 - tid] : -2;
        if (tid < kMaxNQ) sm->n_run[tid] = 0;
        if (tid < P.k_tab) X.chain_ok[tid] = 0;
        team_sync();

        // ---- extended model bigram of the last token (rank r on lane r), by the team's last warp
        if (warp == T - 1 && (P.flags & SPEC_FLAG_MODEL_FILL) && L >= 1) model_chain(P, sm->tq[0], lane, X.chain, X.chain_ok);

        // ---- context N-grams
        const int n_scan = L - P.w;
        const int t0 = sm->tq[0], t1 = sm->tq[1], t2 = sm->tq[2], t3 = sm->tq[3];
        constexpr bool partial = PT;
        bool any_q = false;
        for (int qi = 0; qi < P.n_q; ++qi) any_q = any_q || (L >= P.qs[qi] + (partial ? 1 : P.w));
        int R = 1;
        bool gave_up = false;
        while (any_q && (n_scan >= 1 || (partial && L >= 2))) {
            team_sync();
            if (tid < kMaxNQ) sm->n_run[tid] = 0;
            bool overflowed = false;
            for (int r = 0; r < R && !overflowed; ++r) {
                for (int i = tid; i < P.slots; i += TT) {
                    tab.rep[i] = -1;
                    tab.cnt[i] = 0;
                    tab.last[i] = -1;
                }
                if (tid == 0) {
                    sm->n_groups = 0;
                    sm->overflow = 0;
                }
                team_sync();
                const int reached = scan_pass<4, PT>(P, h, L, R, r, t0, t1, t2, t3, tab, wq, tid, TT);
                if (tid == 0) sm->reached = reached;
                team_sync();  // the team's matches are in the table
                if (*((volatile int*)&sm->overflow)) {
                    overflowed = true;
                    break;
                }
                rank_pass(P, tab, X, tid, TT, team_sync);
            }
            if (!overflowed) break;
            R = next_pass_count(R, sm->reached, (max(n_scan, 0) + 3) >> 2);
            if (R > kMaxPasses) {
                gave_up = true;
                break;
            }
        }
        mix_and_emit(P, s, h, L, gave_up, X, tid, TT, team_sync);
    }

    // The CTA that leaves last re-arms the work counter for the next batch.  (Every CTA has stopped taking
    // sequences by the time it counts itself out.)
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int done = atomicAdd(&work[1], 1u);
        if (done == gridDim.x - 1) {
            work[0] = 0u;
            work[1] = 0u;
        }
    }
}

static int round_up16(int x) { return (x + 15) & ~15; }

int launch_draft_team(spec_ctx* ctx, DraftParams& P, cudaStream_t st) {
    const int sms = ctx->num_sms;
    // Table: filled to at most three quarters (groups are found by linear probing from a mixed hash).  A query
    // of one token matches up to a tenth of the positions on natural token statistics and most of those
    // matches differ in their continuation (cap / 8 groups at the most on Zipf 1.1 over 32000 tokens), longer
    // queries around one in a hundred.  A table that overflows costs whole rescans, a larger table costs
    // sequences in flight (it is most of a team's shared memory): 4096 x 2048 tokens with a one-token query
    // take 128 us with 256 groups, 80 us with 512 groups in 1024 slots and less again with 384 groups in 512.
    const int expect = P.q_min >= 2 || P.n_q == 0 ? P.cap / 72 : P.cap / 6;
    int slots = 256;
    while (slots / 4 * 3 < expect && slots < 2048) slots <<= 1;
    P.slots = slots;
    P.max_groups = slots / 4 * 3;
    P.stage_hist = 1;
    P.hist_off = 0;
    // warps per team: enough teams per SM (of its 32 warps) to hold the batch's share of sequences
    const int per_sm = (P.S + sms - 1) / sms;
    int T = 16;
    while (T > 1 && 32 / T < per_sm) T >>= 1;
    // ... but at least a warp per 512 tokens of history (measured: 1024 tokens run best with two warps, 2048 with
    // four; a scan spread thinner leaves the sequence's serial phases to too few threads)
    int t_len = 1;
    while (t_len < 16 && t_len * 2 * 512 <= P.cap) t_len <<= 1;
    if (T < t_len) T = t_len;
#ifdef NGRAM_SPEC_TUNING
    if (const char* ov = getenv("NGRAM_SPEC_TEAM")) {  // tuning builds only: warps per team
        const int t = atoi(ov);
        if (t == 1 || t == 2 || t == 4 || t == 8 || t == 16) T = t;
    }
    if (const char* ov = getenv("NGRAM_SPEC_TEAM_SLOTS")) {  // ... and table slots
        const int t = atoi(ov);
        if (t >= 64 && t <= 4096 && (t & (t - 1)) == 0) {
            P.slots = t;
            P.max_groups = t / 4 * 3;
        }
    }
#endif
    TeamLayout Y{};
    Y.n_cand_max = P.n_q * P.topk + P.k_tab;
    Y.gkey_cap = P.max_groups + P.n_q * P.topk;
    for (;; T <<= 1) {
        int off = 0;
        Y.table = off;
        off += round_up16((P.slots * 3 + P.max_groups) * 4);
        Y.gkey = off;
        off += round_up16(Y.gkey_cap * 8);
        Y.rank = off;
        off += round_up16(Y.gkey_cap * 4);
        Y.run_key = off;
        off += round_up16((P.n_q > 0 ? P.n_q : 1) * P.topk * 8);
        Y.cand_rows = off;
        off += round_up16((Y.n_cand_max > 0 ? Y.n_cand_max : 1) * P.w * 4);
        Y.cand = off;
        off += round_up16(4 * (Y.n_cand_max > 0 ? Y.n_cand_max : 1) * 4);
        Y.row_of = off;
        off += round_up16(P.B * 4);
        Y.chain = off;
        off += round_up16((P.k_tab * P.w + kMaxKTab) * 4);
        Y.queue = off;
        off += round_up16(T * kMatchQueue * 4);
        Y.misc = off;
        off += round_up16((int)sizeof(TeamMisc));
        Y.hist = off;
        off += round_up16(P.cap * 4);
        Y.bytes = off;
        // teams per CTA: what fits beside each other (a team of several warps needs a named barrier of its own)
        int teams = TEAM_SMEM_BUDGET / Y.bytes;
        if (teams > TEAM_MAX_WARPS / T) teams = TEAM_MAX_WARPS / T;
        if (T > 1 && teams > 8) teams = 8;
        Y.teams = teams;
        if (teams == 1 && T < 16) continue;    // room for one sequence only: all 16 warps work on it
        if (teams * T >= 8 || T == 16) break;  // at least eight warps per CTA, or the largest team
    }
    if (Y.teams < 1) return kDraftNoFit;
    const size_t smem = (size_t)Y.teams * Y.bytes;
    using Kern = void (*)(const DraftParams, const TeamLayout, unsigned int*);
    static const Kern kerns[2][5] = {
        {draft_team_kernel<1, false>, draft_team_kernel<2, false>, draft_team_kernel<4, false>, draft_team_kernel<8, false>, draft_team_kernel<16, false>},
        {draft_team_kernel<1, true>, draft_team_kernel<2, true>, draft_team_kernel<4, true>, draft_team_kernel<8, true>, draft_team_kernel<16, true>}};
    const int pt = (P.flags & SPEC_FLAG_PARTIAL_TAIL) ? 1 : 0;
    const int ti0 = T == 1 ? 0 : T == 2 ? 1 : T == 4 ? 2 : T == 8 ? 3 : 4;
    const Kern kern = kerns[pt][ti0];
    {
        static bool attr_set[64][10] = {};
        const int ti = pt * 5 + ti0;
        std::lock_guard<std::mutex> lock(host_mutex());
        if (!attr_set[ctx->device & 63][ti]) {
            int rc = check_cuda(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TEAM_SMEM_BUDGET),
                                "draft (batch): cudaFuncSetAttribute");
            if (rc) return rc;
            attr_set[ctx->device & 63][ti] = true;
        }
    }
    // two CTAs per SM, but no more CTAs than there are sequences to start with
    long long grid = 2ll * sms;
    const long long want = ((long long)P.S + Y.teams - 1) / Y.teams;
    if (grid > want) grid = want;
    if (grid < 1) grid = 1;
    cudaError_t e = launch_pdl(kern, dim3((unsigned)grid), dim3((unsigned)(Y.teams * T * 32)), smem, st, P, Y, ctx->d_draft_work);
    ctx->launches += 1;
    return check_cuda(ctx, e, "draft_context_ngrams (batch) launch");
}

}  // namespace ngs
