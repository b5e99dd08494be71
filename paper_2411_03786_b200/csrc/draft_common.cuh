// Declarations shared by the two drafting kernels: the latency kernel (one CTA or one cluster per
// sequence, draft.cu) and the batch kernel (persistent CTAs whose warp teams pull sequences from a
// queue, draft_team.cu).
#pragma once
#include <type_traits>

#include "common.cuh"

namespace ngs {

struct DraftParams {
    const int32_t* hist;
    const int32_t* len;
    int S, cap;
    int qs[kMaxNQ];
    int n_q, q_max, q_min;
    int topk, B, w, flags;
    const int32_t* tab;
    int k_tab;
    const int32_t* ext;
    int w_ext;
    int V;
    int32_t* drafts;
    int32_t* ndrafts;
    int32_t* src;
    int32_t* counts;
    int* status;
    int slots;       // hash table size (power of two)
    int max_groups;  // groups one pass may open: half to three quarters of the slots
    int stage_hist;  // latency kernel: 1 = copy the history into shared memory first (single CTA, short history)
    int hist_off;    // where that copy lives, in ints from the start of the hash table
};

constexpr int kMaxPasses = 1024;
constexpr int kMaxCand = kMaxNQ * kMaxB + kMaxKTab;    // candidate rows before duplicates are dropped
constexpr int kMatchQueue = 128;                       // matches a warp queues before it groups them

__device__ __forceinline__ uint32_t fmix32(uint32_t h) {
    h ^= h >> 16;
    h *= 0x85EBCA6Bu;
    h ^= h >> 13;
    h *= 0xC2B2AE35u;
    h ^= h >> 16;
    return h;
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    return v;
}

// Token t of the continuation that starts at p.  With SPEC_FLAG_PARTIAL_TAIL (Lw = history length, else 0) a
// continuation that runs past the end of the history repeats the tokens it has.
__device__ __forceinline__ int cont_tok(const int32_t* __restrict__ h, int Lw, int p, int t) {
    int i = p + t;
    if (Lw != 0 && i >= Lw) i = p + t % (Lw - p);
    return h[i];
}
// The same with the variant fixed at compile time: the grouping of matches is bound by instructions, and the
// plain rule should not carry the other one's tests (they cost the batch kernels a third of their time).
template <bool PT>
__device__ __forceinline__ int cont_tok_t(const int32_t* __restrict__ h, int Lw, int p, int t) {
    if constexpr (PT) return cont_tok(h, Lw, p, t);
    else return h[p + t];
}

// Group the match whose continuation starts at p (query index qi) in an open-addressing table:
// rep[slot] = (qi << 28 | start of the group's first-seen continuation), cnt, last; a collision is
// resolved by comparing the actual tokens, so grouping is exact.  n_groups / overflow are the table's
// counters; once overflow is set the pass is void and nothing more is inserted.
template <bool PT = false>
__device__ __forceinline__ void insert_match(const int32_t* __restrict__ h, int p, int qi, int key_len, uint32_t hsh,
                                             int slots, int max_groups, int* rep, int* cnt, int* last,
                                             int* grp_slot, int* n_groups, int* overflow, int Lw = 0) {
    if (*((volatile int*)overflow)) return;  // this pass is void already: do not fill the table further
    uint32_t slot = hsh & (uint32_t)(slots - 1);
    const int me = (qi << 28) | p;
    for (int probe = 0; probe < slots; ++probe) {
        int cur = *((volatile int*)&rep[slot]);
        if (cur == -1) {
            int old = atomicCAS(&rep[slot], -1, me);
            if (old == -1) {
                int g = atomicAdd(n_groups, 1);
                if (g >= max_groups) {
                    *overflow = 1;
                    return;
                }
                grp_slot[g] = (int)slot;
                atomicAdd(&cnt[slot], 1);
                atomicMax(&last[slot], p);
                return;
            }
            cur = old;
        }
        if ((cur >> 28) == qi) {
            const int rp = cur & 0x0FFFFFFF;
            bool same = true;
            for (int t = 0; t < key_len; ++t)
                if (cont_tok_t<PT>(h, Lw, rp, t) != cont_tok_t<PT>(h, Lw, p, t)) {
                    same = false;
                    break;
                }
            if (same) {
                atomicAdd(&cnt[slot], 1);
                atomicMax(&last[slot], p);
                return;
            }
        }
        slot = (slot + 1) & (uint32_t)(slots - 1);
    }
    *overflow = 1;
}

// ------------------------------------------------------------------------------------------ building blocks
// The batch kernels (draft_team.cu, draft_stream.cu) are assembled from the pieces below.  Each piece is
// run by a group of `nthr` threads (whole warps; `tid` = index inside the group); `sync` is the group's
// barrier.  Pointers named rep / cnt / last / grp_slot are one hash table (see insert_match).

struct DraftTable {
    int* rep;
    int* cnt;
    int* last;
    int* grp_slot;
    int* n_groups;
    int* overflow;
};

// Extended model bigram of the last token x: rank r on lane r of one warp (chain[r * w + j], chain_ok[r]).
__device__ __forceinline__ void model_chain(const DraftParams& P, int x, int lane, int* chain, int* chain_ok) {
    const int w = P.w;
    if (x < 0 || x >= P.V) {
        if (lane == 0) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
    } else if (lane < P.k_tab) {
        bool ok = true;
        if (P.ext != nullptr && w <= P.w_ext) {
            const int32_t* e = P.ext + ((size_t)x * P.k_tab + lane) * P.w_ext;
            for (int j = 0; j < w; ++j) {
                const int t = e[j];
                ok = ok && (t >= 0 && t < P.V);
                chain[lane * w + j] = t;
            }
        } else {
            int t = P.tab[(size_t)x * P.k_tab + lane];
            for (int j = 0; j < w; ++j) {
                if (t < 0 || t >= P.V) {
                    ok = false;
                    break;
                }
                chain[lane * w + j] = t;
                t = P.tab[(size_t)t * P.k_tab];
            }
        }
        chain_ok[lane] = ok ? 1 : 0;
        if (!ok) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
    }
}

// One pass of the scan over history h (length L; h may point to global or to shared memory): every
// position whose preceding tokens equal the last q tokens (tq[0] = last token, tq[1] the one before, ...)
// is grouped by its continuation in table T, for every query length at once.  With R > 1 only the groups
// whose hash falls in residue class r are kept.  The scan itself only detects - per 128-bit vector one
// comparison chain, per warp iteration one vote; positions go into the warp's queue wq (kMatchQueue
// ints) and a queue-full is grouped at once, one match per lane, so that the dependent reads a match
// needs overlap.  No barrier inside: the caller synchronises before (table cleared) and after.
// Returns how many vectors of the history the calling warp had gone past when it stopped (all of them unless
// the table overflowed): the caller sizes the next round of passes from it.
template <int U = 4, bool PT = false>  // U: 128-bit loads a thread keeps in flight; PT: SPEC_FLAG_PARTIAL_TAIL (the caller passes what P.flags says)
__device__ __forceinline__ int scan_pass(const DraftParams& P, const int32_t* __restrict__ h, int L, int R, int r,
                                          int t0, int t1, int t2, int t3, const DraftTable& T, int* wq, int tid, int nthr) {
    const int w = P.w, lane = tid & 31;
    const int n_scan = L - w;  // token index x = p - 1 runs over [0, n_scan)
    const int key_len = (P.flags & SPEC_FLAG_KEY_NEXT_TOKEN) ? 1 : w;
    const bool need2 = P.q_min >= 2;  // every query has at least two tokens: test the second one in registers
    constexpr bool partial = PT;  // occurrences with fewer than w following tokens count too
    const int Lw = partial ? L : 0;
    const int4* h4 = reinterpret_cast<const int4*>(h);
    const int n_vec = (max(n_scan, 0) + 3) >> 2;
    // bits of one vector; `before` is the token left of the vector's first one
    auto vec_hits = [&](const int4& v, int before, int xb) -> unsigned {
        bool px = true, py = true, pz = true, pw = true;
        if (need2) {
            px = before == t1;
            py = v.x == t1;
            pz = v.y == t1;
            pw = v.z == t1;
        }
        return (unsigned)(v.x == t0 && px && xb + 0 < n_scan) | (unsigned)(v.y == t0 && py && xb + 1 < n_scan) << 1 |
               (unsigned)(v.z == t0 && pz && xb + 2 < n_scan) << 2 | (unsigned)(v.w == t0 && pw && xb + 3 < n_scan) << 3;
    };
    // group the match at token index x (the continuation starts at x + 1)
    auto handle_match = [&](int x) {
        // length of the common suffix of hist[0..x] and the whole history, up to q_max
        int m = 1;
        if (P.q_max > 1 && x >= 1 && h[x - 1] == t1) {
            m = 2;
            if (P.q_max > 2 && x >= 2 && h[x - 2] == t2) {
                m = 3;
                if (P.q_max > 3 && x >= 3 && h[x - 3] == t3) m = 4;
            }
        }
        const int p = x + 1;
        uint32_t hc = 0x9E3779B9u;  // one multiply-add per token, mixed once per query length below
        for (int t = 0; t < key_len; ++t) hc = hc * 0x85EBCA6Bu + (uint32_t)cont_tok_t<PT>(h, Lw, p, t);
        for (int qi = 0; qi < P.n_q; ++qi) {
            const int q = P.qs[qi];
            if (m < q || (!partial && L < q + w)) continue;
            const uint32_t hq = fmix32(hc + (uint32_t)qi * 0x632BE5ABu);
            if (R > 1 && (int)(fmix32(hq ^ 0xA511E9B3u) % (uint32_t)R) != r) continue;
            insert_match<PT>(h, p, qi, key_len, hq, P.slots, P.max_groups, T.rep, T.cnt, T.last, T.grp_slot, T.n_groups, T.overflow, Lw);
        }
    };
    int qn = 0;  // queued matches (the same in every lane)
    auto flush_matches = [&]() {
        __syncwarp();
        for (int i = lane; i < qn; i += 32) handle_match(wq[i]);
        __syncwarp();
        qn = 0;
    };
    // v0 = the lane's first vector of the block, its u-th vector is v0 + 32 u
    auto handle_hits = [&](unsigned hits, int v0) {
        const int nh = __popc(hits);
        int incl = nh;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (total == 0) return;  // (the block was flagged by the filter only)
        if (total > kMatchQueue) {  // denser than the queue: group them in place
            while (hits) {
                const int bit = __ffs(hits) - 1;
                hits &= hits - 1;
                handle_match(((v0 + (bit >> 2) * 32) << 2) + (bit & 3));
            }
            return;
        }
        if (qn + total > kMatchQueue) flush_matches();
        int at = qn + incl - nh;
        while (hits) {
            const int bit = __ffs(hits) - 1;
            hits &= hits - 1;
            wq[at++] = ((v0 + (bit >> 2) * 32) << 2) + (bit & 3);
        }
        qn += total;
        // a warp's worth of matches is grouped now, while the other warps keep streaming, rather than at
        // the end of the scan, where nothing would overlap it
        if (qn >= 32) flush_matches();
    };
    // The scan is bound by integer instructions as much as by memory, so the common case - no match in the
    // block - costs as few of them as possible.  A warp takes a contiguous block of U * 32 vectors (U
    // 128-bit loads per thread in flight): the token left of a vector then comes from the neighbouring lane,
    // and for lane 0 from lane 31's previous vector (one rotating shuffle per vector), with a single extra
    // load per block.  Positions are first tested with a filter of one multiply-add and one comparison per
    // token - left * K + token equals t1 * K + t0 wherever the pair matches (and, rarely, elsewhere) - and
    // one vote per block; only a flagged block works out exact positions.  Full blocks carry no bounds tests.
    const int wv = tid >> 5, nwarps = nthr >> 5;
    constexpr uint32_t K = 0x9E3779B1u;
    const uint32_t target = need2 ? (uint32_t)t1 * K + (uint32_t)t0 : (uint32_t)t0;
    const int rot_src = (lane + 31) & 31;
    int reached = n_vec;
    auto scan_blocks = [&](auto two_tokens) {
        constexpr bool N2 = decltype(two_tokens)::value;
        for (int base = wv * (U * 32); base < n_vec; base += nwarps * (U * 32)) {  // warp-uniform
            // too many groups for one pass: the caller rescans with more passes
            if (__any_sync(0xffffffffu, *((volatile int*)T.overflow))) {
                reached = base;
                break;
            }
            const int v0 = base + lane;
            int4 vv[U];
            int left[U];
            int carry = -5;  // lane 0: the token before its next vector
            if (base + U * 32 <= n_vec) {
#pragma unroll
                for (int u = 0; u < U; ++u) vv[u] = h4[v0 + u * 32];
            } else {
#pragma unroll
                for (int u = 0; u < U; ++u) vv[u] = (v0 + u * 32 < n_vec) ? h4[v0 + u * 32] : make_int4(-3, -3, -3, -3);
            }
            if (N2 && lane == 0 && base > 0) carry = h[(base << 2) - 1];
            bool some = false;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int4 v = vv[u];
                if (N2) {
                    const int rot = __shfl_sync(0xffffffffu, v.w, rot_src);  // lane l gets lane l-1's, lane 0 gets lane 31's
                    left[u] = lane ? rot : carry;
                    carry = rot;
                    some = some || ((uint32_t)left[u] * K + (uint32_t)v.x == target) || ((uint32_t)v.x * K + (uint32_t)v.y == target) ||
                           ((uint32_t)v.y * K + (uint32_t)v.z == target) || ((uint32_t)v.z * K + (uint32_t)v.w == target);
                } else {
                    left[u] = -5;
                    some = some || ((uint32_t)v.x == target) || ((uint32_t)v.y == target) || ((uint32_t)v.z == target) || ((uint32_t)v.w == target);
                }
            }
            if (!__any_sync(0xffffffffu, some)) continue;
            unsigned hits = 0;  // bit 4u + c: component c of the lane's u-th vector
#pragma unroll
            for (int u = 0; u < U; ++u) hits |= vec_hits(vv[u], left[u], (v0 + u * 32) << 2) << (4 * u);
            handle_hits(hits, v0);
        }
    };
    if (need2) scan_blocks(std::true_type{});
    else scan_blocks(std::false_type{});
    flush_matches();
    if (partial && tid < 32) {  // the last w - 1 positions, by the group's first warp: continuations that run past the end
        for (int x = max(n_scan, 0) + lane; x <= L - 2; x += 32)
            if (h[x] == t0) handle_match(x);
    }
    return reached;
}

// Passes for the next round after a pass of a round of R overflowed when about `reached` of `n_vec` vectors had
// been scanned: the groups seen so far filled the table, so the whole history needs about n_vec / reached
// tables' worth per residue class - with a margin, at least twice as many as before, as a power of two.
__device__ __forceinline__ int next_pass_count(int R, int reached, int n_vec) {
    const long long est = (long long)R * n_vec * 5 / (4ll * (reached > 0 ? reached : 1)) + 1;
    int next = 2 * R;
    while (next < est && next <= kMaxPasses) next *= 2;
    return next;
}

// Scratch of the ranking and mixing steps (one per group of threads; see the layouts of the kernels).
struct DraftScratch {
    unsigned long long* gkey;     // [max_groups + n_q * topk]: (query index << 60 | count << 32 | start)
    int* rank_acc;                // [max_groups + n_q * topk]
    unsigned long long* run_key;  // [n_q][topk]: the winners so far, ranked
    int* n_run;                   // [kMaxNQ] winners per query length
    int* n_cnt;                   // [kMaxNQ]
    int32_t* cand;                // [n_cand][w] candidate rows
    int* cand_src;                // [n_cand_max] each, then cand_cnt, cand_keep, dropped
    int* cand_cnt;
    int* cand_keep;
    int* dropped;
    int* row_of;                  // [B]
    int* chain;                   // [k_tab][w]
    int* chain_ok;                // [k_tab]
    int* cand_off;                // [kMaxNQ + 2]
    int* n_out;
    int* n_surv;                  // keys at or above the thresholds
    unsigned long long* tau;      // [kMaxNQ] threshold per query length
};

// Rank a finished pass's groups together with the winners of earlier passes: rank r < topk (by count, then by
// the later start, within one query length) lands in slot r of run_key.  Keys are distinct (a group's latest
// start belongs to no other group of that query length).  Ends with a barrier.
//
// A key's rank is the number of larger keys of its query length, found by walking over the other keys - but a
// key that ranks high has to walk over all of them, a serial chain that sets the length of the whole step.  So
// with many keys a threshold per query length comes first: 32 keys sampled at regular intervals are ranked
// among themselves inside a warp, and the sample with topk - 1 larger samples is a lower bound of the
// topk-th largest key, so only the keys at or above it (about topk / 32 of them) can be emitted; their rank
// among themselves is their rank among all.  The table's memory holds the survivors (the table itself is no
// longer needed once the keys are built).
constexpr int kRankDirect = 96;  // up to this many keys are ranked directly
// Ranks the n_keys keys in X.gkey (rank_acc zeroed, n_cnt zeroed, *n_surv = 0, all before a barrier); `skey` is
// room for n_keys more keys.  Writes run_key / n_run.  Ends with a barrier.
template <class Sync>
__device__ __forceinline__ void rank_keys(const DraftParams& P, int n_keys, unsigned long long* skey, const DraftScratch& X, int tid,
                                          int nthr, Sync&& sync) {
    const int topk = P.topk, lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const unsigned long long* keys = X.gkey;
    int m = n_keys;
    if (n_keys > kRankDirect) {
        for (int qi = warp; qi < P.n_q; qi += nwarps) {  // warp-uniform
            // lane l samples the first key of this query length among (up to 8 of) its own 1/32 of the keys
            const int lo = (int)((long long)lane * n_keys / 32), hi = (int)((long long)(lane + 1) * n_keys / 32);
            unsigned long long mine = 0;
            for (int o = lo; o < hi && o < lo + 8; ++o) {
                const unsigned long long k = X.gkey[o];
                if ((int)(k >> 60) == qi) {
                    mine = k;
                    break;
                }
            }
            int larger = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const unsigned long long other = __shfl_sync(0xffffffffu, mine, j);
                larger += other > mine ? 1 : 0;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, mine != 0ull && larger == topk - 1);
            unsigned long long tau = 0ull;  // fewer than topk samples: no threshold for this query length
            if (hit) tau = __shfl_sync(0xffffffffu, mine, __ffs(hit) - 1);
            if (lane == 0) X.tau[qi] = tau;
        }
        sync();
        for (int g = tid; g < n_keys; g += nthr) {
            const unsigned long long k = X.gkey[g];
            if (k >= X.tau[(int)(k >> 60)]) {
                const int idx = atomicAdd(X.n_surv, 1);
                skey[idx] = k;
                X.rank_acc[idx] = 0;
            }
        }
        sync();
        keys = skey;
        m = *X.n_surv;
    }
    // A key with topk larger keys cannot be emitted, so a thread stops counting there.  Groups are created
    // in scan order, so the later ones tend to hold the later starts, i.e. the larger keys: the walk runs
    // backwards from the newest group, eight keys at a time (independent loads).  With fewer keys than
    // threads the comparisons of one key are dealt out to `parts` threads, interleaved.
    int parts = 1;
    while (parts < 32 && m * parts * 2 <= nthr) parts <<= 1;
    for (int item = tid; item < m * parts; item += nthr) {
        const int g = item / parts, part = item - g * parts;
        const unsigned long long mine = keys[g];
        int rank = 0;
        for (int o = m - 1 - part; o >= 0 && rank < topk; o -= 8 * parts) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int idx = o - k * parts;
                if (idx >= 0) {
                    const unsigned long long other = keys[idx];
                    rank += ((other >> 60) == (mine >> 60) && other > mine) ? 1 : 0;
                }
            }
        }
        if (rank) atomicAdd(&X.rank_acc[g], rank);
    }
    sync();
    for (int g = tid; g < m; g += nthr) {
        const unsigned long long mine = keys[g];
        const int rank = X.rank_acc[g];
        if (rank < topk) {  // ranks are distinct, so the rows kept are 0 .. max rank
            X.run_key[(int)(mine >> 60) * topk + rank] = mine & 0x0FFFFFFFFFFFFFFFull;
            atomicMax(&X.n_cnt[(int)(mine >> 60)], rank + 1);
        }
    }
    sync();
    if (tid < kMaxNQ) X.n_run[tid] = X.n_cnt[tid];
    sync();
}

// A finished pass: the keys of table T's groups and of the winners so far, then rank_keys.  The table's
// memory holds the survivors (the table itself is no longer needed once the keys are built).
template <class Sync>
__device__ __forceinline__ void rank_pass(const DraftParams& P, const DraftTable& T, const DraftScratch& X, int tid, int nthr,
                                          Sync&& sync) {
    const int topk = P.topk;
    const int n_groups = *T.n_groups;
    int n_old = 0;
    for (int qi = 0; qi < P.n_q; ++qi) n_old += X.n_run[qi];
    const int n_keys = n_groups + n_old;
    for (int g = tid; g < n_groups; g += nthr) {
        const int slot = T.grp_slot[g];
        const unsigned long long qi = (unsigned long long)(T.rep[slot] >> 28);
        X.gkey[g] = (qi << 60) | ((unsigned long long)(uint32_t)T.cnt[slot] << 32) | (uint32_t)T.last[slot];
        X.rank_acc[g] = 0;
    }
    for (int j = tid; j < n_old; j += nthr) {
        int qi = 0, o = j;
        while (o >= X.n_run[qi]) o -= X.n_run[qi++];
        X.gkey[n_groups + j] = ((unsigned long long)qi << 60) | X.run_key[qi * topk + o];
        X.rank_acc[n_groups + j] = 0;
    }
    if (tid < kMaxNQ) X.n_cnt[tid] = 0;
    if (tid == 0) *X.n_surv = 0;
    sync();
    rank_keys(P, n_keys, reinterpret_cast<unsigned long long*>(T.rep), X, tid, nthr, sync);
}

// Mixed allocation of sequence s: context rows in query order, then model rows by rank; duplicates dropped;
// the first B survivors become the drafts.  Writes the four outputs.  Starts and ends with a barrier.
template <class Sync>
__device__ __forceinline__ void mix_and_emit(const DraftParams& P, int s, const int32_t* __restrict__ h, int L, bool gave_up,
                                             const DraftScratch& X, int tid, int nthr, Sync&& sync) {
    const int w = P.w, topk = P.topk, lane = tid & 31, warp = tid >> 5;
    const int Lw = (P.flags & SPEC_FLAG_PARTIAL_TAIL) ? L : 0;
    const bool dedup = (P.flags & SPEC_FLAG_DEDUP) != 0;
    sync();
    if (tid == 0) {
        if (gave_up) {  // too many distinct continuations even for 1024 passes: no context rows, and say so
            for (int li = 0; li < kMaxNQ; ++li) X.n_run[li] = 0;
            atomicOr(P.status, SPEC_STATUS_GROUPS);
        }
        int off = 0;
        for (int li = 0; li < P.n_q; ++li) {
            X.cand_off[li] = off;
            off += X.n_run[li];
        }
        X.cand_off[P.n_q] = off;
        off += (P.flags & SPEC_FLAG_MODEL_FILL) ? P.k_tab : 0;
        X.cand_off[P.n_q + 1] = off;
    }
    sync();
    int32_t* cand = X.cand;
    const int n_cand = X.cand_off[P.n_q + 1];
    for (int i = tid; i < n_cand * w; i += nthr) {
        const int ci = i / w, t = i - ci * w;
        int li = 0;
        while (ci >= X.cand_off[li + 1]) ++li;
        const int r = ci - X.cand_off[li];
        int tok, keep = 1, src = 0, count = 0;
        if (li == P.n_q) {
            keep = X.chain_ok[r];
            tok = keep ? X.chain[r * w + t] : -1;
        } else {
            const unsigned long long key = X.run_key[li * topk + r];
            const int start = (int)(uint32_t)key;
            tok = cont_tok(h, Lw, start, t);
            src = P.qs[li];
            count = (int)(key >> 32);
            if (t == 0) {  // a context row that carries a token outside the vocabulary is dropped
                bool in_range = true;
                for (int u = 0; u < w; ++u) {
                    const int tk = cont_tok(h, Lw, start, u);
                    in_range = in_range && tk >= 0 && tk < P.V;
                }
                keep = in_range ? 1 : 0;
                if (!in_range) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
            }
        }
        cand[i] = tok;
        if (t == 0) {
            X.cand_src[ci] = src;
            X.cand_cnt[ci] = count;
            X.cand_keep[ci] = keep;
            X.dropped[ci] = 0;
        }
    }
    sync();
    // Rows reserved for the model strategy: the context strategies together take at most B - reserve.
    const int reserve = min(P.B, (P.flags >> 8) & 0xFF);
    const int n_ctx = X.cand_off[P.n_q];
    // all (earlier, later) pairs in [pair_lo, pair_hi) side by side: a later row equal to an earlier live row is dropped
    auto mark_duplicates = [&](int pair_lo, int pair_hi) {
        for (int pi = pair_lo + tid; pi < pair_hi; pi += nthr) {
            // pair index -> (ci, j) with j < ci: ci is the largest integer with ci (ci - 1) / 2 <= pi
            int ci = (int)((1.0f + sqrtf(1.0f + 8.0f * (float)pi)) * 0.5f);
            while (ci * (ci - 1) / 2 > pi) --ci;
            while ((ci + 1) * ci / 2 <= pi) ++ci;
            const int j = pi - ci * (ci - 1) / 2;
            if (!X.cand_keep[ci] || !X.cand_keep[j]) continue;
            bool same = true;
            for (int t = 0; t < w && same; ++t) same = cand[j * w + t] == cand[ci * w + t];
            if (same) X.dropped[ci] = 1;
        }
        sync();
    };
    // warp 0: live candidates in [c_lo, c_hi) get draft rows first_row, first_row + 1, ... below row_limit;
    // the others are switched off.  Returns the next free row.
    auto assign_rows = [&](int c_lo, int c_hi, int first_row, int row_limit) {
        int nxt = first_row;
        for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
            const int ci = c0 + lane;
            const bool k = ci < c_hi && X.cand_keep[ci] != 0 && X.dropped[ci] == 0;
            const unsigned mask = __ballot_sync(0xffffffffu, k);
            const int pos = nxt + __popc(mask & ((1u << lane) - 1u));
            if (k && pos < row_limit) X.row_of[pos] = ci;
            else if (ci < c_hi) X.cand_keep[ci] = 0;
            nxt += __popc(mask);
        }
        return min(nxt, row_limit);
    };
    const int all_pairs = n_cand * (n_cand - 1) / 2;
    if (reserve == 0) {
        // a row is a duplicate if any earlier candidate equals it: the rows beyond B are never
        // followed by a row that is taken, so comparing with every earlier candidate is exact
        if (dedup) mark_duplicates(0, all_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(0, n_cand, 0, P.B);
            if (lane == 0) *X.n_out = n_rows;
        }
    } else {
        // context rows first, cut at B - reserve; model rows are then compared with the rows taken only
        const int ctx_pairs = n_ctx * (n_ctx - 1) / 2;
        if (dedup) mark_duplicates(0, ctx_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(0, n_ctx, 0, P.B - reserve);
            if (lane == 0) *X.n_out = n_rows;
        }
        sync();
        if (dedup) mark_duplicates(ctx_pairs, all_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(n_ctx, n_cand, *X.n_out, P.B);
            __syncwarp();
            if (lane == 0) *X.n_out = n_rows;
        }
    }
    sync();
    const int n = *X.n_out;
    for (int i = tid; i < P.B * w; i += nthr) {
        const int b = i / w, t = i - b * w;
        P.drafts[(size_t)s * P.B * w + i] = (b < n) ? cand[X.row_of[b] * w + t] : -1;
    }
    for (int b = tid; b < P.B; b += nthr) {
        if (P.src) P.src[(size_t)s * P.B + b] = (b < n) ? X.cand_src[X.row_of[b]] : -1;
        if (P.counts) P.counts[(size_t)s * P.B + b] = (b < n) ? X.cand_cnt[X.row_of[b]] : 0;
    }
    if (tid == 0) P.ndrafts[s] = n;
    sync();
}

// draft.cu
DraftParams make_draft_params(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs, int n_q,
                              int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts, int32_t* d_src,
                              int32_t* d_counts);
// ctx_index.cu
int launch_draft_indexed(spec_ctx* ctx, DraftParams& P, cudaStream_t st);

// draft_team.cu / draft_stream.cu
constexpr int kDraftNoFit = 1;  // launch_draft_team: the staged layout does not fit (nothing was launched)
int launch_draft_team(spec_ctx* ctx, DraftParams& P, cudaStream_t st);
int launch_draft_stream(spec_ctx* ctx, DraftParams& P, cudaStream_t st);

}  // namespace ngs
