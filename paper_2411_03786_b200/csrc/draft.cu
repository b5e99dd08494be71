// Context N-gram drafting and mixed allocation, latency path: one CTA per sequence, or for long
// histories one thread-block cluster per sequence whose CTAs each scan a slice of the history and group
// their matches in the leader CTA's hash table through distributed shared memory.  (Batches of many
// sequences take the team kernel in draft_team.cu.)
//
// One streaming pass over the history serves every query length at once.  A position p is the
// start of a continuation for query length q when the q tokens before p equal the last q tokens
// of the history; the q values are nested (a q=3 match is also a q=2 and q=1 match), so the scan
// computes the length of the common suffix once per position.  Each match is grouped by its
// w-token continuation in a shared-memory hash table that resolves collisions by comparing the
// actual tokens, so grouping is exact.  If a sequence has more distinct continuations than the
// table holds, the scan is repeated in R passes, pass r keeping only the groups whose hash falls
// in residue class r, and the per-pass winners are merged: still exact, only slower.
//
// A history of up to 8192 tokens is first copied into shared memory (one round of 128-bit loads);
// the scan, the key comparisons and the candidate rows then never wait for global memory again,
// which is what the latency of a single short sequence is made of.
#include <cooperative_groups.h>

#include "draft_common.cuh"

namespace cg = cooperative_groups;

namespace ngs {

constexpr int kRankMax = 512;                          // groups ranked by counting (all threads) up to here

struct DraftSmem {
    unsigned long long run_key[kMaxNQ][kMaxB];  // per query length: ranked (count << 32 | start) keys
    unsigned long long gkey[kRankMax];          // (query index << 60 | count << 32 | start) per group
    int32_t cand_src[kMaxCand];
    int32_t cand_cnt[kMaxCand];
    int32_t cand_keep[kMaxCand];
    int32_t row_of[kMaxB];                      // candidate that became draft row b
    int32_t row_of_tmp[kMaxCand];               // duplicate flags
    int cand_off[kMaxNQ + 2];
    int n_cnt[kMaxNQ];
    int rank_acc[kRankMax];   // groups of the same query length with a larger key
    int32_t chain[kMaxKTab][kMaxW];
    int chain_ok[kMaxKTab];
    int n_run[kMaxNQ];
    int tq[kMaxQ];
    int n_groups;
    int overflow;
    int n_out;
};

// The kernel carries nothing it does not execute: a decode step's drafting latency is sensitive to its
// code size (a quarter of it is cold instruction fetch).
__global__ void __launch_bounds__(1024, 1) draft_kernel(const DraftParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DraftSmem* sm = reinterpret_cast<DraftSmem*>(smem_raw);
    int* rep = reinterpret_cast<int*>(smem_raw + ((sizeof(DraftSmem) + 15) & ~size_t(15)));
    int* cnt = rep + P.slots;
    int* last = cnt + P.slots;
    int* grp_slot = last + P.slots;

    // The cluster's CTAs share one sequence; rank 0 (the leader) owns the table and writes the result.
    // Every cluster-wide barrier below is reached by all CTAs: the loop bounds depend only on the
    // sequence length, the launch parameters and a flag every CTA reads between two barriers.
    cg::cluster_group cluster = cg::this_cluster();
    const int csize = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
    const bool leader = crank == 0;
    DraftSmem* lsm = cluster.map_shared_rank(sm, 0);
    int* lrep = cluster.map_shared_rank(rep, 0);
    int* lcnt = cluster.map_shared_rank(cnt, 0);
    int* llast = cluster.map_shared_rank(last, 0);
    int* lgrp_slot = cluster.map_shared_rank(grp_slot, 0);

    // barrier over all CTAs of the sequence (a plain CTA barrier when there is only one: much cheaper)
    auto pass_sync = [&]() {
        if (csize == 1) __syncthreads();
        else cluster.sync();
    };

    const int tid = threadIdx.x, nthr = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int s = (int)blockIdx.x / csize;
    const int32_t* __restrict__ h = P.hist + (size_t)s * P.cap;
    const int w = P.w;
    int32_t* hist_s = rep + P.hist_off;

    grid_launch_dependents();  // the verify kernel may start streaming weights while this one runs
    // the first pass's empty table does not depend on the inputs: prepare it while the previous kernel drains
    if (leader) {
        for (int i = tid; i < P.slots; i += nthr) {
            rep[i] = -1;
            cnt[i] = 0;
            last[i] = -1;
        }
        if (tid == 0) {
            sm->n_groups = 0;
            sm->overflow = 0;
        }
    }
    grid_dependency_wait();    // history and lengths come from the previous step's commit
    int L = P.len[s];
    if (L < 0 || L > P.cap) {
        if (tid == 0 && leader) atomicOr(P.status, SPEC_STATUS_CAPACITY);
        L = 0;
    }
    if (P.stage_hist) {
        const int4* g4 = reinterpret_cast<const int4*>(h);
        int4* s4 = reinterpret_cast<int4*>(hist_s);
        const int n4 = (L + 3) >> 2;  // cap % 4 == 0 and L <= cap: the last vector stays inside the row
#pragma unroll 4
        for (int i = tid; i < n4; i += nthr) s4[i] = g4[i];
        __syncthreads();
        h = hist_s;
    }
    if (tid < kMaxQ) sm->tq[tid] = (tid < L) ? h[L - 1 - tid] : -2;
    if (tid < kMaxNQ) sm->n_run[tid] = 0;
    if (tid < kMaxKTab) sm->chain_ok[tid] = 0;
    __syncthreads();

    // ---- extended model bigram of the last token (rank r on lane r), overlapped with the scan
    if (leader && warp == nwarps - 1 && (P.flags & SPEC_FLAG_MODEL_FILL) && L >= 1) {
        const int x = sm->tq[0];
        if (x < 0 || x >= P.V) {
            if (lane == 0) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
        } else if (lane < P.k_tab) {
            bool ok = true;
            if (P.ext != nullptr && w <= P.w_ext) {
                const int32_t* e = P.ext + ((size_t)x * P.k_tab + lane) * P.w_ext;
                int t[kMaxW];  // all loads first, so they are in flight together
#pragma unroll
                for (int j = 0; j < kMaxW; ++j) t[j] = (j < w) ? e[j] : 0;
#pragma unroll
                for (int j = 0; j < kMaxW; ++j)
                    if (j < w) {
                        ok = ok && (t[j] >= 0 && t[j] < P.V);
                        sm->chain[lane][j] = t[j];
                    }
            } else {
                int t = P.tab[(size_t)x * P.k_tab + lane];
                for (int j = 0; j < w; ++j) {
                    if (t < 0 || t >= P.V) {
                        ok = false;
                        break;
                    }
                    sm->chain[lane][j] = t;
                    t = P.tab[(size_t)t * P.k_tab];
                }
            }
            sm->chain_ok[lane] = ok ? 1 : 0;
            if (!ok) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
        }
    }

    // ---- context N-grams
    const int n_scan = L - w;  // token index x = p - 1 runs over [0, n_scan)
    // continuation tokens that identify a group: all w (the paper's rule) or the next token only
    const int key_len = (P.flags & SPEC_FLAG_KEY_NEXT_TOKEN) ? 1 : w;
    const int t0 = sm->tq[0], t1 = sm->tq[1], t2 = sm->tq[2], t3 = sm->tq[3];
    bool any_q = false;
    for (int qi = 0; qi < P.n_q; ++qi) any_q = any_q || (L >= P.qs[qi] + w);

    const int4* h4 = reinterpret_cast<const int4*>(h);
    const int n_vec_all = (max(n_scan, 0) + 3) >> 2;
    const int v_chunk = (n_vec_all + csize - 1) / csize;  // this CTA's slice of the history
    const int n_vec = min(n_vec_all, (crank + 1) * v_chunk);

    int R = 1;
    bool gave_up = false;
    while (any_q && n_scan >= 1) {
        __syncthreads();
        if (tid < kMaxNQ) sm->n_run[tid] = 0;
        bool overflowed = false;
        for (int r = 0; r < R && !overflowed; ++r) {
            if (leader && (R > 1 || r > 0)) {  // (the table of the very first pass was prepared at kernel entry)
                for (int i = tid; i < P.slots; i += nthr) {
                    rep[i] = -1;
                    cnt[i] = 0;
                    last[i] = -1;
                }
                if (tid == 0) {
                    sm->n_groups = 0;
                    sm->overflow = 0;
                }
            }
            pass_sync();  // the leader's table is ready
            // scan: positions holding the last token are collected in a bit mask and handled one by
            // one (they are rare).  `hits` has bit 4u+c for component c of the lane's u-th vector.
            const bool need2 = P.q_min >= 2;  // every query has at least two tokens: test the second one in registers
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
                uint32_t hc = 0x9E3779B9u;
                for (int t = 0; t < key_len; ++t) hc = fmix32(hc ^ (uint32_t)h[p + t]) + 0x7F4A7C15u;
                for (int qi = 0; qi < P.n_q; ++qi) {
                    const int q = P.qs[qi];
                    if (m < q || L < q + w) continue;
                    const uint32_t hq = fmix32(hc + (uint32_t)qi * 0x632BE5ABu);
                    if (R > 1 && (int)(fmix32(hq ^ 0xA511E9B3u) % (uint32_t)R) != r) continue;
                    insert_match(h, p, qi, key_len, hq, P.slots, P.max_groups, lrep, lcnt, llast, lgrp_slot, &lsm->n_groups, &lsm->overflow);
                }
            };
            // v0 = the lane's first vector, its u-th vector is v0 + u * ustride; a match is grouped where it is found
            auto handle_hits = [&](unsigned hits, int v0, int ustride) {
                while (hits) {
                    const int bit = __ffs(hits) - 1;
                    hits &= hits - 1;
                    handle_match(((v0 + (bit >> 2) * ustride) << 2) + (bit & 3));
                }
            };
            // 128-bit loads, four per thread in flight.  The common case (no match among the warp's
            // 512 tokens) is decided by one comparison chain per vector and one vote; only then are
            // the positions worked out.
            for (int vw = crank * v_chunk + (tid - lane); vw < n_vec; vw += 4 * nthr) {  // warp-uniform trip count
                // too many groups for one pass: rescan with more passes
                if (__any_sync(0xffffffffu, *((volatile int*)&lsm->overflow))) break;
                const int v0 = vw + lane;
                int4 vv[4];
                int left[4];  // token before the vector
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int vi = v0 + u * nthr;
                    vv[u] = (vi < n_vec) ? h4[vi] : make_int4(-3, -3, -3, -3);
                }
                if (need2) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int vi = v0 + u * nthr;
                        left[u] = __shfl_up_sync(0xffffffffu, vv[u].w, 1);
                        if (lane == 0) left[u] = (vi > 0 && vi < n_vec) ? h[(vi << 2) - 1] : -5;
                    }
                }
                unsigned hits = 0;
#pragma unroll
                for (int u = 0; u < 4; ++u) hits |= vec_hits(vv[u], left[u], (v0 + u * nthr) << 2) << (4 * u);
                handle_hits(hits, v0, nthr);
            }
            pass_sync();  // every CTA's matches are in the table
            const int ov = *((volatile int*)&lsm->overflow);
            pass_sync();  // every CTA has read the flag before the leader may reset it
            if (ov) {
                overflowed = true;
                break;
            }
            if (!leader) continue;
            if (R == 1 && sm->n_groups <= kRankMax) {
                // Few groups (the usual case).
                // Every group is ranked by counting the groups of the same query length with a larger
                // (count, start) key; the comparisons of one group are split over `parts` threads so that
                // all threads stay busy.  Rank r < topk lands in slot r.
                const int n_groups = sm->n_groups;
                if (tid < kMaxNQ) sm->n_cnt[tid] = 0;
                for (int g = tid; g < n_groups; g += nthr) {
                    const int slot = grp_slot[g];
                    const unsigned long long qi = (unsigned long long)(rep[slot] >> 28);
                    sm->gkey[g] = (qi << 60) | ((unsigned long long)(uint32_t)cnt[slot] << 32) | (uint32_t)last[slot];
                    sm->rank_acc[g] = 0;
                }
                __syncthreads();
                int parts = 1;
                while (parts < 8 && n_groups * parts < 2 * nthr) parts <<= 1;
                const int span = (n_groups + parts - 1) / parts;
                for (int item = tid; item < n_groups * parts; item += nthr) {
                    const int g = item / parts, part = item - g * parts;
                    const unsigned long long mine = sm->gkey[g];
                    const int o_end = min(n_groups, (part + 1) * span);
                    int rank = 0;
                    // a group with topk larger keys cannot be emitted: most groups (single occurrences) stop early
                    for (int o = part * span; o < o_end && rank < P.topk; ++o) {
                        const unsigned long long other = sm->gkey[o];
                        rank += ((other >> 60) == (mine >> 60) && other > mine) ? 1 : 0;
                    }
                    if (rank) atomicAdd(&sm->rank_acc[g], rank);
                }
                __syncthreads();
                for (int g = tid; g < n_groups; g += nthr) {
                    const unsigned long long mine = sm->gkey[g];
                    const int rank = sm->rank_acc[g];
                    if (rank < P.topk) {  // ranks are distinct, so the rows kept are 0 .. max rank
                        sm->run_key[(int)(mine >> 60)][rank] = mine & 0x0FFFFFFFFFFFFFFFull;
                        atomicMax(&sm->n_cnt[(int)(mine >> 60)], rank + 1);
                    }
                }
                __syncthreads();
                if (tid < kMaxNQ) sm->n_run[tid] = sm->n_cnt[tid];
            } else if (warp < P.n_q) {
                // rank this pass's groups together with the winners of earlier passes: warp qi
                const int qi = warp;
                const int n_groups = sm->n_groups;
                const int n_old = sm->n_run[qi];
                unsigned long long keep0 = 0, keep1 = 0, prev = ~0ull;
                int n_new = 0;
                for (int rr = 0; rr < P.topk; ++rr) {
                    unsigned long long best = 0;
                    for (int g = lane; g < n_groups; g += 32) {
                        const int slot = grp_slot[g];
                        if ((rep[slot] >> 28) != qi) continue;
                        unsigned long long key = ((unsigned long long)(uint32_t)cnt[slot] << 32) | (uint32_t)last[slot];
                        if (key < prev && key > best) best = key;
                    }
                    for (int j = lane; j < n_old; j += 32) {
                        unsigned long long key = sm->run_key[qi][j];
                        if (key < prev && key > best) best = key;
                    }
                    best = warp_max_u64(best);
                    if (best == 0) break;
                    if ((rr & 31) == lane) {
                        if (rr < 32) keep0 = best; else keep1 = best;
                    }
                    prev = best;
                    ++n_new;
                }
                __syncwarp();
                if (lane < n_new) sm->run_key[qi][lane] = keep0;
                if (lane + 32 < n_new) sm->run_key[qi][lane + 32] = keep1;
                if (lane == 0) sm->n_run[qi] = n_new;
            }
            __syncthreads();
        }
        if (!overflowed) break;
        R *= 2;
        if (R > kMaxPasses) {
            gave_up = true;
            break;
        }
    }
    if (!leader) return;  // nobody reads a non-leader's shared memory, and no cluster barrier follows
    __syncthreads();

    // ---- mixed allocation: context rows in query order, then model rows by rank; drop duplicates.
    // Candidate rows are gathered side by side, a row is a duplicate if any earlier candidate equals
    // it (equality is transitive, so this is the same as comparing with the rows already taken),
    // and the first B survivors become the drafts.  (With rows reserved for the model the
    // comparison is staged: see below.)
    const bool dedup = (P.flags & SPEC_FLAG_DEDUP) != 0;
    if (tid == 0) {
        if (gave_up) {  // too many distinct continuations even for 1024 passes: no context rows, and say so
            for (int li = 0; li < kMaxNQ; ++li) sm->n_run[li] = 0;
            atomicOr(P.status, SPEC_STATUS_GROUPS);
        }
        int off = 0;
        for (int li = 0; li < P.n_q; ++li) {
            sm->cand_off[li] = off;
            off += sm->n_run[li];
        }
        sm->cand_off[P.n_q] = off;
        off += (P.flags & SPEC_FLAG_MODEL_FILL) ? P.k_tab : 0;
        sm->cand_off[P.n_q + 1] = off;
    }
    __syncthreads();
    int32_t* cand = rep;  // the hash table is no longer needed: [n_cand][w] token rows
    const int n_cand = sm->cand_off[P.n_q + 1];
    for (int i = tid; i < n_cand * w; i += nthr) {
        const int ci = i / w, t = i - ci * w;
        int li = 0;
        while (ci >= sm->cand_off[li + 1]) ++li;
        const int r = ci - sm->cand_off[li];
        int tok, keep = 1, src = 0, count = 0;
        if (li == P.n_q) {
            keep = sm->chain_ok[r];
            tok = keep ? sm->chain[r][t] : -1;
        } else {
            const unsigned long long key = sm->run_key[li][r];
            const int start = (int)(uint32_t)key;
            tok = h[start + t];
            src = P.qs[li];
            count = (int)(key >> 32);
            if (t == 0) {
                // a context row that carries a token outside the vocabulary (a corrupt history) is dropped, like
                // a model row whose chain left it: the caller indexes its embedding table with these tokens
                bool in_range = true;
                for (int u = 0; u < w; ++u) {
                    const int tk = h[start + u];
                    in_range = in_range && tk >= 0 && tk < P.V;
                }
                keep = in_range ? 1 : 0;
                if (!in_range) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
            }
        }
        cand[i] = tok;
        if (t == 0) {
            sm->cand_src[ci] = src;
            sm->cand_cnt[ci] = count;
            sm->cand_keep[ci] = keep;
            sm->row_of_tmp[ci] = 0;  // duplicate flag
        }
    }
    __syncthreads();

    // Rows reserved for the model strategy: the context strategies together take at most B - reserve.
    const int reserve = min(P.B, (P.flags >> 8) & 0xFF);
    const int n_ctx = sm->cand_off[P.n_q];
    int32_t* dropped = sm->row_of_tmp;
    // all (earlier, later) pairs in [pair_lo, pair_hi) side by side: a later row equal to an earlier live row is dropped
    auto mark_duplicates = [&](int pair_lo, int pair_hi) {
        for (int pi = pair_lo + tid; pi < pair_hi; pi += nthr) {
            // pair index -> (ci, j) with j < ci: ci is the largest integer with ci (ci - 1) / 2 <= pi
            int ci = (int)((1.0f + sqrtf(1.0f + 8.0f * (float)pi)) * 0.5f);
            while (ci * (ci - 1) / 2 > pi) --ci;
            while ((ci + 1) * ci / 2 <= pi) ++ci;
            const int j = pi - ci * (ci - 1) / 2;
            if (!sm->cand_keep[ci] || !sm->cand_keep[j]) continue;
            bool same = true;
            for (int t = 0; t < w && same; ++t) same = cand[j * w + t] == cand[ci * w + t];
            if (same) dropped[ci] = 1;
        }
        __syncthreads();
    };
    // warp 0: live candidates in [c_lo, c_hi) get draft rows first_row, first_row + 1, ... below row_limit;
    // the others are switched off.  Returns the next free row.
    auto assign_rows = [&](int c_lo, int c_hi, int first_row, int row_limit) {
        int base = first_row;
        for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
            const int ci = c0 + lane;
            const bool k = ci < c_hi && sm->cand_keep[ci] != 0 && dropped[ci] == 0;
            const unsigned mask = __ballot_sync(0xffffffffu, k);
            const int pos = base + __popc(mask & ((1u << lane) - 1u));
            if (k && pos < row_limit) sm->row_of[pos] = ci;
            else if (ci < c_hi) sm->cand_keep[ci] = 0;
            base += __popc(mask);
        }
        return min(base, row_limit);
    };
    const int all_pairs = n_cand * (n_cand - 1) / 2;
    if (reserve == 0) {
        // a row is a duplicate if any earlier candidate equals it: the rows beyond B are never
        // followed by a row that is taken, so comparing with every earlier candidate is exact
        if (dedup) mark_duplicates(0, all_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(0, n_cand, 0, P.B);
            if (lane == 0) sm->n_out = n_rows;
        }
    } else {
        // context rows first, cut at B - reserve; model rows are then compared with the rows taken only
        const int ctx_pairs = n_ctx * (n_ctx - 1) / 2;
        if (dedup) mark_duplicates(0, ctx_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(0, n_ctx, 0, P.B - reserve);
            if (lane == 0) sm->n_out = n_rows;
        }
        __syncthreads();
        if (dedup) mark_duplicates(ctx_pairs, all_pairs);
        if (warp == 0) {
            const int n_rows = assign_rows(n_ctx, n_cand, sm->n_out, P.B);
            __syncwarp();
            if (lane == 0) sm->n_out = n_rows;
        }
    }
    __syncthreads();
    const int n = sm->n_out;
    for (int i = tid; i < P.B * w; i += nthr) {
        const int b = i / w, t = i - b * w;
        P.drafts[(size_t)s * P.B * w + i] = (b < n) ? cand[sm->row_of[b] * w + t] : -1;
    }
    for (int b = tid; b < P.B; b += nthr) {
        if (P.src) P.src[(size_t)s * P.B + b] = (b < n) ? sm->cand_src[sm->row_of[b]] : -1;
        if (P.counts) P.counts[(size_t)s * P.B + b] = (b < n) ? sm->cand_cnt[sm->row_of[b]] : 0;
    }
    if (tid == 0) P.ndrafts[s] = n;
}

DraftParams make_draft_params(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs, int n_q,
                              int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts, int32_t* d_src,
                              int32_t* d_counts) {
    DraftParams P;
    P.hist = d_hist;
    P.len = d_len;
    P.S = S;
    P.cap = cap;
    P.n_q = n_q;
    P.q_max = 0;
    P.q_min = kMaxQ;
    for (int i = 0; i < kMaxNQ; ++i) {
        P.qs[i] = i < n_q ? qs[i] : 0;
        if (i < n_q && qs[i] > P.q_max) P.q_max = qs[i];
        if (i < n_q && qs[i] < P.q_min) P.q_min = qs[i];
    }
    P.topk = topk;
    P.B = B;
    P.w = w;
    P.flags = flags;
    P.tab = ctx->tab_idx;
    P.k_tab = ctx->k_tab;
    P.ext = ctx->ext;
    P.w_ext = ctx->w_ext;
    P.V = ctx->V;
    P.drafts = d_drafts;
    P.ndrafts = d_ndrafts;
    P.src = d_src;
    P.counts = d_counts;
    P.status = ctx->d_status;
    P.slots = 0;
    P.max_groups = 0;
    P.stage_hist = 0;
    P.hist_off = 0;
    return P;
}

int launch_draft(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs, int n_q,
                 int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts, int32_t* d_src,
                 int32_t* d_counts, cudaStream_t st) {
    DraftParams P = make_draft_params(ctx, d_hist, d_len, S, cap, qs, n_q, topk, B, w, flags, d_drafts, d_ndrafts, d_src, d_counts);
    int slots = 1024;  // at most slots / 2 distinct continuations are grouped in one pass
    while (slots < cap / 2 && slots < 8192) slots <<= 1;
    int threads = cap >= 16384 ? 1024 : (cap >= 2048 ? 256 : 128);
#ifdef NGRAM_SPEC_TUNING
    // Tuning builds only: NGRAM_SPEC_DRAFT_SHAPE="threads,slots" overrides the choice (values are clamped).
    if (const char* ov = getenv("NGRAM_SPEC_DRAFT_SHAPE")) {
        int t = 0, sl = 0;
        if (sscanf(ov, "%d,%d", &t, &sl) == 2) {
            if (t >= 128 && t <= 1024 && t % 32 == 0) threads = t;
            if (sl >= 1024 && sl <= 8192 && (sl & (sl - 1)) == 0) slots = sl;
        }
    }
#endif
    // CTAs per sequence: one per 16K tokens of capacity, at most 8, and only while the batch alone
    // cannot fill the GPU (with many sequences the team kernel streams them)
    unsigned csize = 1;
    while (csize < 8 && (int)(csize * 2) * 16384 <= cap && (long long)S * (csize * 2) <= ctx->num_sms) csize <<= 1;
    // (continuations that run past the end of the history are the batch kernels' business: this kernel carries
    // only the paper's rule)
    const bool partial = (flags & SPEC_FLAG_PARTIAL_TAIL) != 0;
    if (partial) csize = 1;
    const bool stage = csize == 1 && cap <= 8192 && !partial;
    if (csize == 1) {
        // Batches: histories of up to 16384 tokens are staged in shared memory by warp teams (when the batch
        // fills the GPU more than twice over, or a history is too long for the staging of this kernel);
        // longer ones are streamed by the scanner / finisher kernel.
        const bool batch = S > 2 * ctx->num_sms || partial;
        if (cap <= 16384 && (batch || !stage)) {
            const int rc = launch_draft_team(ctx, P, st);
            if (rc != kDraftNoFit) return rc;  // (the largest draft shapes leave no room for the staged history)
        }
        if (!stage) return launch_draft_stream(ctx, P, st);
    }
    P.slots = slots;
    P.max_groups = slots / 2;
    const size_t table_bytes = (size_t)slots * 3 * sizeof(int) + (size_t)P.max_groups * sizeof(int);
    const size_t cand_bytes = (size_t)(n_q * topk + kMaxKTab) * w * sizeof(int32_t);  // aliases the table
    const size_t work_bytes = ((table_bytes > cand_bytes ? table_bytes : cand_bytes) + 15) & ~size_t(15);
    P.stage_hist = stage ? 1 : 0;
    P.hist_off = (int)(work_bytes / sizeof(int));
    const size_t smem = ((sizeof(DraftSmem) + 15) & ~size_t(15)) + work_bytes + (P.stage_hist ? (size_t)cap * sizeof(int32_t) : 0);
    static bool attr_set[64] = {false};
    std::unique_lock<std::mutex> lock(host_mutex());
    bool& attr_done = attr_set[ctx->device & 63];
    if (!attr_done) {
        int rc = check_cuda(ctx, cudaFuncSetAttribute(draft_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024),
                            "draft: cudaFuncSetAttribute");
        if (rc) return rc;
        attr_done = true;
    }
    lock.unlock();
    cudaError_t e = launch_pdl_cluster(draft_kernel, dim3((unsigned)S * csize), dim3(threads), smem, st, csize, P);
    ctx->launches += 1;
    return check_cuda(ctx, e, "draft_context_ngrams launch");
}

}  // namespace ngs
