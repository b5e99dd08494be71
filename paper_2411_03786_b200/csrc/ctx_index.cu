// Incremental context index: drafting without scanning the history.
//
// The scan kernels find the earlier occurrences of the last q tokens by reading the whole history at every
// step.  The index keeps what that scan would find: per sequence and query length q, a hash table of the
// groups (q-gram, continuation) -> (count, latest start) over every complete window of q + w tokens of the
// history.  Committing a step's tokens adds the few windows that became complete; drafting looks up the
// current q-gram and ranks its groups.  Results are those of the scan (same windows, same grouping, same
// order): the index is a cache of it, and whenever it cannot answer (never built, out of step with the
// history, a table that ran out of probes, more groups than the lookup can rank) the sequence is drafted by
// scanning, never by guessing.
//
// Table layout: open addressing with linear probing, home slot = hash of the q-gram, so all groups of one
// q-gram lie on one probe run and a warp reads them 32 entries at a time.  An entry is 16 bytes:
//   key   = tag << 32 | start of the first-seen continuation (the tokens themselves stay in the history:
//           the q-gram is hist[start - q .. start), the continuation hist[start .. start + w));
//           tag = 16 bits of a second q-gram hash | 16 bits of a continuation hash (a filter: equality is
//           always confirmed on the tokens)
//   count = windows in the group,  last = latest continuation start of the group.
// A table has at least 1.5 times as many slots as the history capacity, so it never fills.
#include "accept.cuh"
#include "draft_common.cuh"

namespace ngs {

constexpr unsigned long long kIndexEmpty = ~0ull;
constexpr int kIndexHeaderInts = 32;
constexpr int kIndexMaxGroups = 2048;   // groups of one sequence's current q-grams the lookup ranks
constexpr int kIndexThreads = 128;
constexpr int kIndexFallbackSlots = 1024;

struct IndexEntry {
    unsigned long long key;
    int count;
    int last;
};

struct IndexView {
    int S, cap, n_q, w, key_len, slots;
    int qs[kMaxNQ];
    int* state;          // [S][2]: indexed length, valid
    IndexEntry* tables;  // [S][n_q][slots]
};

static size_t index_state_bytes(int S) { return ((size_t)S * 8 + 15) & ~size_t(15); }
static int index_slots(int cap) {  // a power of two at least 1.5 times the capacity: never more than two thirds full
    int s = 64;
    while (2 * s < 3 * cap) s <<= 1;
    return s;
}

static IndexView make_view(const spec_ctx::IndexMeta& m) {
    IndexView v;
    v.S = m.S;
    v.cap = m.cap;
    v.n_q = m.n_q;
    v.w = m.w;
    v.key_len = m.key_len;
    v.slots = m.slots;
    for (int i = 0; i < kMaxNQ; ++i) v.qs[i] = m.qs[i];
    char* base = reinterpret_cast<char*>(m.ptr);
    v.state = reinterpret_cast<int*>(base + kIndexHeaderInts * 4);
    v.tables = reinterpret_cast<IndexEntry*>(base + kIndexHeaderInts * 4 + index_state_bytes(m.S));
    return v;
}

// Hash of n tokens held in registers (n <= N).
template <int N>
__device__ __forceinline__ uint32_t hash_tokens(const int (&t)[N], int n, uint32_t seed) {
    uint32_t hsh = seed;
#pragma unroll
    for (int i = 0; i < N; ++i)
        if (i < n) hsh = hsh * 0x85EBCA6Bu + (uint32_t)t[i];
    return fmix32(hsh);
}

// A window in registers: qg[t] = the q-gram's token t + 1 places before the continuation start, ct[t] = the
// continuation's token t.  All loads are issued before the first use (one memory latency, not q + w of them).
struct Window {
    int qg[kMaxQ];
    int ct[kMaxW];
};
__device__ __forceinline__ Window load_window(const int32_t* h, int p, int q, int key_len) {
    Window wv;
#pragma unroll
    for (int t = 0; t < kMaxQ; ++t) wv.qg[t] = t < q ? h[p - 1 - t] : 0;
#pragma unroll
    for (int t = 0; t < kMaxW; ++t) wv.ct[t] = t < key_len ? h[p + t] : 0;
    return wv;
}
__device__ __forceinline__ bool same_window(const Window& a, const int32_t* h, int rp, int q, int key_len) {
    int diff = 0;
#pragma unroll
    for (int t = 0; t < kMaxQ; ++t)
        if (t < q) diff |= h[rp - 1 - t] ^ a.qg[t];
#pragma unroll
    for (int t = 0; t < kMaxW; ++t)
        if (t < key_len) diff |= h[rp + t] ^ a.ct[t];
    return diff == 0;
}
__device__ __forceinline__ uint32_t qgram_hash(const int (&qg)[kMaxQ], int q) { return hash_tokens(qg, q, 0x9E3779B9u); }
__device__ __forceinline__ uint32_t qgram_tag16(uint32_t qh) { return fmix32(qh + 0x632BE5ABu) >> 16; }

// Adds the window wv whose continuation starts at p (q-gram hist[p - q .. p), p >= q, p + w <= length) to
// table `tbl`.  Safe against concurrent inserts into the same table.  Returns false if the probe run never ended.
__device__ __forceinline__ bool index_insert(IndexEntry* tbl, int slots, const int32_t* h, const Window& wv, int p, int q, int key_len) {
    const uint32_t qh = qgram_hash(wv.qg, q);
    const uint32_t ch = hash_tokens(wv.ct, key_len, 0x7F4A7C15u);
    const uint32_t tag = (qgram_tag16(qh) << 16) | (ch >> 16);
    const unsigned long long mine = ((unsigned long long)tag << 32) | (uint32_t)p;
    uint32_t slot = qh & (uint32_t)(slots - 1);
    for (int probe = 0; probe < slots; ++probe) {
        unsigned long long cur = *((volatile unsigned long long*)&tbl[slot].key);
        if (cur == kIndexEmpty) {
            const unsigned long long old = atomicCAS(&tbl[slot].key, kIndexEmpty, mine);
            if (old == kIndexEmpty) {
                atomicAdd(&tbl[slot].count, 1);
                atomicMax(&tbl[slot].last, p);
                return true;
            }
            cur = old;
        }
        if ((uint32_t)(cur >> 32) == tag && same_window(wv, h, (int)(uint32_t)cur, q, key_len)) {
            atomicAdd(&tbl[slot].count, 1);
            atomicMax(&tbl[slot].last, p);
            return true;
        }
        slot = (slot + 1) & (uint32_t)(slots - 1);
    }
    return false;
}

__global__ void index_init_kernel(IndexView ix, int* header) {
    const size_t n = (size_t)ix.S * ix.n_q * ix.slots;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        ix.tables[i].key = kIndexEmpty;
        ix.tables[i].count = 0;
        ix.tables[i].last = -1;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        header[0] = 0x4E474958;
        header[1] = ix.S;
        header[2] = ix.cap;
        header[3] = ix.n_q;
        for (int i = 0; i < kMaxNQ; ++i) header[4 + i] = ix.qs[i];
        header[8] = ix.w;
        header[9] = ix.key_len;
        header[10] = ix.slots;
    }
}

// Every complete window of every sequence, one thread per (sequence, query length, continuation start).
__global__ void index_build_kernel(IndexView ix, const int32_t* __restrict__ hist, const int32_t* __restrict__ len, int* status) {
    const size_t n = (size_t)ix.S * ix.n_q * ix.cap;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int p = (int)(i % ix.cap);
        const int qi = (int)((i / ix.cap) % ix.n_q);
        const int s = (int)(i / ((size_t)ix.cap * ix.n_q));
        int L = len[s];
        const bool bad_len = L < 0 || L > ix.cap;
        if (bad_len) L = 0;
        if (p == 0 && qi == 0) {
            ix.state[2 * s] = L;
            if (bad_len) {
                ix.state[2 * s + 1] = 0;
                atomicOr(status, SPEC_STATUS_CAPACITY);
            }
        }
        const int q = ix.qs[qi];
        if (p < q || p + ix.w > L) continue;
        const int32_t* h = hist + (size_t)s * ix.cap;
        const Window wv = load_window(h, p, q, ix.key_len);
        if (!index_insert(ix.tables + ((size_t)s * ix.n_q + qi) * ix.slots, ix.slots, h, wv, p, q, ix.key_len)) {
            ix.state[2 * s + 1] = 0;
            atomicOr(status, SPEC_STATUS_INDEX);
        }
    }
}

__global__ void index_mark_valid_kernel(IndexView ix) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < ix.S) ix.state[2 * s + 1] = 1;
}

// The same insertion by a whole warp (every lane holds the same window): the probe run is read 32 slots at a
// time, so a q-gram with hundreds of groups costs a few steps, not hundreds of dependent loads.  Safe against
// other warps inserting into the same table.
__device__ __forceinline__ bool index_insert_warp(IndexEntry* tbl, int slots, const int32_t* h, const Window& wv, int p, int q, int key_len,
                                                  int lane) {
    const uint32_t qh = qgram_hash(wv.qg, q);
    const uint32_t ch = hash_tokens(wv.ct, key_len, 0x7F4A7C15u);
    const uint32_t tag = (qgram_tag16(qh) << 16) | (ch >> 16);
    const unsigned long long mine = ((unsigned long long)tag << 32) | (uint32_t)p;
    const uint32_t home = qh & (uint32_t)(slots - 1);
    int retries = 0;
    for (int it = 0; it * 32 < slots; ++it) {
        const uint32_t slot = (home + it * 32 + lane) & (uint32_t)(slots - 1);
        const unsigned long long cur = *((volatile unsigned long long*)&tbl[slot].key);
        const bool empty = cur == kIndexEmpty;
        const unsigned eb = __ballot_sync(0xffffffffu, empty);
        const bool before_end = eb == 0u || lane < __ffs(eb) - 1;  // the run ends at its first empty slot
        const bool found = before_end && (uint32_t)(cur >> 32) == tag && same_window(wv, h, (int)(uint32_t)cur, q, key_len);
        const unsigned fb = __ballot_sync(0xffffffffu, found);
        if (fb) {
            if (lane == __ffs(fb) - 1) {
                atomicAdd(&tbl[slot].count, 1);
                atomicMax(&tbl[slot].last, p);
            }
            return true;
        }
        if (eb) {  // the group is new: it takes the slot that ends the run
            const int first = __ffs(eb) - 1;
            unsigned long long old = 0ull;
            if (lane == first) old = atomicCAS(&tbl[slot].key, kIndexEmpty, mine);
            old = __shfl_sync(0xffffffffu, old, first);
            if (old == kIndexEmpty) {
                if (lane == first) {
                    atomicAdd(&tbl[slot].count, 1);
                    atomicMax(&tbl[slot].last, p);
                }
                return true;
            }
            if (++retries > 64) return false;
            --it;  // another warp took that slot meanwhile: look at these 32 slots again
        }
    }
    return false;
}

// Greedy acceptance and commit (as accept_commit_kernel), then the windows that the committed tokens completed
// are added to the index.  One CTA of four warps per sequence: warp 0 accepts and commits, then every warp
// inserts some of the (window, query length) pairs, a pair at a time.
__global__ void __launch_bounds__(128) accept_commit_index_kernel(const AcceptArgs a, IndexView ix) {
    __shared__ int sh_old, sh_new, sh_fail;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int s = blockIdx.x;
    grid_launch_dependents();
    grid_dependency_wait();
    if (warp == 0) {
        const int L_old = a.len[s];
        __syncwarp();
        accept_sequence(a, s, lane);
        __threadfence();
        __syncwarp();  // the committed tokens and the new length are visible to the whole warp
        if (lane == 0) {
            sh_old = L_old;
            sh_new = *((volatile int*)&a.len[s]);
            sh_fail = 0;
        }
    }
    __syncthreads();  // ... and, through the fence above, to the whole CTA
    const int L_old = sh_old, L_new = sh_new;
    int* st = ix.state + 2 * s;
    const bool in_step = st[1] != 0 && st[0] == L_old && L_old >= 0 && L_new <= ix.cap;
    __syncthreads();
    if (!in_step) {  // not built, or the history moved without the index: it stays unusable until it is rebuilt
        if (threadIdx.x == 0) st[1] = 0;
        return;
    }
    if (L_new == L_old) return;  // nothing was committed (no room)
    const int32_t* h = a.hist + (size_t)s * a.cap;  // (written a moment ago: plain loads)
    const int p_lo = L_old - ix.w + 1, n_new = L_new - L_old;  // continuation starts p_lo .. p_lo + n_new - 1
    for (int item = warp; item < n_new * ix.n_q; item += 4) {
        const int p = p_lo + item / ix.n_q, qi = item % ix.n_q, q = ix.qs[qi];
        if (p < q) continue;
        const Window wv = load_window(h, p, q, ix.key_len);
        if (!index_insert_warp(ix.tables + ((size_t)s * ix.n_q + qi) * ix.slots, ix.slots, h, wv, p, q, ix.key_len, lane) && lane == 0) sh_fail = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        st[0] = L_new;
        if (sh_fail) {
            st[1] = 0;
            atomicOr(a.status, SPEC_STATUS_INDEX);
        }
    }
}

// ------------------------------------------------------------------------------------------ drafting from the index
struct IndexDraftLayout {
    int gkey, skey, rank, run_key, cand_rows, cand, row_of, chain, table, queue, misc, bytes;
    int n_cand_max;
};

struct IndexDraftMisc {
    int n_keys;
    int use_scan;
    int n_groups;
    int overflow;
    int n_out;
    int n_surv;
    int reached;
    int pad_;
    int n_run[kMaxNQ];
    int n_cnt[kMaxNQ];
    int tq[kMaxQ];
    int cand_off[kMaxNQ + 2];
    unsigned long long tau[kMaxNQ];
};

// One CTA per sequence.  `qmap[i]` = position of the draft's i-th query length in the index.
__global__ void __launch_bounds__(kIndexThreads) draft_index_kernel(const DraftParams P, const IndexDraftLayout Y, IndexView ix,
                                                                   int qmap0, int qmap1, int qmap2, int qmap3) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NT = kIndexThreads, NW = kIndexThreads / 32;
    IndexDraftMisc* sm = reinterpret_cast<IndexDraftMisc*>(smem_raw + Y.misc);
    DraftScratch X;
    X.gkey = reinterpret_cast<unsigned long long*>(smem_raw + Y.gkey);
    X.rank_acc = reinterpret_cast<int*>(smem_raw + Y.rank);
    X.run_key = reinterpret_cast<unsigned long long*>(smem_raw + Y.run_key);
    X.n_run = sm->n_run;
    X.n_cnt = sm->n_cnt;
    X.cand = reinterpret_cast<int32_t*>(smem_raw + Y.cand_rows);
    X.cand_src = reinterpret_cast<int*>(smem_raw + Y.cand);
    X.cand_cnt = X.cand_src + Y.n_cand_max;
    X.cand_keep = X.cand_cnt + Y.n_cand_max;
    X.dropped = X.cand_keep + Y.n_cand_max;
    X.row_of = reinterpret_cast<int*>(smem_raw + Y.row_of);
    X.chain = reinterpret_cast<int*>(smem_raw + Y.chain);
    X.chain_ok = X.chain + P.k_tab * P.w;
    X.cand_off = sm->cand_off;
    X.n_out = &sm->n_out;
    X.n_surv = &sm->n_surv;
    X.tau = sm->tau;
    unsigned long long* skey = reinterpret_cast<unsigned long long*>(smem_raw + Y.skey);
    auto sync = [&]() { __syncthreads(); };

    const int s = blockIdx.x;
    grid_launch_dependents();
    grid_dependency_wait();  // history, lengths and the index come from the previous step's commit
    const int32_t* __restrict__ h = P.hist + (size_t)s * P.cap;
    int L = P.len[s];
    if (L < 0 || L > P.cap) {
        if (tid == 0) atomicOr(P.status, SPEC_STATUS_CAPACITY);
        L = 0;
    }
    const int* st = ix.state + 2 * s;
    if (tid == 0) {
        sm->n_keys = 0;
        sm->n_surv = 0;
        sm->use_scan = (st[1] != 0 && st[0] == L) ? 0 : 1;  // the index answers only when it is in step with the history
    }
    if (tid < kMaxQ) sm->tq[tid] = (tid < L) ? h[L - 1 - tid] : -2;
    if (tid < kMaxNQ) {
        sm->n_run[tid] = 0;
        sm->n_cnt[tid] = 0;
    }
    if (tid < P.k_tab) X.chain_ok[tid] = 0;
    __syncthreads();
    // extended model bigram of the last token (rank r on lane r), by the last warp
    if (warp == NW - 1 && (P.flags & SPEC_FLAG_MODEL_FILL) && L >= 1) model_chain(P, sm->tq[0], lane, X.chain, X.chain_ok);

    if (!sm->use_scan) {
        // ---- look the current q-grams up: warp i takes the draft's i-th query length
        const int qmap[kMaxNQ] = {qmap0, qmap1, qmap2, qmap3};
        for (int qi = warp; qi < P.n_q; qi += NW) {
            const int q = P.qs[qi];
            if (L < q + P.w) continue;  // no complete window yet
            const IndexEntry* tbl = ix.tables + ((size_t)s * ix.n_q + qmap[qi]) * ix.slots;
            int qg[kMaxQ];
#pragma unroll
            for (int t = 0; t < kMaxQ; ++t) qg[t] = sm->tq[t];  // tq[t] = the token t + 1 places before the end
            const uint32_t qh = qgram_hash(qg, q);
            const uint32_t qtag = qgram_tag16(qh);
            const uint32_t home = qh & (uint32_t)(ix.slots - 1);
            for (int it = 0; it * 32 < ix.slots; ++it) {
                const IndexEntry e = tbl[(home + it * 32 + lane) & (uint32_t)(ix.slots - 1)];
                const bool empty = e.key == kIndexEmpty;
                const unsigned eb = __ballot_sync(0xffffffffu, empty);
                const bool before_end = eb == 0u || lane < __ffs(eb) - 1;  // the run ends at its first empty slot
                bool match = before_end && !empty && (uint32_t)(e.key >> 48) == qtag;
                if (match) {
                    const int rp = (int)(uint32_t)e.key;
                    int diff = 0;
#pragma unroll
                    for (int t = 0; t < kMaxQ; ++t)
                        if (t < q) diff |= h[rp - 1 - t] ^ qg[t];
                    match = diff == 0;
                }
                if (match) {
                    const int idx = atomicAdd(&sm->n_keys, 1);
                    if (idx < kIndexMaxGroups) {
                        X.gkey[idx] = ((unsigned long long)qi << 60) | ((unsigned long long)(uint32_t)e.count << 32) | (uint32_t)e.last;
                        X.rank_acc[idx] = 0;
                    }
                }
                if (eb) break;
            }
        }
        __syncthreads();
        if (sm->n_keys > kIndexMaxGroups) {  // more groups than the lookup ranks: this sequence is scanned instead
            __syncthreads();
            if (tid == 0) sm->use_scan = 1;
            if (tid < kMaxNQ) sm->n_cnt[tid] = 0;
            __syncthreads();
        } else {
            rank_keys(P, sm->n_keys, skey, X, tid, NT, sync);
        }
    }
    if (sm->use_scan) {
        // ---- the scan, as in the batch kernels (history read from global memory, a small table, as many passes as it takes)
        DraftTable tab;
        tab.rep = reinterpret_cast<int*>(smem_raw + Y.table);
        tab.cnt = tab.rep + P.slots;
        tab.last = tab.cnt + P.slots;
        tab.grp_slot = tab.last + P.slots;
        tab.n_groups = &sm->n_groups;
        tab.overflow = &sm->overflow;
        int* wq = reinterpret_cast<int*>(smem_raw + Y.queue) + warp * kMatchQueue;
        const int n_scan = L - P.w;
        const int t0 = sm->tq[0], t1 = sm->tq[1], t2 = sm->tq[2], t3 = sm->tq[3];
        bool any_q = false;
        for (int qi = 0; qi < P.n_q; ++qi) any_q = any_q || (L >= P.qs[qi] + P.w);
        int R = 1;
        bool gave_up = false;
        while (any_q && n_scan >= 1) {
            __syncthreads();
            if (tid < kMaxNQ) sm->n_run[tid] = 0;
            bool overflowed = false;
            for (int r = 0; r < R && !overflowed; ++r) {
                for (int i = tid; i < P.slots; i += NT) {
                    tab.rep[i] = -1;
                    tab.cnt[i] = 0;
                    tab.last[i] = -1;
                }
                if (tid == 0) {
                    sm->n_groups = 0;
                    sm->overflow = 0;
                }
                __syncthreads();
                const int reached = scan_pass(P, h, L, R, r, t0, t1, t2, t3, tab, wq, tid, NT);
                if (tid == 0) sm->reached = reached;
                __syncthreads();
                if (*((volatile int*)&sm->overflow)) {
                    overflowed = true;
                    break;
                }
                rank_pass(P, tab, X, tid, NT, sync);
            }
            if (!overflowed) break;
            R = next_pass_count(R, sm->reached, (max(n_scan, 0) + 3) >> 2);
            if (R > kMaxPasses) {
                gave_up = true;
                break;
            }
        }
        mix_and_emit(P, s, h, L, gave_up, X, tid, NT, sync);
    } else {
        mix_and_emit(P, s, h, L, false, X, tid, NT, sync);
    }
}

static int round_up16(int x) { return (x + 15) & ~15; }

// ------------------------------------------------------------------------------------------ host side
size_t context_index_bytes(int S, int cap, int n_q) {
    return (size_t)kIndexHeaderInts * 4 + index_state_bytes(S) + (size_t)S * n_q * index_slots(cap) * sizeof(IndexEntry);
}

int launch_index_build(spec_ctx* ctx, void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs,
                       int n_q, int w, int key_len, cudaStream_t st) {
    spec_ctx::IndexMeta& m = ctx->index;
    m.ptr = d_index;
    m.S = S;
    m.cap = cap;
    m.n_q = n_q;
    for (int i = 0; i < kMaxNQ; ++i) m.qs[i] = i < n_q ? qs[i] : 0;
    m.w = w;
    m.key_len = key_len;
    m.slots = index_slots(cap);
    const IndexView ix = make_view(m);
    const int blocks = ctx->num_sms * 8;
    index_init_kernel<<<blocks, 256, 0, st>>>(ix, reinterpret_cast<int*>(d_index));
    index_mark_valid_kernel<<<(S + 127) / 128, 128, 0, st>>>(ix);
    index_build_kernel<<<blocks, 256, 0, st>>>(ix, d_hist, d_len, ctx->d_status);
    ctx->launches += 3;
    return check_cuda(ctx, cudaGetLastError(), "spec_context_index_build launch");
}

int launch_accept_indexed(spec_ctx* ctx, const AcceptArgs& a, cudaStream_t st) {
    const IndexView ix = make_view(ctx->index);
    cudaError_t e = launch_pdl(accept_commit_index_kernel, dim3((unsigned)a.S), dim3(128), 0, st, a, ix);
    ctx->launches += 1;
    return check_cuda(ctx, e, "accept_and_commit_indexed launch");
}

int launch_draft_indexed(spec_ctx* ctx, DraftParams& P, cudaStream_t st) {
    const spec_ctx::IndexMeta& m = ctx->index;
    int qmap[kMaxNQ] = {0, 0, 0, 0};
    for (int i = 0; i < P.n_q; ++i) {
        int at = -1;
        for (int j = 0; j < m.n_q; ++j)
            if (m.qs[j] == P.qs[i]) at = j;
        if (at < 0) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: the index was not built for q = %d", P.qs[i]);
        qmap[i] = at;
    }
    P.slots = kIndexFallbackSlots;
    P.max_groups = P.slots / 2;
    P.stage_hist = 0;
    P.hist_off = 0;
    IndexDraftLayout Y{};
    Y.n_cand_max = P.n_q * P.topk + P.k_tab;
    if (Y.n_cand_max < 1) Y.n_cand_max = 1;
    const int key_cap = kIndexMaxGroups + P.n_q * P.topk;  // (also covers the scan's max_groups + winners)
    int off = 0;
    Y.gkey = off;
    off += round_up16(key_cap * 8);
    Y.skey = off;
    off += round_up16(key_cap * 8);
    Y.rank = off;
    off += round_up16(key_cap * 4);
    Y.run_key = off;
    off += round_up16((P.n_q > 0 ? P.n_q : 1) * P.topk * 8);
    Y.cand_rows = off;
    off += round_up16(Y.n_cand_max * P.w * 4);
    Y.cand = off;
    off += round_up16(4 * Y.n_cand_max * 4);
    Y.row_of = off;
    off += round_up16(P.B * 4);
    Y.chain = off;
    off += round_up16((P.k_tab * P.w + kMaxKTab) * 4);
    Y.table = off;
    off += round_up16((P.slots * 3 + P.max_groups) * 4);
    Y.queue = off;
    off += round_up16((kIndexThreads / 32) * kMatchQueue * 4);
    Y.misc = off;
    off += round_up16((int)sizeof(IndexDraftMisc));
    Y.bytes = off;
    {
        static bool attr_set[64] = {};
        std::lock_guard<std::mutex> lock(host_mutex());
        if (!attr_set[ctx->device & 63]) {
            int rc = check_cuda(ctx, cudaFuncSetAttribute(draft_index_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024),
                                "draft (indexed): cudaFuncSetAttribute");
            if (rc) return rc;
            attr_set[ctx->device & 63] = true;
        }
    }
    const IndexView ix = make_view(m);
    cudaError_t e = launch_pdl(draft_index_kernel, dim3((unsigned)P.S), dim3(kIndexThreads), (size_t)Y.bytes, st, P, Y, ix, qmap[0], qmap[1],
                               qmap[2], qmap[3]);
    ctx->launches += 1;
    return check_cuda(ctx, e, "draft_context_ngrams_indexed launch");
}

}  // namespace ngs
