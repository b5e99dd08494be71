// Context N-gram drafting for batches of long histories (too long to stage in shared memory): one
// persistent CTA per SM whose warps are split into scanners, finishers and a fetcher.
//
// Streaming a long history is bound by memory bandwidth; everything around the scan of a sequence (its
// number, length and last tokens - three dependent loads that each take microseconds while the memory
// system is saturated -, clearing the table, ranking the groups, mixing, dropping duplicates, writing
// the drafts) is a chain of short phases separated by barriers and dependent loads, about as long as
// the scan of 100K tokens itself.  When every CTA does all of it, the CTAs of an SM run in lockstep - all
// scan, then all finish - and the memory pipe idles half of the time.  Here the jobs belong to
// different warps of one CTA:
//   - 24 scanner warps stream the history of one sequence after the other (128-bit loads, several per
//     thread in flight) and group the matches in a hash table in shared memory; between two sequences
//     they do nothing but two barrier hand-shakes;
//   - 7 finisher warps take a finished table, rank its groups, clear the table and give it back, then mix
//     the rows and write the outputs of that sequence, while the scanners are already streaming the next
//     sequence into the other table;
//   - 1 fetcher warp runs two sequences ahead: it takes the next sequence from the global counter and
//     reads its length and last tokens, so that the scanners find them in shared memory.
// Tables and sequence descriptors are handed over with named barriers in the producer / consumer form
// (the producer arrives at `full`, the consumer waits on it, and the other way round for `empty`).  A
// sequence with more distinct continuations than a table holds is scanned in R = 2, 4, ... hash-residue
// passes, one table hand-over per pass, the finishers merging each pass's groups with the winners so far
// (exact, as in the other drafting kernels).  Sequences come from a global counter, so SMs balance; the
// CTA that exits last re-arms it.
// Semantics are those of the latency kernel in draft.cu; results are bit-identical.
#include "draft_common.cuh"

namespace ngs {

constexpr int STREAM_SCAN_WARPS = 24, STREAM_POST_WARPS = 7;
constexpr int SWT = STREAM_SCAN_WARPS * 32, PWT = STREAM_POST_WARPS * 32;
constexpr int STREAM_THREADS = SWT + PWT + 32;
#ifndef NGRAM_STREAM_LOADS
#define NGRAM_STREAM_LOADS 6
#endif
constexpr int STREAM_LOADS = NGRAM_STREAM_LOADS;  // 128-bit loads a scanner thread keeps in flight
// named barriers (barrier 0 is the CTA's); + b = table, + k = descriptor slot
constexpr int BAR_FULL = 1;     // table b complete               (scanners arrive, finishers wait)
constexpr int BAR_EMPTY = 3;    // table b cleared and free       (finishers arrive, scanners wait)
constexpr int BAR_SCAN = 5;     // the scanner warps among themselves
constexpr int BAR_POST = 6;     // the finisher warps among themselves
constexpr int BAR_FFULL = 7;    // sequence descriptor k written  (fetcher arrives, scanners wait)
constexpr int BAR_FEMPTY = 9;   // sequence descriptor k read     (scanners arrive, fetcher waits)
constexpr int TABLE_COUNT = SWT + PWT, FETCH_COUNT = SWT + 32;

enum { PASS_FIRST = 1, PASS_LAST = 2, PASS_VOID = 4, PASS_GAVE_UP = 8, PASS_EXIT = 16 };

struct PassDesc {
    int seq, L, flags, pad;
};
struct SeqDesc {
    int seq, L;
    int tq[kMaxQ];
    int pad[2];
};

struct StreamLayout {
    int table[2];  // int rep[slots], cnt[slots], last[slots], grp_slot[max_groups]
    int gkey, rank, run_key, cand_rows, cand, row_of, chain, queue, misc;
    int bytes;
    int n_cand_max, gkey_cap;
};

struct StreamMisc {
    PassDesc desc[2];
    SeqDesc seqd[2];
    int n_groups[2];
    int overflow[2];
    int n_out;
    int n_run[kMaxNQ];
    int n_cnt[kMaxNQ];
    int cand_off[kMaxNQ + 2];
    int n_surv;
    int reached;
    unsigned long long tau[kMaxNQ];
};

__device__ __forceinline__ void named_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int count) {
    __threadfence_block();  // what this thread wrote to shared memory is visible to the threads that wait on the barrier
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

template <bool PT>  // PT: SPEC_FLAG_PARTIAL_TAIL
__global__ void __launch_bounds__(STREAM_THREADS, 1) draft_stream_kernel(const DraftParams P, const StreamLayout Y, unsigned int* work) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    StreamMisc* sm = reinterpret_cast<StreamMisc*>(smem_raw + Y.misc);
    auto table = [&](int b) {
        DraftTable t;
        t.rep = reinterpret_cast<int*>(smem_raw + Y.table[b]);
        t.cnt = t.rep + P.slots;
        t.last = t.cnt + P.slots;
        t.grp_slot = t.last + P.slots;
        t.n_groups = &sm->n_groups[b];
        t.overflow = &sm->overflow[b];
        return t;
    };

    grid_launch_dependents();
    grid_dependency_wait();  // histories and lengths come from the previous step's commit; the counter from the previous batch

    if (threadIdx.x < SWT) {
        // ------------------------------------------------------------------ scanners
        const int tid = (int)threadIdx.x, warp = tid >> 5;
        int* wq = reinterpret_cast<int*>(smem_raw + Y.queue) + warp * kMatchQueue;
        int buf = 0, k = 0;
        for (;;) {
            named_sync(BAR_FFULL + k, FETCH_COUNT);  // the fetcher has prepared this sequence
            const int s = sm->seqd[k].seq, L = sm->seqd[k].L;
            const int t0 = sm->seqd[k].tq[0], t1 = sm->seqd[k].tq[1], t2 = sm->seqd[k].tq[2], t3 = sm->seqd[k].tq[3];
            if (s >= P.S) break;
            named_arrive(BAR_FEMPTY + k, FETCH_COUNT);
            k ^= 1;
            const int32_t* __restrict__ h = P.hist + (size_t)s * P.cap;
            constexpr bool partial = PT;
            bool any_q = false;
            for (int qi = 0; qi < P.n_q; ++qi) any_q = any_q || (L >= P.qs[qi] + (partial ? 1 : P.w));
            const bool scan = any_q && (L - P.w >= 1 || (partial && L >= 2));
            int R = 1;
            for (;;) {
                bool overflowed = false;
                const bool gave_up = R > kMaxPasses;  // one more hand-over, of an empty table marked PASS_GAVE_UP
                for (int r = 0; r < R && !overflowed; ++r) {
                    named_sync(BAR_EMPTY + buf, TABLE_COUNT);  // the finishers have cleared and released this table
                    const DraftTable T = table(buf);
                    if (tid == 0) {
                        sm->desc[buf].seq = s;
                        sm->desc[buf].L = L;
                        sm->desc[buf].flags = (r == 0 ? PASS_FIRST : 0) | ((r == R - 1 || gave_up) ? PASS_LAST : 0) | (gave_up ? PASS_GAVE_UP : 0);
                    }
                    int reached = 0;
                    if (scan && !gave_up) reached = scan_pass<STREAM_LOADS, PT>(P, h, L, R, r, t0, t1, t2, t3, T, wq, tid, SWT);
                    if (tid == 0) sm->reached = reached;
                    named_sync(BAR_SCAN, SWT);  // every scanner's matches are in the table
                    overflowed = *((volatile int*)T.overflow) != 0;
                    if (overflowed && tid == 0) sm->desc[buf].flags |= PASS_VOID;  // this pass does not count: more passes follow
                    named_arrive(BAR_FULL + buf, TABLE_COUNT);
                    buf ^= 1;
                    if (gave_up) break;
                }
                if (!overflowed || gave_up) break;
                R = next_pass_count(R, sm->reached, (max(L - P.w, 0) + 3) >> 2);
            }
        }
        // tell the finishers to stop, then wait until they have released the other table too
        named_sync(BAR_EMPTY + buf, TABLE_COUNT);
        if (tid == 0) sm->desc[buf].flags = PASS_EXIT;
        named_arrive(BAR_FULL + buf, TABLE_COUNT);
        named_sync(BAR_EMPTY + (buf ^ 1), TABLE_COUNT);
    } else if (threadIdx.x < SWT + PWT) {
        // ------------------------------------------------------------------ finishers
        const int tid = (int)threadIdx.x - SWT, lane = tid & 31, warp = tid >> 5;
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
        auto post_sync = [&]() { named_sync(BAR_POST, PWT); };
        // clear table b and hand it to the scanners
        auto release = [&](int b) {
            const DraftTable T = table(b);
            for (int i = tid; i < P.slots; i += PWT) {
                T.rep[i] = -1;
                T.cnt[i] = 0;
                T.last[i] = -1;
            }
            if (tid == 0) {
                *T.n_groups = 0;
                *T.overflow = 0;
            }
            named_arrive(BAR_EMPTY + b, TABLE_COUNT);
        };
        release(0);
        release(1);
        int buf = 0;
        for (;;) {
            named_sync(BAR_FULL + buf, TABLE_COUNT);
            const int flags = sm->desc[buf].flags, s = sm->desc[buf].seq, L = sm->desc[buf].L;
            if (flags & PASS_EXIT) break;
            const int32_t* __restrict__ h = P.hist + (size_t)s * P.cap;
            if (flags & PASS_FIRST) {  // a new sequence, or a new round of passes: forget the winners so far
                if (tid < kMaxNQ) sm->n_run[tid] = 0;
                if (tid < P.k_tab) X.chain_ok[tid] = 0;
                post_sync();
                // extended model bigram of the last token (rank r on lane r), by the last finisher warp
                if (warp == STREAM_POST_WARPS - 1 && (P.flags & SPEC_FLAG_MODEL_FILL) && L >= 1) model_chain(P, h[L - 1], lane, X.chain, X.chain_ok);
            }
            if (!(flags & PASS_VOID)) rank_pass(P, table(buf), X, tid, PWT, post_sync);
            else post_sync();
            release(buf);  // the winners live in run_key: the scanners may fill this table again
            if ((flags & PASS_LAST) && !(flags & PASS_VOID)) mix_and_emit(P, s, h, L, (flags & PASS_GAVE_UP) != 0, X, tid, PWT, post_sync);
            buf ^= 1;
        }
    } else {
        // ------------------------------------------------------------------ fetcher (one warp)
        const int lane = (int)threadIdx.x & 31;
        int k = 0;
        int used[2] = {0, 0};
        for (;;) {
            if (used[k] > 0) named_sync(BAR_FEMPTY + k, FETCH_COUNT);  // the scanners have read what this slot held
            int s = 0;
            if (lane == 0) s = (int)atomicAdd(&work[0], 1u);
            s = __shfl_sync(0xffffffffu, s, 0);
            int L = 0, tok = -2;
            if (s < P.S) {
                L = P.len[s];
                if (L < 0 || L > P.cap) {
                    if (lane == 0) atomicOr(P.status, SPEC_STATUS_CAPACITY);
                    L = 0;
                }
                if (lane < kMaxQ && lane < L) tok = P.hist[(size_t)s * P.cap + L - 1 - lane];
            }
            if (lane == 0) {
                sm->seqd[k].seq = s;
                sm->seqd[k].L = L;
            }
            if (lane < kMaxQ) sm->seqd[k].tq[lane] = tok;
            named_arrive(BAR_FFULL + k, FETCH_COUNT);
            used[k] += 1;
            if (s >= P.S) break;  // (the scanners do not release the slot that tells them to stop)
            k ^= 1;
        }
        if (used[k ^ 1] > 0) named_sync(BAR_FEMPTY + (k ^ 1), FETCH_COUNT);  // the release of the last real sequence's slot
    }

    // The CTA that leaves last re-arms the work counter for the next batch.
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

int launch_draft_stream(spec_ctx* ctx, DraftParams& P, cudaStream_t st) {
    P.slots = 4096;  // two tables of 2048 groups each
    P.max_groups = P.slots / 2;
    P.stage_hist = 0;
    P.hist_off = 0;
    StreamLayout Y{};
    Y.n_cand_max = P.n_q * P.topk + P.k_tab;
    if (Y.n_cand_max < 1) Y.n_cand_max = 1;
    Y.gkey_cap = P.max_groups + P.n_q * P.topk;
    int off = 0;
    for (int b = 0; b < 2; ++b) {
        Y.table[b] = off;
        off += round_up16((P.slots * 3 + P.max_groups) * 4);
    }
    Y.gkey = off;
    off += round_up16(Y.gkey_cap * 8);
    Y.rank = off;
    off += round_up16(Y.gkey_cap * 4);
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
    Y.queue = off;
    off += round_up16(STREAM_SCAN_WARPS * kMatchQueue * 4);
    Y.misc = off;
    off += round_up16((int)sizeof(StreamMisc));
    Y.bytes = off;  // at most about 190 KB (largest draft shape)
    const int pt = (P.flags & SPEC_FLAG_PARTIAL_TAIL) ? 1 : 0;
    void (*kern)(const DraftParams, const StreamLayout, unsigned int*) = pt ? draft_stream_kernel<true> : draft_stream_kernel<false>;
    {
        static bool attr_set[64][2] = {};
        std::lock_guard<std::mutex> lock(host_mutex());
        if (!attr_set[ctx->device & 63][pt]) {
            int rc = check_cuda(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024),
                                "draft (long histories): cudaFuncSetAttribute");
            if (rc) return rc;
            attr_set[ctx->device & 63][pt] = true;
        }
    }
    const int grid = P.S < ctx->num_sms ? P.S : ctx->num_sms;
    cudaError_t e = launch_pdl(kern, dim3((unsigned)grid), dim3(STREAM_THREADS), (size_t)Y.bytes, st, P, Y, ctx->d_draft_work);
    ctx->launches += 1;
    return check_cuda(ctx, e, "draft_context_ngrams (long histories) launch");
}

}  // namespace ngs
