// Context N-gram drafting and mixed allocation: one CTA per sequence.
//
// One streaming pass over the history serves every query length at once.  A position p is the
// start of a continuation for query length q when the q tokens before p equal the last q tokens
// of the history; the q values are nested (a q=3 match is also a q=2 and q=1 match), so the scan
// computes the length of the common suffix once per position.  Each match is grouped by its
// w-token continuation in a shared-memory hash table that resolves collisions by comparing the
// actual tokens, so grouping is exact.  If a sequence has more distinct continuations than the
// table holds, the scan is repeated in R passes, pass r keeping only the groups whose hash falls
// in residue class r, and the per-pass winners are merged: still exact, only slower.
#include "common.cuh"

namespace ngs {

struct DraftParams {
    const int32_t* hist;
    const int32_t* len;
    int S, cap;
    int qs[kMaxNQ];
    int n_q, q_max;
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
    int max_groups;  // slots / 2
};

constexpr int kMaxPasses = 1024;

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

struct DraftSmem {
    unsigned long long run_key[kMaxNQ][kMaxB];  // per query length: ranked (count << 32 | start) keys
    int32_t out[kMaxB][kMaxW];
    int32_t out_src[kMaxB];
    int32_t out_cnt[kMaxB];
    int32_t chain[kMaxKTab][kMaxW];
    int chain_ok[kMaxKTab];
    int n_run[kMaxNQ];
    int tq[kMaxQ];
    int n_groups;
    int overflow;
    int n_out;
};

// Group the match whose continuation starts at p (query index qi).
__device__ __forceinline__ void insert_match(const int32_t* __restrict__ h, int p, int qi, int w, uint32_t hsh,
                                             int slots, int max_groups, int* rep, int* cnt, int* last,
                                             int* grp_slot, DraftSmem* sm) {
    uint32_t slot = hsh & (uint32_t)(slots - 1);
    const int me = (qi << 28) | p;
    for (int probe = 0; probe < slots; ++probe) {
        int cur = *((volatile int*)&rep[slot]);
        if (cur == -1) {
            int old = atomicCAS(&rep[slot], -1, me);
            if (old == -1) {
                int g = atomicAdd(&sm->n_groups, 1);
                if (g >= max_groups) {
                    sm->overflow = 1;
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
            for (int t = 0; t < w; ++t)
                if (h[rp + t] != h[p + t]) {
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
    sm->overflow = 1;
}

__global__ void __launch_bounds__(1024) draft_kernel(const DraftParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DraftSmem* sm = reinterpret_cast<DraftSmem*>(smem_raw);
    int* rep = reinterpret_cast<int*>(smem_raw + ((sizeof(DraftSmem) + 15) & ~size_t(15)));
    int* cnt = rep + P.slots;
    int* last = cnt + P.slots;
    int* grp_slot = last + P.slots;

    const int tid = threadIdx.x, nthr = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
    const int s = blockIdx.x;
    const int32_t* __restrict__ h = P.hist + (size_t)s * P.cap;
    const int w = P.w;

    int L = P.len[s];
    if (L < 0 || L > P.cap) {
        if (tid == 0) atomicOr(P.status, SPEC_STATUS_CAPACITY);
        L = 0;
    }
    if (tid < kMaxQ) sm->tq[tid] = (tid < L) ? h[L - 1 - tid] : -2;
    if (tid < kMaxNQ) sm->n_run[tid] = 0;
    if (tid < kMaxKTab) sm->chain_ok[tid] = 0;
    __syncthreads();

    // ---- extended model bigram of the last token (rank r on lane r), overlapped with the scan
    if (warp == nwarps - 1 && (P.flags & SPEC_FLAG_MODEL_FILL) && L >= 1) {
        const int x = sm->tq[0];
        if (x < 0 || x >= P.V) {
            if (lane == 0) atomicOr(P.status, SPEC_STATUS_TOKEN_RANGE);
        } else if (lane < P.k_tab) {
            bool ok = true;
            if (P.ext != nullptr && w <= P.w_ext) {
                const int32_t* e = P.ext + ((size_t)x * P.k_tab + lane) * P.w_ext;
                for (int j = 0; j < w; ++j) {
                    int t = e[j];
                    ok = ok && (t >= 0 && t < P.V);
                    sm->chain[lane][j] = t;
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
    const int t0 = sm->tq[0], t1 = sm->tq[1], t2 = sm->tq[2], t3 = sm->tq[3];
    bool any_q = false;
    for (int qi = 0; qi < P.n_q; ++qi) any_q = any_q || (L >= P.qs[qi] + w);

    int R = 1;
    bool gave_up = false;
    while (any_q && n_scan >= 1) {
        __syncthreads();
        if (tid < kMaxNQ) sm->n_run[tid] = 0;
        bool overflowed = false;
        for (int r = 0; r < R && !overflowed; ++r) {
            for (int i = tid; i < P.slots; i += nthr) {
                rep[i] = -1;
                cnt[i] = 0;
                last[i] = -1;
            }
            if (tid == 0) {
                sm->n_groups = 0;
                sm->overflow = 0;
            }
            __syncthreads();
            // scan: 128-bit loads, four token positions per thread per step, two steps in flight
            const int4* h4 = reinterpret_cast<const int4*>(h);
            const int n_vec = (n_scan + 3) >> 2;
            for (int v0 = tid; v0 < n_vec; v0 += 2 * nthr) {
                int4 va = h4[v0];
                const int v1 = v0 + nthr;
                int4 vb = (v1 < n_vec) ? h4[v1] : make_int4(-3, -3, -3, -3);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int4 vv = half ? vb : va;
                    const int xb = (half ? v1 : v0) << 2;
                    const int toks[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int x = xb + e;
                        if (toks[e] != t0 || x >= n_scan) continue;
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
                        for (int t = 0; t < w; ++t) hc = fmix32(hc ^ (uint32_t)h[p + t]) + 0x7F4A7C15u;
                        for (int qi = 0; qi < P.n_q; ++qi) {
                            const int q = P.qs[qi];
                            if (m < q || L < q + w) continue;
                            const uint32_t hq = fmix32(hc + (uint32_t)qi * 0x632BE5ABu);
                            if (R > 1 && (int)(fmix32(hq ^ 0xA511E9B3u) % (uint32_t)R) != r) continue;
                            insert_match(h, p, qi, w, hq, P.slots, P.max_groups, rep, cnt, last, grp_slot, sm);
                        }
                    }
                }
            }
            __syncthreads();
            if (sm->overflow) {
                overflowed = true;
                break;
            }
            // rank this pass's groups together with the winners of earlier passes: warp qi
            if (warp < P.n_q) {
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
    __syncthreads();
    if (gave_up) {
        if (tid < kMaxNQ) sm->n_run[tid] = 0;
        if (tid == 0) atomicOr(P.status, SPEC_STATUS_GROUPS);
    }
    __syncthreads();

    // ---- mixed allocation: context rows in query order, then model rows by rank; drop duplicates
    if (warp == 0) {
        int n = 0;
        const bool dedup = (P.flags & SPEC_FLAG_DEDUP) != 0;
        const int n_model = (P.flags & SPEC_FLAG_MODEL_FILL) ? P.k_tab : 0;
        const int n_lists = P.n_q + 1;
        for (int li = 0; li < n_lists && n < P.B; ++li) {
            const bool model = (li == P.n_q);
            const int n_cand = model ? n_model : sm->n_run[li];
            for (int r = 0; r < n_cand && n < P.B; ++r) {
                int tok = -1, count = 0;
                if (model) {
                    if (!sm->chain_ok[r]) continue;
                    if (lane < w) tok = sm->chain[r][lane];
                } else {
                    const unsigned long long key = sm->run_key[li][r];
                    const int p = (int)(uint32_t)key;
                    count = (int)(key >> 32);
                    if (lane < w) tok = h[p + lane];
                }
                bool dup = false;
                if (dedup) {
                    for (int b = 0; b < n && !dup; ++b) {
                        const bool eq = (lane < w) ? (sm->out[b][lane] == tok) : true;
                        dup = __all_sync(0xffffffffu, eq);
                    }
                }
                if (dup) continue;
                if (lane < w) sm->out[n][lane] = tok;
                if (lane == 0) {
                    sm->out_src[n] = model ? 0 : P.qs[li];
                    sm->out_cnt[n] = count;
                }
                __syncwarp();
                ++n;
            }
        }
        if (lane == 0) sm->n_out = n;
    }
    __syncthreads();
    const int n = sm->n_out;
    for (int i = tid; i < P.B * w; i += nthr) {
        const int b = i / w, t = i - b * w;
        P.drafts[(size_t)s * P.B * w + i] = (b < n) ? sm->out[b][t] : -1;
    }
    for (int b = tid; b < P.B; b += nthr) {
        if (P.src) P.src[(size_t)s * P.B + b] = (b < n) ? sm->out_src[b] : -1;
        if (P.counts) P.counts[(size_t)s * P.B + b] = (b < n) ? sm->out_cnt[b] : 0;
    }
    if (tid == 0) P.ndrafts[s] = n;
}

int launch_draft(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs, int n_q,
                 int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts, int32_t* d_src,
                 int32_t* d_counts, cudaStream_t st) {
    DraftParams P;
    P.hist = d_hist;
    P.len = d_len;
    P.S = S;
    P.cap = cap;
    P.n_q = n_q;
    P.q_max = 0;
    for (int i = 0; i < kMaxNQ; ++i) {
        P.qs[i] = i < n_q ? qs[i] : 0;
        if (i < n_q && qs[i] > P.q_max) P.q_max = qs[i];
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
    int slots = 1024;
    while (slots < cap && slots < 8192) slots <<= 1;
    P.slots = slots;
    P.max_groups = slots / 2;
    const int threads = cap >= 16384 ? 1024 : (cap >= 2048 ? 256 : 128);
    const size_t smem = ((sizeof(DraftSmem) + 15) & ~size_t(15)) + (size_t)slots * 3 * sizeof(int) +
                        (size_t)P.max_groups * sizeof(int);
    static bool attr_set[64] = {false};
    bool& attr_done = attr_set[ctx->device & 63];
    if (!attr_done) {
        int rc = check_cuda(ctx, cudaFuncSetAttribute(draft_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024),
                            "draft: cudaFuncSetAttribute");
        if (rc) return rc;
        attr_done = true;
    }
    draft_kernel<<<S, threads, smem, st>>>(P);
    ctx->launches += 1;
    return check_cuda(ctx, cudaGetLastError(), "draft_context_ngrams launch");
}

}  // namespace ngs
