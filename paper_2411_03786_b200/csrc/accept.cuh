// Greedy acceptance of one sequence by one warp (shared by the stand-alone kernel and the fused verify).
#pragma once
#include "common.cuh"

namespace ngs {

struct AcceptArgs {
    const int32_t* drafts;   // [S, B, w]
    const int32_t* ndrafts;  // [S]
    const int32_t* argmax;   // [S, B, w + 1]
    int S, B, w;
    int32_t* hist;           // [S, cap]
    int32_t* len;            // [S]
    int cap;
    int32_t* acc_len;        // [S]
    int32_t* best_row;       // [S]
    int32_t* committed;      // [S, w + 1]
    int* status;
};

// Lane l owns draft rows l and l+32.  a_b = longest prefix with drafts[b][j] == argmax[b][j]
// (argmax[b][j] is the model's greedy token after column j of the verify block, whose column
// j+1 holds drafts[b][j]).  The warp keeps the row with the longest prefix, lowest b on ties,
// and appends that prefix plus the bonus token argmax[b][a] to the history.
__device__ __forceinline__ void accept_sequence(const AcceptArgs& q, int s, int lane) {
    const int B = q.B, w = q.w;
    const int32_t* ds = q.drafts + (size_t)s * B * w;
    const int32_t* ps = q.argmax + (size_t)s * B * (w + 1);
    int nb = q.ndrafts[s];
    nb = nb < 0 ? 0 : (nb > B ? B : nb);
    unsigned key = 0;  // (a << 8) | (255 - b): the maximum is the longest prefix, lowest row
    for (int b = lane; b < nb; b += 32) {
        int a = 0;
        while (a < w && ds[b * w + a] == ps[b * (w + 1) + a]) ++a;
        unsigned k = ((unsigned)a << 8) | (unsigned)(255 - b);
        key = k > key ? k : key;
    }
    key = __reduce_max_sync(0xffffffffu, key);
    int a = 0, b = 0;
    if (nb > 0) {
        a = (int)(key >> 8);
        b = 255 - (int)(key & 255u);
    }
    const int L = q.len[s];
    const bool fits = (L >= 0) && (L + a + 1 <= q.cap);
    int32_t tok = -1;
    if (fits && lane <= a) tok = (lane < a) ? ds[b * w + lane] : ps[b * (w + 1) + a];
    if (lane <= w) q.committed[(size_t)s * (w + 1) + lane] = tok;
    if (fits && lane <= a) q.hist[(size_t)s * q.cap + L + lane] = tok;
    if (lane == 0) {
        if (fits) {
            q.len[s] = L + a + 1;
            q.acc_len[s] = a;
            q.best_row[s] = b;
        } else {
            q.acc_len[s] = -1;
            q.best_row[s] = -1;
            atomicOr(q.status, SPEC_STATUS_CAPACITY);
        }
    }
}

}  // namespace ngs
