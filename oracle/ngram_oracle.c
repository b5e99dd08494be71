/*
 * CPU oracle for the batched N-gram speculation step ("The N-Grammys",
 * arXiv 2411.03786).  TEST INFRASTRUCTURE ONLY: plain, slow, written for a
 * reader to check against the paper by eye.  It shares no code with the CUDA
 * library and the product never calls it.  Floating point is fp64 over the
 * bf16-rounded inputs the tensor-core path also sees.
 *
 * Every routine is the definition written out; no blocking, no fusion.
 * OpenMP, where present, only spreads independent rows / sequences over cores.
 *
 * Pins (tests/test_oracle_*.py): brute force on tiny inputs, a hand-worked
 * example, closed forms (tied unit-norm weights, permutation weights),
 * library matmul/unique cross-checks and the toy-model losslessness
 * invariant; for the 8-bit head the format's closed form, a nearest-value
 * search and a library cast.  No routine here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ bf16 storage */

/* bfloat16 = the upper 16 bits of an IEEE binary32. */
static double bf16_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* binary32 -> bfloat16, round to nearest, ties to even.  The Tiny configuration
 * hands fp32 weights to a bf16 tensor-core path; both sides round once, like this. */
uint16_t oracle_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x40u); /* NaN */
    uint32_t keep = u >> 16, rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;
    return (uint16_t)keep;
}

void oracle_round_to_bf16(const float* in, uint16_t* out, long n) {
    for (long i = 0; i < n; ++i) out[i] = oracle_f32_to_bf16(in[i]);
}

/* ------------------------------------------------------------------ context N-gram (Section 4.2)
 *
 * Query = the last q tokens of the history.  Every earlier full window of q+w
 * tokens (stride 1, overlaps allowed) whose first q tokens equal the query is a
 * match; the w tokens after it are its continuation.  Each distinct continuation
 * gets count = number of matches and last = the largest window start among them.
 * Order: count descending, ties by the later occurrence (last descending).
 * Returns the number of rows written (<= topk).  rows is [topk, w].
 */
int oracle_context_draft_keyed(const int32_t* hist, int L, int q, int w, int key_len, int topk,
                               int32_t* rows, int32_t* counts, int32_t* lasts);

int oracle_context_draft(const int32_t* hist, int L, int q, int w, int topk,
                         int32_t* rows, int32_t* counts, int32_t* lasts) {
    return oracle_context_draft_keyed(hist, L, q, w, w, topk, rows, counts, lasts);
}

/* The same with matches grouped by the first key_len tokens of the continuation only (key_len = w is
 * the paper's rule; key_len = 1 counts "the tokens that follow each occurrence", one at a time).  The
 * row emitted for a group is the w tokens after its latest occurrence. */
int oracle_context_draft_keyed(const int32_t* hist, int L, int q, int w, int key_len, int topk,
                               int32_t* rows, int32_t* counts, int32_t* lasts) {
    if (q < 1 || w < 1 || topk < 1 || L < q + w) return 0;
    const int32_t* query = hist + (L - q);
    int n_windows = L - q - w + 1;
    int* g_first = (int*)malloc(sizeof(int) * (size_t)n_windows); /* a window start representing the group */
    int* g_count = (int*)malloc(sizeof(int) * (size_t)n_windows);
    int* g_last = (int*)malloc(sizeof(int) * (size_t)n_windows);
    char* g_taken = (char*)calloc((size_t)n_windows, 1);
    int n_groups = 0;
    for (int i = 0; i < n_windows; ++i) {
        int match = 1;
        for (int t = 0; t < q; ++t)
            if (hist[i + t] != query[t]) { match = 0; break; }
        if (!match) continue;
        const int32_t* c = hist + i + q;
        int g = -1;
        for (int j = 0; j < n_groups && g < 0; ++j) {
            const int32_t* cj = hist + g_first[j] + q;
            int same = 1;
            for (int t = 0; t < key_len; ++t)
                if (c[t] != cj[t]) { same = 0; break; }
            if (same) g = j;
        }
        if (g < 0) {
            g = n_groups++;
            g_first[g] = i;
            g_count[g] = 0;
            g_last[g] = i;
        }
        g_count[g] += 1;
        if (i > g_last[g]) g_last[g] = i;
    }
    int n_out = 0;
    while (n_out < topk && n_out < n_groups) {
        int best = -1;
        for (int j = 0; j < n_groups; ++j) {
            if (g_taken[j]) continue;
            if (best < 0 || g_count[j] > g_count[best] ||
                (g_count[j] == g_count[best] && g_last[j] > g_last[best]))
                best = j;
        }
        g_taken[best] = 1;
        for (int t = 0; t < w; ++t) rows[n_out * w + t] = hist[g_last[best] + q + t];
        if (counts) counts[n_out] = g_count[best];
        if (lasts) lasts[n_out] = g_last[best];
        ++n_out;
    }
    free(g_first); free(g_count); free(g_last); free(g_taken);
    return n_out;
}

/* A variant the paper does not have (its listing slides full windows only, which hides the most recent
 * repeats): occurrences of the query with fewer than w tokens after them count too.  Such an occurrence at
 * window start i has d = L - (i + q) >= 1 following tokens; its continuation is read as if the history went
 * on repeating them: c[t] = hist[i + q + (t mod d)] once i + q + t reaches L (the way an overlapping copy
 * extends itself).  For a window with w tokens after it this is the plain continuation.  Grouping, counts,
 * `last` and the order are as in oracle_context_draft_keyed, over the windows i = 0 .. L - q - 1. */
static int32_t wrapped_token(const int32_t* hist, int L, int p, int t) {
    return p + t < L ? hist[p + t] : hist[p + t % (L - p)];
}

int oracle_context_draft_partial(const int32_t* hist, int L, int q, int w, int key_len, int topk,
                                 int32_t* rows, int32_t* counts, int32_t* lasts) {
    if (q < 1 || w < 1 || topk < 1 || L < q + 1) return 0;
    const int32_t* query = hist + (L - q);
    int n_windows = L - q; /* i = 0 .. L - q - 1: at least one token follows, and the query itself is not a window */
    int* g_first = (int*)malloc(sizeof(int) * (size_t)n_windows);
    int* g_count = (int*)malloc(sizeof(int) * (size_t)n_windows);
    int* g_last = (int*)malloc(sizeof(int) * (size_t)n_windows);
    char* g_taken = (char*)calloc((size_t)n_windows, 1);
    int n_groups = 0;
    for (int i = 0; i < n_windows; ++i) {
        int match = 1;
        for (int t = 0; t < q; ++t)
            if (hist[i + t] != query[t]) { match = 0; break; }
        if (!match) continue;
        int g = -1;
        for (int j = 0; j < n_groups && g < 0; ++j) {
            int same = 1;
            for (int t = 0; t < key_len; ++t)
                if (wrapped_token(hist, L, i + q, t) != wrapped_token(hist, L, g_first[j] + q, t)) { same = 0; break; }
            if (same) g = j;
        }
        if (g < 0) {
            g = n_groups++;
            g_first[g] = i;
            g_count[g] = 0;
            g_last[g] = i;
        }
        g_count[g] += 1;
        if (i > g_last[g]) g_last[g] = i;
    }
    int n_out = 0;
    while (n_out < topk && n_out < n_groups) {
        int best = -1;
        for (int j = 0; j < n_groups; ++j) {
            if (g_taken[j]) continue;
            if (best < 0 || g_count[j] > g_count[best] ||
                (g_count[j] == g_count[best] && g_last[j] > g_last[best]))
                best = j;
        }
        g_taken[best] = 1;
        for (int t = 0; t < w; ++t) rows[n_out * w + t] = wrapped_token(hist, L, g_last[best] + q, t);
        if (counts) counts[n_out] = g_count[best];
        if (lasts) lasts[n_out] = g_last[best];
        ++n_out;
    }
    free(g_first); free(g_count); free(g_last); free(g_taken);
    return n_out;
}

/* ------------------------------------------------------------------ extended model bigram (Section 4.1, "Extensions")
 *
 * T[V, k_tab] holds, per token x, the k_tab most likely next tokens of the model
 * bigram in rank order.  The rank-r draft of width w after x starts with T[x][r]
 * and continues by the top-1 bigram: s_{j+1} = T[s_j][0].
 * ext is [V, k_tab, w].
 */
void oracle_extend_table(const int32_t* T, int V, int k_tab, int w, int32_t* ext) {
    for (int x = 0; x < V; ++x)
        for (int r = 0; r < k_tab; ++r) {
            int32_t s = T[(long)x * k_tab + r];
            for (int j = 0; j < w; ++j) {
                ext[((long)x * k_tab + r) * w + j] = s;
                s = T[(long)s * k_tab + 0];
            }
        }
}

/* ------------------------------------------------------------------ mixed strategy (Section 4.3)
 *
 * Fill the B draft rows of one sequence: context N-gram rows first, query lengths
 * in the caller's priority order, at most topk rows each; then, if asked, the
 * extended model bigram of the last token in rank order.  With dedup a row equal
 * in all w tokens to one already taken is skipped.  Unused rows are -1.
 * flags: bit0 = dedup, bit1 = model fill, bit2 = group matches by their next token only, bit3 = occurrences with fewer than w
 * following tokens count too (oracle_context_draft_partial), bits 8..15 = rows reserved for the model strategy (the
 * context strategies together take at most B minus that many rows; the paper leaves the
 * allocation between strategies open, Section 5.2).
 * src[b] = q of the strategy that produced row b, 0 for the model, -1 unused.
 */
int oracle_draft_sequence(const int32_t* hist, int L, const int* qs, int n_q, int topk, int B, int w,
                          int flags, const int32_t* T, int V, int k_tab,
                          int32_t* drafts, int32_t* src, int32_t* counts) {
    int dedup = flags & 1, model_fill = flags & 2;
    int reserve = (flags >> 8) & 0xFF;
    int ctx_cap = reserve >= B ? 0 : B - reserve;
    int n = 0;
    for (int i = 0; i < B * w; ++i) drafts[i] = -1;
    for (int b = 0; b < B; ++b) { src[b] = -1; counts[b] = 0; }
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)(topk > k_tab ? topk : k_tab) * (size_t)w);
    int32_t* cnt = (int32_t*)malloc(sizeof(int32_t) * (size_t)(topk > 0 ? topk : 1));
    for (int qi = 0; qi < n_q && n < ctx_cap; ++qi) {
        int m = (flags & 8) ? oracle_context_draft_partial(hist, L, qs[qi], w, (flags & 4) ? 1 : w, topk, cand, cnt, NULL)
                            : oracle_context_draft_keyed(hist, L, qs[qi], w, (flags & 4) ? 1 : w, topk, cand, cnt, NULL);
        for (int r = 0; r < m && n < ctx_cap; ++r) {
            int dup = 0;
            /* The paper's tokens are elements of the vocabulary by definition (Section 2).  When the
             * vocabulary size is known (V > 0), a ranked continuation that carries a token outside
             * [0, V) -- a corrupt history -- is passed over: it takes no draft row. */
            int in_range = 1;
            for (int t = 0; t < w && V > 0; ++t)
                if (cand[r * w + t] < 0 || cand[r * w + t] >= V) in_range = 0;
            if (!in_range) continue;
            if (dedup)
                for (int b = 0; b < n && !dup; ++b)
                    if (memcmp(drafts + b * w, cand + r * w, sizeof(int32_t) * (size_t)w) == 0) dup = 1;
            if (dup) continue;
            memcpy(drafts + n * w, cand + r * w, sizeof(int32_t) * (size_t)w);
            src[n] = qs[qi];
            counts[n] = cnt[r];
            ++n;
        }
    }
    if (model_fill && T && L >= 1) {
        int32_t x = hist[L - 1];
        for (int r = 0; r < k_tab && n < B; ++r) {
            int32_t s = T[(long)x * k_tab + r];
            for (int j = 0; j < w; ++j) {
                cand[j] = s;
                s = T[(long)s * k_tab + 0];
            }
            int dup = 0;
            if (dedup)
                for (int b = 0; b < n && !dup; ++b)
                    if (memcmp(drafts + b * w, cand, sizeof(int32_t) * (size_t)w) == 0) dup = 1;
            if (dup) continue;
            memcpy(drafts + n * w, cand, sizeof(int32_t) * (size_t)w);
            src[n] = 0;
            counts[n] = 0;
            ++n;
        }
    }
    free(cand); free(cnt);
    return n;
}

/* All S sequences; hist is [S, cap]. */
void oracle_draft_batch(const int32_t* hist, const int32_t* len, int S, int cap, const int* qs, int n_q,
                        int topk, int B, int w, int flags, const int32_t* T, int V, int k_tab,
                        int32_t* drafts, int32_t* n_drafts, int32_t* src, int32_t* counts) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < S; ++s)
        n_drafts[s] = oracle_draft_sequence(hist + (long)s * cap, len[s], qs, n_q, topk, B, w, flags, T, V, k_tab,
                                            drafts + (long)s * B * w, src + (long)s * B, counts + (long)s * B);
}

/* ------------------------------------------------------------------ LM head (Sections 3 and 4.1)
 *
 * z[y] = sum_t A[x, t] * W[y, t], bf16 inputs, fp64 products and sums.
 * A has its own row count; W is [V, d].  rowsel (or NULL = 0..n_rows-1) picks
 * which rows of A are evaluated, so large problems can be sampled row by row.
 */
static void logits_row(const uint16_t* a, const uint16_t* W, int V, int d, double* z) {
    for (int y = 0; y < V; ++y) {
        const uint16_t* wy = W + (long)y * d;
        double acc = 0.0;
        for (int t = 0; t < d; ++t) acc += bf16_to_double(a[t]) * bf16_to_double(wy[t]);
        z[y] = acc;
    }
}

void oracle_logits_rows(const uint16_t* A, const int64_t* rowsel, int n_rows, const uint16_t* W, int V, int d,
                        double* out /*[n_rows, V]*/) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        long x = rowsel ? (long)rowsel[r] : r;
        logits_row(A + x * d, W, V, d, out + (long)r * V);
    }
}

/* Model bigram table rows: the k largest logits of each selected row, value
 * descending, equal values by ascending token id.  idx/val are [n_rows, k]. */
void oracle_topk_rows(const uint16_t* A, const int64_t* rowsel, int n_rows, const uint16_t* W, int V, int d,
                      int k, int32_t* idx, double* val) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        long x = rowsel ? (long)rowsel[r] : r;
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
        char* used = (char*)calloc((size_t)V, 1);
        logits_row(A + x * d, W, V, d, z);
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int y = 0; y < V; ++y)
                if (!used[y] && (best < 0 || z[y] > z[best])) best = y; /* strict > keeps the lowest id */
            if (best < 0) { idx[(long)r * k + j] = -1; if (val) val[(long)r * k + j] = -INFINITY; continue; }
            used[best] = 1;
            idx[(long)r * k + j] = best;
            if (val) val[(long)r * k + j] = z[best];
        }
        free(z); free(used);
    }
}

/* Verification: the greedy next token at each selected position, lowest id on
 * exact ties, with the winning logit and the gap to the runner-up. */
void oracle_verify_rows(const uint16_t* H, const int64_t* rowsel, int n_rows, const uint16_t* W, int V, int d,
                        int32_t* argmax, double* maxval, double* gap) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        long m = rowsel ? (long)rowsel[r] : r;
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
        logits_row(H + m * d, W, V, d, z);
        int best = 0;
        for (int y = 1; y < V; ++y)
            if (z[y] > z[best]) best = y;
        double second = -INFINITY;
        for (int y = 0; y < V; ++y)
            if (y != best && z[y] > second) second = z[y];
        argmax[r] = best;
        if (maxval) maxval[r] = z[best];
        if (gap) gap[r] = z[best] - second;
        free(z);
    }
}

/* ------------------------------------------------------------------ 8-bit head (an addition: the paper only
 * remarks, in its conclusion, that N-gram speculation composes with quantisation)
 *
 * Storage format: OCP 8-bit floating point E4M3 ("FN" variant): 1 sign bit, 4 exponent bits with
 * bias 7, 3 mantissa bits; no infinities, S.1111.111 is NaN, so the largest finite value is
 * S.1111.110 = 2^8 * 1.75 = 448; exponent field 0 holds the subnormals m/8 * 2^-6.
 *
 * Quantisation of one row x[0..d) of bf16 values (all arithmetic binary32, round to nearest even):
 *   amax  = max_t |x[t]|                       (exact)
 *   scale = amax / 448      (1 when amax = 0)  (one division)
 *   code[t] = E4M3 nearest to x[t] / scale     (one division; ties to the even code; magnitudes
 *                                               above 448 saturate to 448; a zero result is stored
 *                                               as +0 whatever its sign)
 * The head then is z[m][y] = hscale[m] * wscale[y] * sum_t dec(hq[m][t]) * dec(wq[y][t]), fp64 here.
 */
double oracle_e4m3_decode(uint8_t c) {
    int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double mag;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) mag = ldexp((double)m / 8.0, -6);
    else mag = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -mag : mag;
}

/* Nearest E4M3 code of a finite binary32 value.  The 127 finite magnitudes 0x00..0x7E (mag[], from
 * the decoder) are in ascending order, so bisect for the largest one <= |y| and then choose between it
 * and its upper neighbour by exact comparison with their midpoint (all three are exact doubles). */
static void e4m3_magnitudes(double mag[0x7F]) {
    for (int c = 0; c < 0x7F; ++c) mag[c] = oracle_e4m3_decode((uint8_t)c);
}

static uint8_t e4m3_encode_with(const double mag[0x7F], float y) {
    double a = fabs((double)y);
    int lo = 0, hi = 0x7E;
    if (a >= 448.0) lo = 0x7E;
    else {
        while (hi - lo > 1) { /* invariant: mag[lo] <= a < mag[hi] */
            int mid = (lo + hi) / 2;
            if (mag[mid] <= a) lo = mid; else hi = mid;
        }
        double below = mag[lo], above = mag[lo + 1];
        double midpoint = 0.5 * (below + above);
        if (a > midpoint || (a == midpoint && (lo & 1))) lo = lo + 1;
    }
    if (lo == 0) return 0;
    return (uint8_t)(lo | (signbit(y) ? 0x80 : 0));
}

uint8_t oracle_e4m3_encode(float y) {
    double mag[0x7F];
    e4m3_magnitudes(mag);
    return e4m3_encode_with(mag, y);
}

void oracle_quantize_rows_e4m3(const uint16_t* X, long n_rows, int d, uint8_t* codes, float* scale) {
    double mag[0x7F];
    e4m3_magnitudes(mag);
#pragma omp parallel for schedule(static)
    for (long r = 0; r < n_rows; ++r) {
        const uint16_t* x = X + r * d;
        float amax = 0.0f;
        for (int t = 0; t < d; ++t) {
            float v = fabsf((float)bf16_to_double(x[t]));
            if (v > amax) amax = v;
        }
        float sc = amax > 0.0f ? amax / 448.0f : 1.0f;
        scale[r] = sc;
        for (int t = 0; t < d; ++t) {
            float v = (float)bf16_to_double(x[t]);
            codes[r * d + t] = e4m3_encode_with(mag, v / sc);
        }
    }
}

/* Verification over the quantised head: as oracle_verify_rows, on codes and scales. */
void oracle_verify_rows_q8(const uint8_t* Hq, const float* hscale, const int64_t* rowsel, int n_rows, const uint8_t* Wq,
                           const float* wscale, int V, int d, int32_t* argmax, double* maxval, double* gap) {
    double dec[256];
    for (int c = 0; c < 256; ++c) dec[c] = oracle_e4m3_decode((uint8_t)c);
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        long m = rowsel ? (long)rowsel[r] : r;
        const uint8_t* h = Hq + m * d;
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
        for (int y = 0; y < V; ++y) {
            const uint8_t* wy = Wq + (long)y * d;
            double acc = 0.0;
            for (int t = 0; t < d; ++t) acc += dec[h[t]] * dec[wy[t]];
            z[y] = (double)hscale[m] * (double)wscale[y] * acc;
        }
        int best = 0;
        for (int y = 1; y < V; ++y)
            if (z[y] > z[best]) best = y;
        double second = -INFINITY;
        for (int y = 0; y < V; ++y)
            if (y != best && z[y] > second) second = z[y];
        argmax[r] = best;
        if (maxval) maxval[r] = z[best];
        if (gap) gap[r] = z[best] - second;
        free(z);
    }
}

/* ------------------------------------------------------------------ model unigram (Section 4.1, "Unigram")
 *
 * d(x) = || u_x - ubar ||_V where u_x is row x of the output embedding W, ubar the mean row, and the
 * norm comes from <a, b>_V = sum_y (a . v_y)(b . v_y) over the rows v_y of the input embedding E.
 * So d(x)^2 = sum_y ((u_x - ubar) . v_y)^2; p(x) is proportional to exp(-d(x)): the top-k unigram
 * tokens are those with the smallest d (equal values by ascending token id).
 * The centred rows are rounded once to bfloat16 (they feed a bf16 tensor-core contraction), everything
 * else is fp64.  rowsel (or NULL) picks the rows x that are evaluated; dist2 is [n_rows].
 */
void oracle_unigram_dist2(const uint16_t* W, const uint16_t* E, int V, int d, const int64_t* rowsel, int n_rows,
                          double* dist2) {
    double* mean = (double*)calloc((size_t)d, sizeof(double));
    for (int x = 0; x < V; ++x)
        for (int t = 0; t < d; ++t) mean[t] += bf16_to_double(W[(long)x * d + t]);
    for (int t = 0; t < d; ++t) mean[t] /= (double)V;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        long x = rowsel ? (long)rowsel[r] : r;
        double* c = (double*)malloc(sizeof(double) * (size_t)d);
        for (int t = 0; t < d; ++t)
            c[t] = bf16_to_double(oracle_f32_to_bf16((float)(bf16_to_double(W[x * d + t]) - mean[t])));
        double acc = 0.0;
        for (int y = 0; y < V; ++y) {
            double dot = 0.0;
            for (int t = 0; t < d; ++t) dot += c[t] * bf16_to_double(E[(long)y * d + t]);
            acc += dot * dot;
        }
        dist2[r] = acc;
        free(c);
    }
    free(mean);
}

/* The k tokens with the smallest distance, ascending; equal distances by ascending token id. */
void oracle_smallest_k(const double* dist2, int V, int k, int32_t* idx) {
    char* used = (char*)calloc((size_t)V, 1);
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int x = 0; x < V; ++x)
            if (!used[x] && (best < 0 || dist2[x] < dist2[best])) best = x;
        idx[j] = best;
        if (best >= 0) used[best] = 1;
    }
    free(used);
}

/* ------------------------------------------------------------------ greedy acceptance (Sections 1, 5 and Appendix D)
 *
 * Row b of the verify block is [x_L, s_1 .. s_w]; P[b][j] is the model's greedy
 * token after column j.  a_b = the longest prefix with s_{j+1} == P[b][j].  The row
 * with the longest accepted prefix wins (lowest b on ties); its a tokens and the
 * bonus token P[b*][a] are appended to the history: a+1 tokens per call.
 * A sequence whose history cannot take a+1 more tokens commits nothing and
 * reports acc_len = best_row = -1.  With no drafts, row 0 / a = 0 is used.
 * drafts [S,B,w], P [S,B,w+1], hist [S,cap], committed [S,w+1] padded with -1.
 */
void oracle_accept_commit(const int32_t* drafts, const int32_t* n_drafts, const int32_t* P, int S, int B, int w,
                          int32_t* hist, int32_t* len, int cap,
                          int32_t* acc_len, int32_t* best_row, int32_t* committed) {
#pragma omp parallel for schedule(static)
    for (int s = 0; s < S; ++s) {
        const int32_t* ds = drafts + (long)s * B * w;
        const int32_t* ps = P + (long)s * B * (w + 1);
        int nb = n_drafts[s];
        int best_b = 0, best_a = 0;
        for (int b = 0; b < nb; ++b) {
            int a = 0;
            while (a < w && ds[b * w + a] == ps[b * (w + 1) + a]) ++a;
            if (a > best_a) { best_a = a; best_b = b; }
        }
        for (int j = 0; j <= w; ++j) committed[(long)s * (w + 1) + j] = -1;
        int L = len[s];
        if (L + best_a + 1 > cap) {
            acc_len[s] = -1;
            best_row[s] = -1;
            continue;
        }
        for (int j = 0; j < best_a; ++j) committed[(long)s * (w + 1) + j] = ds[best_b * w + j];
        committed[(long)s * (w + 1) + best_a] = ps[best_b * (w + 1) + best_a];
        for (int j = 0; j <= best_a; ++j) hist[(long)s * cap + L + j] = committed[(long)s * (w + 1) + j];
        len[s] = L + best_a + 1;
        acc_len[s] = best_a;
        best_row[s] = best_b;
    }
}

/* ------------------------------------------------------------------ ablation counters (Section 5.2)
 *
 * Running histograms over decode steps, as in the paper's ablation: accepted length (0..w), row index
 * of the accepted draft among the B rows (counted when something was accepted), strategy of that row
 * (q, 0 = model), and rows allocated per strategy.  stats layout: [w+1] [B] [5] [5] int64.
 */
void oracle_accumulate_stats(const int32_t* acc_len, const int32_t* best_row, const int32_t* src, int S, int B, int w,
                             long long* stats) {
    long long* h_acc = stats;
    long long* h_row = stats + (w + 1);
    long long* h_src = h_row + B;
    long long* h_alloc = h_src + 5;
    for (int s = 0; s < S; ++s) {
        for (int b = 0; b < B; ++b) {
            int q = src[(long)s * B + b];
            if (q >= 0 && q <= 4) h_alloc[q] += 1;
        }
        int a = acc_len[s];
        if (a < 0) continue; /* the sequence could not commit */
        h_acc[a > w ? w : a] += 1;
        if (a > 0) {
            int b = best_row[s];
            h_row[b] += 1;
            int q = src[(long)s * B + b];
            if (q >= 0 && q <= 4) h_src[q] += 1;
        }
    }
}
