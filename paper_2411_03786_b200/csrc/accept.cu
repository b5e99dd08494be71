// Greedy acceptance, best-row choice and history commit: one warp per sequence.
#include "common.cuh"

namespace ngs {

// Lane l owns draft rows l and l+32.  a_b = longest prefix with drafts[b][j] == argmax[b][j]
// (argmax[b][j] is the model's greedy token after column j of the verify block, whose column
// j+1 holds drafts[b][j]).  The warp keeps the row with the longest prefix, lowest b on ties.
__global__ void __launch_bounds__(128) accept_commit_kernel(
    const int32_t* __restrict__ drafts, const int32_t* __restrict__ ndrafts, const int32_t* __restrict__ argmax,
    int S, int B, int w, int32_t* __restrict__ hist, int32_t* __restrict__ len, int cap,
    int32_t* __restrict__ acc_len, int32_t* __restrict__ best_row, int32_t* __restrict__ committed,
    int* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    grid_launch_dependents();
    grid_dependency_wait();  // drafts and predictions come from the kernels before this one
    if (s >= S) return;
    const int32_t* ds = drafts + (size_t)s * B * w;
    const int32_t* ps = argmax + (size_t)s * B * (w + 1);
    int nb = ndrafts[s];
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
    const int L = len[s];
    const bool fits = (L >= 0) && (L + a + 1 <= cap);
    int32_t tok = -1;
    if (fits && lane <= a) tok = (lane < a) ? ds[b * w + lane] : ps[b * (w + 1) + a];
    if (lane <= w) committed[(size_t)s * (w + 1) + lane] = tok;
    if (fits && lane <= a) hist[(size_t)s * cap + L + lane] = tok;
    if (lane == 0) {
        if (fits) {
            len[s] = L + a + 1;
            acc_len[s] = a;
            best_row[s] = b;
        } else {
            acc_len[s] = -1;
            best_row[s] = -1;
            atomicOr(status, SPEC_STATUS_CAPACITY);
        }
    }
}

int launch_accept(spec_ctx* ctx, const int32_t* d_drafts, const int32_t* d_ndrafts, const int32_t* d_argmax, int S,
                  int B, int w, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len, int32_t* d_best_row,
                  int32_t* d_committed, cudaStream_t st) {
    const int warps = 4;
    cudaError_t e = launch_pdl(accept_commit_kernel, dim3((S + warps - 1) / warps), dim3(warps * 32), 0, st, d_drafts, d_ndrafts,
                               d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row, d_committed, ctx->d_status);
    ctx->launches += 1;
    return check_cuda(ctx, e, "accept_and_commit launch");
}

}  // namespace ngs
