// Greedy acceptance, best-row choice and history commit: one warp per sequence.
#include "accept.cuh"

namespace ngs {

__global__ void __launch_bounds__(128) accept_commit_kernel(const AcceptArgs q) {
    const int lane = threadIdx.x & 31;
    const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    grid_launch_dependents();
    grid_dependency_wait();  // drafts and predictions come from the kernels before this one
    if (s >= q.S) return;
    accept_sequence(q, s, lane);
}

// Running histograms for the paper's ablation (Section 5.2): accepted length, accepted row index,
// strategy of the accepted row, rows allocated per strategy.  stats = [w+1] [B] [5] [5] int64.
__global__ void accumulate_stats_kernel(const int32_t* __restrict__ acc_len, const int32_t* __restrict__ best_row,
                                        const int32_t* __restrict__ src, int S, int B, int w,
                                        unsigned long long* __restrict__ stats) {
    grid_dependency_wait();
    unsigned long long* h_acc = stats;
    unsigned long long* h_row = stats + (w + 1);
    unsigned long long* h_src = h_row + B;
    unsigned long long* h_alloc = h_src + 5;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < S * B) {
        const int q = src[i];
        if (q >= 0 && q <= 4) atomicAdd(&h_alloc[q], 1ull);
    }
    if (i < S) {
        const int a = acc_len[i];
        if (a >= 0) {
            atomicAdd(&h_acc[a > w ? w : a], 1ull);
            if (a > 0) {
                const int b = best_row[i];
                if (b >= 0 && b < B) {
                    atomicAdd(&h_row[b], 1ull);
                    const int q = src[(size_t)i * B + b];
                    if (q >= 0 && q <= 4) atomicAdd(&h_src[q], 1ull);
                }
            }
        }
    }
}

int launch_stats(spec_ctx* ctx, const int32_t* d_acc_len, const int32_t* d_best_row, const int32_t* d_src, int S, int B,
                 int w, long long* d_stats, cudaStream_t st) {
    const int n = S * B;
    cudaError_t e = launch_pdl(accumulate_stats_kernel, dim3((n + 255) / 256), dim3(256), 0, st, d_acc_len, d_best_row, d_src,
                               S, B, w, reinterpret_cast<unsigned long long*>(d_stats));
    ctx->launches += 1;
    return check_cuda(ctx, e, "spec_accumulate_stats launch");
}

int launch_accept(spec_ctx* ctx, const int32_t* d_drafts, const int32_t* d_ndrafts, const int32_t* d_argmax, int S,
                  int B, int w, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len, int32_t* d_best_row,
                  int32_t* d_committed, cudaStream_t st) {
    const int warps = 4;
    const AcceptArgs q{d_drafts, d_ndrafts, d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row, d_committed, ctx->d_status};
    cudaError_t e = launch_pdl(accept_commit_kernel, dim3((S + warps - 1) / warps), dim3(warps * 32), 0, st, q);
    ctx->launches += 1;
    return check_cuda(ctx, e, "accept_and_commit launch");
}

}  // namespace ngs
