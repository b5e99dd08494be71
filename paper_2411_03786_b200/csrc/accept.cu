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
