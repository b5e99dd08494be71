// Shared declarations of the N-gram speculation library (host side + small device helpers).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <mutex>
#include <utility>

#include "../../include/ngram_spec.h"

namespace ngs {

constexpr int kMaxB = 64;
constexpr int kMaxW = 16;
constexpr int kMaxQ = 4;
constexpr int kMaxNQ = 4;
constexpr int kMaxKTab = 32;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor maps of one [V, d] matrix as the B operand of the head contraction, with 256-, 128-, 64-, 32- and
// 16-row boxes: a tile of any multiple of 16 rows is fetched with one copy per set bit of its row count.
struct WMaps {
    CUtensorMap m[5];
};

}  // namespace ngs

struct spec_ctx {
    int device = 0;
    int V = 0, d = 0;
    int num_sms = 0;
    const void* embed = nullptr;    // bf16 [V, d]
    const void* unembed = nullptr;  // bf16 [V, d]
    void* owned_embed = nullptr;    // set when converted from fp32
    void* owned_unembed = nullptr;
    int* d_status = nullptr;        // device status word
    // verify merge scratch: one packed (value, ~index) key per row + completion ticket
    unsigned long long* d_keys = nullptr;
    unsigned int* d_ticket = nullptr;  // [0] CTAs finished, [1] CTAs that gave up on a bounded wait
    unsigned int* d_draft_work = nullptr;  // batch drafting: [0] next sequence to take, [1] CTAs that have left
    // table-build scratch: partial top-k lists per vocabulary chunk
    float* d_part_val = nullptr;
    int32_t* d_part_idx = nullptr;
    size_t part_capacity = 0;  // entries
    // model table remembered for drafting
    const int32_t* tab_idx = nullptr;
    int k_tab = 0;
    const int32_t* ext = nullptr;
    int w_ext = 0;
    ngs::EncodeTiledFn encode = nullptr;
    // B operand of every contraction: tensor maps of the unembedding, encoded on first use (host-side work only)
    ngs::WMaps tm_w;
    bool tm_w_ready = false;
    ngs::WMaps tm_e;  // same for the embedding (B operand of the unigram contraction)
    bool tm_e_ready = false;
    // 8-bit copy of the unembedding (E4M3 codes + one fp32 scale per row), borrowed from the caller
    const uint8_t* wq = nullptr;
    const float* wscale = nullptr;
    ngs::WMaps tm_q;
    bool tm_q_ready = false;
    bool wq_fresh = false;  // the 8-bit head was set since the last verification over it
    // tensor maps of the most recent A operands (hidden states), so a decode loop that verifies from the
    // same buffer every step does not re-encode the map on every call
    struct AMap {
        const void* base = nullptr;
        int rows = 0, box_rows = 0, elem_bytes = 0;
        CUtensorMap tm;
    } a_maps[4];
    int a_map_next = 0;
    // the incremental context index registered with this context (caller-owned memory)
    struct IndexMeta {
        void* ptr = nullptr;
        int S = 0, cap = 0, n_q = 0, w = 0, key_len = 0, slots = 0;
        int qs[4] = {0, 0, 0, 0};
    } index;
    void* d_centred = nullptr;  // unigram scratch: bf16 [V, d] output embeddings minus their mean
    float* d_colsum = nullptr;  // unigram scratch: [64 + 1, d] partial column sums and the mean
    long long launches = 0;
    char err[256] = {0};
};

namespace ngs {

// Launch with programmatic dependent launch allowed: the grid may be scheduled while the previous
// kernel of the stream is still running (once that kernel has let its dependents go, or has
// finished), and must execute griddepcontrol.wait before it touches memory the previous work
// produces.  Behaves like a plain launch after work that never lets dependents go early.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Same, for a kernel whose CTAs form thread-block clusters of `cluster_x` (distributed shared memory).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      unsigned cluster_x, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// Wait until the kernels this grid depends on have completed and their writes are visible.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allow the next kernel in the stream to be scheduled (it still waits before consuming our results).
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// Guards the process-wide host-side caches (launch shapes, per-device kernel attributes): contexts on
// different host threads may call into the library at the same time.
std::mutex& host_mutex();

int fail(spec_ctx* ctx, int code, const char* fmt, ...);
int check_cuda(spec_ctx* ctx, cudaError_t e, const char* what);
bool aligned16(const void* p);

// 2-D row-major [rows, cols] tensor map of bf16 (elem_bytes = 2) or one-byte elements, 128-byte swizzle,
// box = [box_rows, 128 bytes].
int make_tensor_map(spec_ctx* ctx, CUtensorMap* tm, const void* base, int rows, int cols, int box_rows, int elem_bytes = 2);

// The five maps of a [V, d] B operand (see WMaps).
int make_w_maps(spec_ctx* ctx, WMaps* maps, const void* base, int elem_bytes);
// Cached form of make_tensor_map for an A operand; *out stays valid until four other operands were mapped.
int a_tensor_map(spec_ctx* ctx, const CUtensorMap** out, const void* base, int rows, int cols, int box_rows, int elem_bytes = 2);

// head_gemm.cu
struct AcceptArgs;
int launch_verify(spec_ctx* ctx, const void* d_hidden, int M, int32_t* d_argmax, float* d_max, cudaStream_t st,
                  const AcceptArgs* fuse, long long* d_keys_out, int idx_offset);
int launch_verify_fp8(spec_ctx* ctx, const uint8_t* d_hq, const float* d_hscale, int M, int32_t* d_argmax, float* d_max,
                      cudaStream_t st);
int launch_quantize_rows(spec_ctx* ctx, const void* d_rows, int n_rows, uint8_t* d_codes, float* d_scale, cudaStream_t st);
int launch_unpack_keys(const long long* d_keys, int M, int V_total, int32_t* d_argmax, float* d_max, cudaStream_t st);
int launch_table(spec_ctx* ctx, const void* d_rows, int n_rows, int k_tab, int32_t* d_tab_idx, float* d_tab_val, cudaStream_t st);
int launch_extend_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, int w_ext, int32_t* d_ext, cudaStream_t st);
int launch_logits(spec_ctx* ctx, const void* d_rows, int m, float* d_logits, cudaStream_t st);
int launch_unigram(spec_ctx* ctx, int k_uni, int32_t* d_uni_idx, float* d_dist2, cudaStream_t st);
int launch_wait_probe(spec_ctx* ctx, unsigned long long limit_ns, int mark_incomplete, cudaStream_t st);
// ctx_index.cu
size_t context_index_bytes(int S, int cap, int n_q);
int launch_index_build(spec_ctx* ctx, void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs,
                       int n_q, int w, int key_len, cudaStream_t st);
int launch_accept_indexed(spec_ctx* ctx, const AcceptArgs& a, cudaStream_t st);
// draft.cu / accept.cu
int launch_draft(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs, int n_q,
                 int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts, int32_t* d_src,
                 int32_t* d_counts, cudaStream_t st);
int launch_stats(spec_ctx* ctx, const int32_t* d_acc_len, const int32_t* d_best_row, const int32_t* d_src, int S, int B,
                 int w, long long* d_stats, cudaStream_t st);
int launch_accept(spec_ctx* ctx, const int32_t* d_drafts, const int32_t* d_ndrafts, const int32_t* d_argmax, int S,
                  int B, int w, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len, int32_t* d_best_row,
                  int32_t* d_committed, cudaStream_t st);

}  // namespace ngs
