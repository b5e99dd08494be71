// Host side of the C ABI: context life cycle, argument checks, error strings.
#include <stdarg.h>
#include <string.h>

#include <mutex>

#include <cuda_bf16.h>

#include "accept.cuh"
#include "common.cuh"
#include "draft_common.cuh"

// Error text of calls that have no context to keep it in: one buffer per host thread.
static thread_local char g_err[256] = "";

namespace ngs {

std::mutex& host_mutex() {
    static std::mutex m;
    return m;
}

int fail(spec_ctx* ctx, int code, const char* fmt, ...) {
    char buf[256];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    strncpy(ctx ? ctx->err : g_err, buf, 255);
    return code;
}

int check_cuda(spec_ctx* ctx, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return SPEC_OK;
    return fail(ctx, SPEC_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int make_tensor_map(spec_ctx* ctx, CUtensorMap* tm, const void* base, int rows, int cols, int box_rows, int elem_bytes) {
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * (cuuint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)box_rows};  // one 128-byte swizzle row wide
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = ctx->encode(tm, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                             const_cast<void*>(base), dims, strides, box,
                             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, SPEC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return SPEC_OK;
}

int make_w_maps(spec_ctx* ctx, WMaps* maps, const void* base, int elem_bytes) {
    for (int i = 0; i < 5; ++i) {
        int rc = make_tensor_map(ctx, &maps->m[i], base, ctx->V, ctx->d, 256 >> i, elem_bytes);
        if (rc) return rc;
    }
    return SPEC_OK;
}

int a_tensor_map(spec_ctx* ctx, const CUtensorMap** out, const void* base, int rows, int cols, int box_rows, int elem_bytes) {
    for (auto& m : ctx->a_maps)
        if (m.base == base && m.rows == rows && m.box_rows == box_rows && m.elem_bytes == elem_bytes) {
            *out = &m.tm;
            return SPEC_OK;
        }
    spec_ctx::AMap& m = ctx->a_maps[ctx->a_map_next];
    ctx->a_map_next = (ctx->a_map_next + 1) % 4;
    m.base = nullptr;
    int rc = make_tensor_map(ctx, &m.tm, base, rows, cols, box_rows, elem_bytes);
    if (rc) return rc;
    m.base = base;
    m.rows = rows;
    m.box_rows = box_rows;
    m.elem_bytes = elem_bytes;
    *out = &m.tm;
    return SPEC_OK;
}

__global__ void round_f32_to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) out[i] = __float2bfloat16_rn(in[i]);
}

}  // namespace ngs

using namespace ngs;

extern "C" {

const char* spec_last_error(spec_ctx* ctx) { return ctx ? ctx->err : g_err; }

long long spec_launch_count(spec_ctx* ctx) { return ctx ? ctx->launches : 0; }

int spec_init(spec_ctx** out, const void* d_embed, const void* d_unembed, int dtype, int V, int d, int device,
              void* stream) {
    if (!out) return fail(nullptr, SPEC_ERR_ARG, "spec_init: out is NULL");
    *out = nullptr;
    if (!d_embed || !d_unembed) return fail(nullptr, SPEC_ERR_ARG, "spec_init: weight pointer is NULL");
    if (!aligned16(d_embed) || !aligned16(d_unembed))
        return fail(nullptr, SPEC_ERR_ARG, "spec_init: weight pointers must be 16-byte aligned");
    if (V <= 0 || d <= 0 || d % 8 != 0) return fail(nullptr, SPEC_ERR_ARG, "spec_init: need V > 0, d > 0, d %% 8 == 0");
    if (dtype != SPEC_F32 && dtype != SPEC_BF16) return fail(nullptr, SPEC_ERR_ARG, "spec_init: unknown dtype %d", dtype);
    int n_dev = 0;
    cudaError_t e = cudaGetDeviceCount(&n_dev);
    if (e != cudaSuccess || n_dev <= 0)
        return fail(nullptr, SPEC_ERR_CUDA, "spec_init: no CUDA device (%s); this library has no CPU path",
                    cudaGetErrorString(e));
    if (device < 0 || device >= n_dev) return fail(nullptr, SPEC_ERR_ARG, "spec_init: device %d out of range", device);
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess) return check_cuda(nullptr, e, "cudaGetDeviceProperties");
    if (prop.major != 10)
        return fail(nullptr, SPEC_ERR_CUDA, "spec_init: device %d is sm_%d%d; the kernels are built for sm_100a only",
                    device, prop.major, prop.minor);
    if ((e = cudaSetDevice(device)) != cudaSuccess) return check_cuda(nullptr, e, "cudaSetDevice");

    spec_ctx* ctx = new spec_ctx();
    ctx->device = device;
    ctx->V = V;
    ctx->d = d;
    ctx->num_sms = prop.multiProcessorCount;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = SPEC_OK;
    do {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) {
            rc = fail(nullptr, SPEC_ERR_CUDA, "spec_init: cuTensorMapEncodeTiled not available from the driver");
            break;
        }
        ctx->encode = (EncodeTiledFn)fn;
        if (dtype == SPEC_F32) {
            size_t n = (size_t)V * d;
            if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->owned_embed, n * 2), "cudaMalloc(embed)"))) break;
            if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->owned_unembed, n * 2), "cudaMalloc(unembed)"))) break;
            int blocks = ctx->num_sms * 8;
            round_f32_to_bf16_kernel<<<blocks, 256, 0, st>>>((const float*)d_embed, (__nv_bfloat16*)ctx->owned_embed, n);
            round_f32_to_bf16_kernel<<<blocks, 256, 0, st>>>((const float*)d_unembed, (__nv_bfloat16*)ctx->owned_unembed, n);
            ctx->launches += 2;
            ctx->embed = ctx->owned_embed;
            ctx->unembed = ctx->owned_unembed;
        } else {
            ctx->embed = d_embed;
            ctx->unembed = d_unembed;
        }
        if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->d_status, sizeof(int)), "cudaMalloc(status)"))) break;
        if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->d_keys, sizeof(unsigned long long) * SPEC_MAX_VERIFY_ROWS),
                             "cudaMalloc(keys)"))) break;
        if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->d_ticket, 2 * sizeof(unsigned int)), "cudaMalloc(ticket)"))) break;
        if ((rc = check_cuda(nullptr, cudaMalloc(&ctx->d_draft_work, 2 * sizeof(unsigned int)), "cudaMalloc(draft work counter)"))) break;
        cudaMemsetAsync(ctx->d_draft_work, 0, 2 * sizeof(unsigned int), st);
        cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st);
        cudaMemsetAsync(ctx->d_keys, 0, sizeof(unsigned long long) * SPEC_MAX_VERIFY_ROWS, st);
        cudaMemsetAsync(ctx->d_ticket, 0, 2 * sizeof(unsigned int), st);
        if ((rc = make_w_maps(ctx, &ctx->tm_w, ctx->unembed, 2))) {
            strncpy(g_err, ctx->err, 255);
            break;
        }
        ctx->tm_w_ready = true;
        if ((rc = check_cuda(nullptr, cudaStreamSynchronize(st), "spec_init: stream sync"))) break;
    } while (0);
    if (rc != SPEC_OK) {
        spec_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return SPEC_OK;
}

int spec_destroy(spec_ctx* ctx) {
    if (!ctx) return SPEC_OK;
    cudaSetDevice(ctx->device);
    cudaFree(ctx->owned_embed);
    cudaFree(ctx->owned_unembed);
    cudaFree(ctx->d_status);
    cudaFree(ctx->d_keys);
    cudaFree(ctx->d_ticket);
    cudaFree(ctx->d_draft_work);
    cudaFree(ctx->d_centred);
    cudaFree(ctx->d_colsum);
    cudaFree(ctx->d_part_val);
    cudaFree(ctx->d_part_idx);
    delete ctx;
    return SPEC_OK;
}

int spec_get_status(spec_ctx* ctx, int* status_bits, void* stream) {
    if (!ctx || !status_bits) return fail(ctx, SPEC_ERR_ARG, "spec_get_status: NULL argument");
    cudaStream_t st = (cudaStream_t)stream;
    int rc = check_cuda(ctx, cudaMemcpyAsync(status_bits, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st),
                        "spec_get_status: copy");
    if (rc) return rc;
    if ((rc = check_cuda(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st), "spec_get_status: clear"))) return rc;
    return check_cuda(ctx, cudaStreamSynchronize(st), "spec_get_status: sync");
}

int spec_set_model_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, const int32_t* d_ext, int w_ext) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_set_model_table: ctx is NULL");
    if (!d_tab_idx || k_tab < 1 || k_tab > kMaxKTab) return fail(ctx, SPEC_ERR_ARG, "spec_set_model_table: bad table");
    if (d_ext && (w_ext < 1 || w_ext > kMaxW)) return fail(ctx, SPEC_ERR_ARG, "spec_set_model_table: bad w_ext");
    ctx->tab_idx = d_tab_idx;
    ctx->k_tab = k_tab;
    ctx->ext = d_ext;
    ctx->w_ext = d_ext ? w_ext : 0;
    return SPEC_OK;
}

int build_model_ngram_tables(spec_ctx* ctx, const void* d_rows, int k_tab, int w_ext, int32_t* d_tab_idx,
                             float* d_tab_val, int32_t* d_ext, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "build_model_ngram_tables: ctx is NULL");
    if (!d_tab_idx) return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_tables: d_tab_idx is NULL");
    if (k_tab < 1 || k_tab > kMaxKTab || k_tab > ctx->V)
        return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_tables: k_tab must be in [1, min(%d, V)]", kMaxKTab);
    if (w_ext < 0 || w_ext > kMaxW) return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_tables: w_ext must be in [0, %d]", kMaxW);
    if ((d_ext != nullptr) != (w_ext > 0))
        return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_tables: d_ext and w_ext must be given together");
    if ((d_rows && !aligned16(d_rows)) || !aligned16(d_tab_idx))
        return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_tables: pointers must be 16-byte aligned");
    cudaSetDevice(ctx->device);
    int rc = launch_table(ctx, d_rows ? d_rows : ctx->embed, ctx->V, k_tab, d_tab_idx, d_tab_val, (cudaStream_t)stream);
    if (rc) return rc;
    if (d_ext && (rc = launch_extend_table(ctx, d_tab_idx, k_tab, w_ext, d_ext, (cudaStream_t)stream))) return rc;
    return spec_set_model_table(ctx, d_tab_idx, k_tab, d_ext, w_ext);
}

int build_model_ngram_table_rows(spec_ctx* ctx, const void* d_rows, int row_begin, int row_count, int k_tab,
                                 int32_t* d_tab_idx, float* d_tab_val, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "build_model_ngram_table_rows: ctx is NULL");
    if (!d_tab_idx) return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_table_rows: d_tab_idx is NULL");
    if (k_tab < 1 || k_tab > kMaxKTab || k_tab > ctx->V)
        return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_table_rows: k_tab must be in [1, min(%d, V)]", kMaxKTab);
    if (row_begin < 0 || row_count < 0 || (long long)row_begin + row_count > ctx->V)
        return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_table_rows: rows [%d, %d + %d) are not inside [0, V)", row_begin, row_begin, row_count);
    if (d_rows && !aligned16(d_rows)) return fail(ctx, SPEC_ERR_ARG, "build_model_ngram_table_rows: d_rows must be 16-byte aligned");
    if (row_count == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    const char* a = (const char*)(d_rows ? d_rows : ctx->embed) + (size_t)row_begin * ctx->d * 2;  // d % 8 == 0: stays 16-byte aligned
    return launch_table(ctx, a, row_count, k_tab, d_tab_idx + (size_t)row_begin * k_tab,
                        d_tab_val ? d_tab_val + (size_t)row_begin * k_tab : nullptr, (cudaStream_t)stream);
}

int spec_extend_model_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, int w_ext, int32_t* d_ext, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_extend_model_table: ctx is NULL");
    if (!d_tab_idx || !d_ext) return fail(ctx, SPEC_ERR_ARG, "spec_extend_model_table: NULL pointer");
    if (k_tab < 1 || k_tab > kMaxKTab) return fail(ctx, SPEC_ERR_ARG, "spec_extend_model_table: k_tab must be in [1, %d]", kMaxKTab);
    if (w_ext < 1 || w_ext > kMaxW) return fail(ctx, SPEC_ERR_ARG, "spec_extend_model_table: w_ext must be in [1, %d]", kMaxW);
    cudaSetDevice(ctx->device);
    int rc = launch_extend_table(ctx, d_tab_idx, k_tab, w_ext, d_ext, (cudaStream_t)stream);
    if (rc) return rc;
    return spec_set_model_table(ctx, d_tab_idx, k_tab, d_ext, w_ext);
}

int draft_context_ngrams(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap, const int* qs,
                         int n_q, int topk, int B, int w, int flags, int32_t* d_drafts, int32_t* d_ndrafts,
                         int32_t* d_src, int32_t* d_counts, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "draft_context_ngrams: ctx is NULL");
    if (!d_hist || !d_len || !d_drafts || !d_ndrafts) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: NULL pointer");
    if (!aligned16(d_hist)) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: d_hist must be 16-byte aligned");
    if (S < 0 || cap <= 0 || cap % 4 != 0 || cap >= (1 << 28))
        return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: need S >= 0, 0 < cap < 2^28, cap %% 4 == 0");
    if (B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: need 1<=B<=%d, 1<=w<=%d", kMaxB, kMaxW);
    if (n_q < 0 || n_q > kMaxNQ || (n_q > 0 && !qs)) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: need 0<=n_q<=%d", kMaxNQ);
    for (int i = 0; i < n_q; ++i)
        if (qs[i] < 1 || qs[i] > kMaxQ) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: q must be in [1, %d]", kMaxQ);
    if (topk < 1 || topk > B) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams: need 1 <= topk <= B");
    if ((flags & SPEC_FLAG_MODEL_FILL) && !ctx->tab_idx)
        return fail(ctx, SPEC_ERR_NOT_BUILT, "draft_context_ngrams: model fill needs build_model_ngram_tables first");
    if (S == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_draft(ctx, d_hist, d_len, S, cap, qs, n_q, topk, B, w, flags, d_drafts, d_ndrafts, d_src, d_counts,
                        (cudaStream_t)stream);
}

size_t spec_context_index_bytes(int S, int cap, int n_q) {
    if (S < 0 || cap <= 0 || n_q < 1 || n_q > kMaxNQ) return 0;
    return context_index_bytes(S, cap, n_q);
}

int spec_context_index_build(spec_ctx* ctx, void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap,
                             const int* qs, int n_q, int w, int flags, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_context_index_build: ctx is NULL");
    if (!d_index || !d_hist || !d_len || !qs) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: NULL pointer");
    if (!aligned16(d_index) || !aligned16(d_hist)) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: d_index and d_hist must be 16-byte aligned");
    if (S < 1 || cap <= 0 || cap % 4 != 0 || cap >= (1 << 28)) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: need S >= 1, 0 < cap < 2^28, cap %% 4 == 0");
    if (n_q < 1 || n_q > kMaxNQ || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: need 1<=n_q<=%d, 1<=w<=%d", kMaxNQ, kMaxW);
    for (int i = 0; i < n_q; ++i) {
        if (qs[i] < 1 || qs[i] > kMaxQ) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: q must be in [1, %d]", kMaxQ);
        for (int j = 0; j < i; ++j)
            if (qs[j] == qs[i]) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: query lengths must be distinct");
    }
    if (flags & ~SPEC_FLAG_KEY_NEXT_TOKEN) return fail(ctx, SPEC_ERR_ARG, "spec_context_index_build: flags may only hold SPEC_FLAG_KEY_NEXT_TOKEN");
    cudaSetDevice(ctx->device);
    return launch_index_build(ctx, d_index, d_hist, d_len, S, cap, qs, n_q, w, (flags & SPEC_FLAG_KEY_NEXT_TOKEN) ? 1 : w, (cudaStream_t)stream);
}

int draft_context_ngrams_indexed(spec_ctx* ctx, const void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap,
                                 const int* qs, int n_q, int topk, int B, int w, int flags, int32_t* d_drafts,
                                 int32_t* d_ndrafts, int32_t* d_src, int32_t* d_counts, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "draft_context_ngrams_indexed: ctx is NULL");
    if (!d_hist || !d_len || !d_drafts || !d_ndrafts) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: NULL pointer");
    if (B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: need 1<=B<=%d, 1<=w<=%d", kMaxB, kMaxW);
    if (n_q < 0 || n_q > kMaxNQ || (n_q > 0 && !qs)) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: need 0<=n_q<=%d", kMaxNQ);
    if (topk < 1 || topk > B) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: need 1 <= topk <= B");
    const spec_ctx::IndexMeta& m = ctx->index;
    if (!d_index || d_index != m.ptr) return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: d_index is not the index registered by spec_context_index_build");
    if (S != m.S || cap != m.cap || w != m.w || ((flags & SPEC_FLAG_KEY_NEXT_TOKEN) ? 1 : w) != m.key_len)
        return fail(ctx, SPEC_ERR_ARG, "draft_context_ngrams_indexed: S, cap, w and the key flag must be those the index was built with");
    if (flags & SPEC_FLAG_PARTIAL_TAIL)
        return fail(ctx, SPEC_ERR_UNSUPPORTED, "draft_context_ngrams_indexed: the index holds complete windows only (SPEC_FLAG_PARTIAL_TAIL needs draft_context_ngrams)");
    if ((flags & SPEC_FLAG_MODEL_FILL) && !ctx->tab_idx)
        return fail(ctx, SPEC_ERR_NOT_BUILT, "draft_context_ngrams_indexed: model fill needs build_model_ngram_tables first");
    cudaSetDevice(ctx->device);
    DraftParams P = make_draft_params(ctx, d_hist, d_len, S, cap, qs, n_q, topk, B, w, flags, d_drafts, d_ndrafts, d_src, d_counts);
    return launch_draft_indexed(ctx, P, (cudaStream_t)stream);
}

int accept_and_commit_indexed(spec_ctx* ctx, void* d_index, const int32_t* d_drafts, const int32_t* d_ndrafts,
                              const int32_t* d_argmax, int S, int B, int w, int32_t* d_hist, int32_t* d_len, int cap,
                              int32_t* d_acc_len, int32_t* d_best_row, int32_t* d_committed, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "accept_and_commit_indexed: ctx is NULL");
    if (!d_drafts || !d_ndrafts || !d_argmax || !d_hist || !d_len || !d_acc_len || !d_best_row || !d_committed)
        return fail(ctx, SPEC_ERR_ARG, "accept_and_commit_indexed: NULL pointer");
    if (B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "accept_and_commit_indexed: need 1<=B<=%d, 1<=w<=%d", kMaxB, kMaxW);
    const spec_ctx::IndexMeta& m = ctx->index;
    if (!d_index || d_index != m.ptr) return fail(ctx, SPEC_ERR_ARG, "accept_and_commit_indexed: d_index is not the index registered by spec_context_index_build");
    if (S != m.S || cap != m.cap || w != m.w) return fail(ctx, SPEC_ERR_ARG, "accept_and_commit_indexed: S, cap and w must be those the index was built with");
    cudaSetDevice(ctx->device);
    const AcceptArgs q{d_drafts, d_ndrafts, d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row, d_committed, ctx->d_status};
    return launch_accept_indexed(ctx, q, (cudaStream_t)stream);
}

int verify_lmhead_argmax(spec_ctx* ctx, const void* d_hidden, int M, int32_t* d_argmax, float* d_max, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax: ctx is NULL");
    if (!d_hidden || !d_argmax) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax: NULL pointer");
    if (!aligned16(d_hidden)) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax: d_hidden must be 16-byte aligned");
    if (M < 0 || M > SPEC_MAX_VERIFY_ROWS) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax: need 0 <= M <= %d", SPEC_MAX_VERIFY_ROWS);
    if (M == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_verify(ctx, d_hidden, M, d_argmax, d_max, (cudaStream_t)stream, nullptr, nullptr, 0);
}

int verify_accept_commit(spec_ctx* ctx, const void* d_hidden, const int32_t* d_drafts, const int32_t* d_ndrafts, int S, int B,
                         int w, int32_t* d_argmax, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len,
                         int32_t* d_best_row, int32_t* d_committed, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "verify_accept_commit: ctx is NULL");
    if (!d_hidden || !d_drafts || !d_ndrafts || !d_argmax || !d_hist || !d_len || !d_acc_len || !d_best_row || !d_committed)
        return fail(ctx, SPEC_ERR_ARG, "verify_accept_commit: NULL pointer");
    if (!aligned16(d_hidden)) return fail(ctx, SPEC_ERR_ARG, "verify_accept_commit: d_hidden must be 16-byte aligned");
    if (S < 0 || cap <= 0) return fail(ctx, SPEC_ERR_ARG, "verify_accept_commit: need S >= 0, cap > 0");
    if (B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "verify_accept_commit: need 1<=B<=%d, 1<=w<=%d", kMaxB, kMaxW);
    const long long M = (long long)S * B * (w + 1);
    if (M > SPEC_MAX_VERIFY_ROWS) return fail(ctx, SPEC_ERR_ARG, "verify_accept_commit: S*B*(w+1) exceeds %d rows", SPEC_MAX_VERIFY_ROWS);
    if (S == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    if (S > 256) {  // many sequences: one warp per sequence in its own kernel is the faster way to accept
        int rc = launch_verify(ctx, d_hidden, (int)M, d_argmax, nullptr, (cudaStream_t)stream, nullptr, nullptr, 0);
        if (rc) return rc;
        return launch_accept(ctx, d_drafts, d_ndrafts, d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row,
                             d_committed, (cudaStream_t)stream);
    }
    const AcceptArgs q{d_drafts, d_ndrafts, d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row, d_committed, nullptr};
    return launch_verify(ctx, d_hidden, (int)M, d_argmax, nullptr, (cudaStream_t)stream, &q, nullptr, 0);
}

int accept_and_commit(spec_ctx* ctx, const int32_t* d_drafts, const int32_t* d_ndrafts, const int32_t* d_argmax, int S,
                      int B, int w, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len, int32_t* d_best_row,
                      int32_t* d_committed, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "accept_and_commit: ctx is NULL");
    if (!d_drafts || !d_ndrafts || !d_argmax || !d_hist || !d_len || !d_acc_len || !d_best_row || !d_committed)
        return fail(ctx, SPEC_ERR_ARG, "accept_and_commit: NULL pointer");
    if (S < 0 || cap <= 0) return fail(ctx, SPEC_ERR_ARG, "accept_and_commit: need S >= 0, cap > 0");
    if (B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "accept_and_commit: need 1<=B<=%d, 1<=w<=%d", kMaxB, kMaxW);
    if (S == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_accept(ctx, d_drafts, d_ndrafts, d_argmax, S, B, w, d_hist, d_len, cap, d_acc_len, d_best_row,
                         d_committed, (cudaStream_t)stream);
}

int build_model_unigram(spec_ctx* ctx, int k_uni, int32_t* d_uni_idx, float* d_dist2, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "build_model_unigram: ctx is NULL");
    if (!d_dist2) return fail(ctx, SPEC_ERR_ARG, "build_model_unigram: d_dist2 is NULL");
    if (k_uni < 0 || k_uni > 1024 || k_uni > ctx->V || (k_uni > 0 && !d_uni_idx))
        return fail(ctx, SPEC_ERR_ARG, "build_model_unigram: need 0 <= k_uni <= min(1024, V) and d_uni_idx for k_uni > 0");
    cudaSetDevice(ctx->device);
    return launch_unigram(ctx, k_uni, d_uni_idx, d_dist2, (cudaStream_t)stream);
}

int verify_lmhead_keys(spec_ctx* ctx, const void* d_hidden, int M, int vocab_offset, long long* d_keys, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_keys: ctx is NULL");
    if (!d_hidden || !d_keys) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_keys: NULL pointer");
    if (!aligned16(d_hidden)) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_keys: d_hidden must be 16-byte aligned");
    if (M < 0 || M > SPEC_MAX_VERIFY_ROWS) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_keys: need 0 <= M <= %d", SPEC_MAX_VERIFY_ROWS);
    if (vocab_offset < 0 || (long long)vocab_offset + ctx->V > 0x7FFFFFFFll)
        return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_keys: vocab_offset + V must fit in int32");
    if (M == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_verify(ctx, d_hidden, M, nullptr, nullptr, (cudaStream_t)stream, nullptr, d_keys, vocab_offset);
}

int spec_unpack_keys(const long long* d_keys, int M, int V_total, int32_t* d_argmax, float* d_max, void* stream) {
    if (!d_keys || !d_argmax || M < 0 || V_total <= 0) return fail(nullptr, SPEC_ERR_ARG, "spec_unpack_keys: bad argument");
    if (M == 0) return SPEC_OK;
    return launch_unpack_keys(d_keys, M, V_total, d_argmax, d_max, (cudaStream_t)stream);
}

int spec_accumulate_stats(spec_ctx* ctx, const int32_t* d_acc_len, const int32_t* d_best_row, const int32_t* d_src, int S,
                          int B, int w, long long* d_stats, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_accumulate_stats: ctx is NULL");
    if (!d_acc_len || !d_best_row || !d_src || !d_stats) return fail(ctx, SPEC_ERR_ARG, "spec_accumulate_stats: NULL pointer");
    if (S < 0 || B < 1 || B > kMaxB || w < 1 || w > kMaxW) return fail(ctx, SPEC_ERR_ARG, "spec_accumulate_stats: bad sizes");
    if (S == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_stats(ctx, d_acc_len, d_best_row, d_src, S, B, w, d_stats, (cudaStream_t)stream);
}

int spec_quantize_rows_fp8(spec_ctx* ctx, const void* d_rows, int n_rows, uint8_t* d_codes, float* d_scale, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_quantize_rows_fp8: ctx is NULL");
    if (!d_rows || !d_codes || !d_scale || n_rows < 0) return fail(ctx, SPEC_ERR_ARG, "spec_quantize_rows_fp8: bad argument");
    if (!aligned16(d_rows) || !aligned16(d_codes)) return fail(ctx, SPEC_ERR_ARG, "spec_quantize_rows_fp8: matrices must be 16-byte aligned");
    if (ctx->d % 16 != 0) return fail(ctx, SPEC_ERR_UNSUPPORTED, "spec_quantize_rows_fp8: the 8-bit head needs d %% 16 == 0");
    if (n_rows == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_quantize_rows(ctx, d_rows, n_rows, d_codes, d_scale, (cudaStream_t)stream);
}

int spec_quantize_head_fp8(spec_ctx* ctx, uint8_t* d_wq, float* d_wscale, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_quantize_head_fp8: ctx is NULL");
    int rc = spec_quantize_rows_fp8(ctx, ctx->unembed, ctx->V, d_wq, d_wscale, stream);
    if (rc) return rc;
    return spec_set_head_fp8(ctx, d_wq, d_wscale);
}

int spec_set_head_fp8(spec_ctx* ctx, const uint8_t* d_wq, const float* d_wscale) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_set_head_fp8: ctx is NULL");
    if (!d_wq || !d_wscale || !aligned16(d_wq)) return fail(ctx, SPEC_ERR_ARG, "spec_set_head_fp8: NULL or misaligned pointer");
    if (ctx->d % 16 != 0) return fail(ctx, SPEC_ERR_UNSUPPORTED, "spec_set_head_fp8: the 8-bit head needs d %% 16 == 0");
    ctx->wq = d_wq;
    ctx->wscale = d_wscale;
    ctx->tm_q_ready = false;
    ctx->wq_fresh = true;
    return SPEC_OK;
}

int verify_lmhead_argmax_fp8(spec_ctx* ctx, const void* d_hidden, int M, uint8_t* d_hq, float* d_hscale, int32_t* d_argmax,
                             float* d_max, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_fp8: ctx is NULL");
    if (!d_hq || !d_hscale || !d_argmax) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax_fp8: NULL pointer");
    if ((d_hidden && !aligned16(d_hidden)) || !aligned16(d_hq))
        return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax_fp8: d_hidden and d_hq must be 16-byte aligned");
    if (M < 0 || M > SPEC_MAX_VERIFY_ROWS) return fail(ctx, SPEC_ERR_ARG, "verify_lmhead_argmax_fp8: need 0 <= M <= %d", SPEC_MAX_VERIFY_ROWS);
    if (!ctx->wq) return fail(ctx, SPEC_ERR_NOT_BUILT, "verify_lmhead_argmax_fp8: call spec_quantize_head_fp8 (or spec_set_head_fp8) first");
    if (M == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    if (d_hidden) {  // NULL: the caller's own producer already left codes and scales in d_hq / d_hscale
        int rc = launch_quantize_rows(ctx, d_hidden, M, d_hq, d_hscale, (cudaStream_t)stream);
        if (rc) return rc;
    }
    return launch_verify_fp8(ctx, d_hq, d_hscale, M, d_argmax, d_max, (cudaStream_t)stream);
}

int spec_debug_logits(spec_ctx* ctx, const void* d_rows, int m, float* d_logits, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_debug_logits: ctx is NULL");
    if (!d_rows || !d_logits || m < 0) return fail(ctx, SPEC_ERR_ARG, "spec_debug_logits: bad argument");
    if (!aligned16(d_rows)) return fail(ctx, SPEC_ERR_ARG, "spec_debug_logits: d_rows must be 16-byte aligned");
    if (m == 0) return SPEC_OK;
    cudaSetDevice(ctx->device);
    return launch_logits(ctx, d_rows, m, d_logits, (cudaStream_t)stream);
}

int spec_debug_expire_wait(spec_ctx* ctx, unsigned long long limit_ns, int mark_verify_incomplete, void* stream) {
    if (!ctx) return fail(nullptr, SPEC_ERR_ARG, "spec_debug_expire_wait: ctx is NULL");
    if (limit_ns > 1000000000ull) return fail(ctx, SPEC_ERR_ARG, "spec_debug_expire_wait: the limit may not exceed one second");
    cudaSetDevice(ctx->device);
    return launch_wait_probe(ctx, limit_ns, mark_verify_incomplete ? 1 : 0, (cudaStream_t)stream);
}

}  // extern "C"
