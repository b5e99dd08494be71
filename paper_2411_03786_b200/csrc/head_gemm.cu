// LM-head contraction Z = A * W^T on the 5th-generation tensor cores (tcgen05, accumulators in
// TMEM, operands staged by TMA) with the row reduction fused into the epilogue, so Z never
// reaches memory:
//   MODE_ARGMAX  verification: per row of A the arg max over the vocabulary   (verify_lmhead_argmax)
//   MODE_TOPK    model bigram table: per row the k largest entries           (build_model_ngram_tables)
//   MODE_STORE   plain fp32 store, for the logits tolerance check            (spec_debug_logits)
//   MODE_SUMSQ   model unigram: per row the sum of squares over all columns  (build_model_unigram)
//   MODE_ARGMAX_Q8  verification over the 8-bit (E4M3) copy of the head          (verify_lmhead_argmax_fp8)
//
// A is [a_rows, d] and W is [V, d], both bf16 and K-major, so both operands use the same
// 128-byte-swizzled K-major shared-memory layout.  (The 8-bit mode reads one-byte elements: a
// 128-byte swizzle row then holds 128 of them and one MMA covers K = 32, so every size counted in
// bytes below is the same for both element types.)  One CTA owns the accumulator of a
// 128 x (<=256) tile: TMEM lane = row of A, TMEM column = vocabulary entry.  An epilogue thread
// therefore owns one row of A and walks its columns in ascending vocabulary order, which makes
// "lowest token id wins ties" a matter of using a strict comparison.
//
// Work is cut into units (m_tile, vocabulary chunk), numbered so that consecutive units are the m-tiles
// of one m-group on the same chunk, and dealt out round-robin over the CTAs: the CTAs at work at any
// moment walk the same few chunks of W together, so W comes from HBM once per m-group, and every SM
// has work until the last round.  Inside a unit the CTA
// sweeps the chunk in tiles of up to 256 columns and keeps the running
// reduction in registers, then flushes once: a 64-bit atomicMax of (value, ~index) for the arg
// max, a partial list for the top-k.  Small M (memory-bound: every SM streams its own slice of
// W exactly once) and large M (tensor-bound) are the same kernel with different unit shapes.
//
// Warp roles (192 threads): warp 0 = TMA producer (+ TMEM allocation), warp 1 = MMA issuer,
// warps 2..5 = epilogue (TMEM lane quadrant = warp % 4).  Every wait on an mbarrier is bounded:
// on expiry the CTA raises SPEC_STATUS_TIMEOUT, stops issuing work, and still frees its TMEM.
#include <cuda_bf16.h>
#include <math.h>
#include <stdlib.h>

#include <algorithm>
#include <map>
#include <tuple>

#include "accept.cuh"
#include "common.cuh"

namespace ngs {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;               // 64 bf16 = one 128-byte swizzle row
constexpr int BLOCK_K_Q8 = 128;           // 128 one-byte elements = one 128-byte swizzle row
constexpr int TILE_N = 256;               // up to 256 columns (rows of W) per tile, in boxes of 16..256 rows
constexpr int MAX_STAGES = 8;
constexpr int A_TILE_BYTES = BLOCK_M * BLOCK_K * 2;     // 16 KB: what one MMA reads of A
constexpr int SMEM_LIMIT = 227 * 1024;                  // dynamic shared memory per CTA on sm_100
constexpr int SMEM_MISC = 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int ACC_COLS = 256;                           // TMEM columns per accumulator stage
constexpr int TMEM_COLS = 512;
constexpr int GEMM_THREADS = 192;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // default limit of every device-side wait

enum { MODE_ARGMAX = 0, MODE_TOPK = 1, MODE_STORE = 2, MODE_SUMSQ = 3, MODE_ARGMAX_Q8 = 4 };

struct GemmParams {
    int a_rows;    // rows of A
    int V;         // rows of W
    int num_kb;    // k-blocks of one swizzle row: ceil(d / 64) for bf16, ceil(d / 128) for one-byte elements
    int n_mtiles;  // ceil(a_rows / 128)
    int box_n;     // rows of W per TMA box (16, 32, 64, 128 or 256)
    int n_boxes;   // ceil(V / box_n)
    int n_chunks;  // vocabulary chunks per m-tile
    int group;     // m-tiles that run side by side on the same W chunk (L2 reuse)
    int n_groups;  // ceil(n_mtiles / group)
    int n_slots;   // slot order: grid = group * n_slots; 0 = round-robin order (see UnitIter)
    int a_box_rows;   // rows of A per TMA box (128, or fewer when A has fewer rows)
    int a2_rows;      // dual: rows of the second m-tile's TMA box (its own tensor map)
    int a_bytes;      // shared-memory bytes reserved for the A tile of a stage (multiple of 1024)
    int stage_bytes;  // a_bytes + boxes per tile * box bytes
    int pad_bytes;    // unused bytes after the last stage (keeps the MMA's 128-row A window in bounds)
    int stages;       // depth of the operand ring
    int dual;         // 1: A has two m-tiles and every CTA computes both against its W slice (argmax only)
    int tile2_m64;    // dual, and the second m-tile has at most 64 rows: it is computed with M = 64 instructions
    unsigned long long* keys;
    unsigned int* ticket;
    int32_t* argmax;
    float* maxv;
    int k_tab;
    float* part_val;   // [n_chunks, a_rows, k_tab]
    int32_t* part_idx;
    float* logits;     // [a_rows, V]
    int* status;
    int fuse_accept;   // argmax mode: the CTA that merges the keys also accepts and commits
    AcceptArgs acc;
    long long* keys_out;  // argmax mode, vocabulary shard: export (value, id) keys instead of ids
    int idx_offset;       // first token id of this shard
    const float* col_scale;  // 8-bit mode: scale of each row of W (= column of the product)
    const float* row_scale;  // 8-bit mode: scale of each row of A (only the reported maximum needs it)
    unsigned long long wait_limit_ns;  // every mbarrier wait gives up after this long
    int prefetch_w;          // 1: the W tiles of the first ring fill are requested before the dependency wait
};

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, one K = 16 slice.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same for E4M3 inputs (kind::f8f6f4), one K = 32 slice.
__device__ __forceinline__ void tc_mma_e4m3(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// One fp32 column of this thread's TMEM lane (the column is the same for the whole warp).
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr) {
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
    return r;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 B apart, 8-row
// groups 1024 B apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t saddr) {
    uint64_t desc = 0;
    desc |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    desc |= (uint64_t)1 << 16;                     // leading byte offset (unused for swizzled K-major)
    desc |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset
    desc |= (uint64_t)1 << 46;                     // descriptor version
    desc |= (uint64_t)2 << 61;                     // SWIZZLE_128B
    return desc;
}
// Instruction descriptor for kind::f16: D = fp32, A = B = bf16, both K-major, M = 128, N given.
__device__ __forceinline__ uint32_t make_idesc_bf16(int n_cols) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
}

// Instruction descriptor for kind::f8f6f4: D = fp32, A = B = E4M3 (format code 0), both K-major.
__device__ __forceinline__ uint32_t make_idesc_e4m3(int n_cols) {
    return (1u << 4) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
}

// Order-preserving map of fp32 onto unsigned integers; key 0 lies below every real value.
__device__ __forceinline__ uint32_t orderable_f32(float v) {
    uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable_f32(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// Arg max of 32 consecutive columns as a tree of independent comparisons (depth 5 instead of a chain
// of 32 dependent ones: this runs at the very end of a memory-bound launch, where nothing hides it).
// A right-hand (higher) column wins only if strictly larger, so equal values keep the lowest column.
// Returns the winning value and its offset in [0, 32).
__device__ __forceinline__ void chunk_argmax(const float (&v)[32], float& best, int& off) {
    float a16[16];
    int i16[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const bool hi = v[2 * j + 1] > v[2 * j];
        a16[j] = hi ? v[2 * j + 1] : v[2 * j];
        i16[j] = 2 * j + (hi ? 1 : 0);
    }
#pragma unroll
    for (int n = 8; n >= 1; n >>= 1) {
#pragma unroll
        for (int j = 0; j < n; ++j) {
            const bool hi = a16[2 * j + 1] > a16[2 * j];
            a16[j] = hi ? a16[2 * j + 1] : a16[2 * j];
            i16[j] = hi ? i16[2 * j + 1] : i16[2 * j];
        }
    }
    best = a16[0];
    off = i16[0];
}

// ------------------------------------------------------------------------------------------ work units
struct Unit {
    int m_tile, chunk, box_begin, box_end;
};
// Units of this CTA in execution order.  Two orders:
//  - slots (chunks that cost a partial result per row and are therefore few and long - top-k lists, sums of
//    squares): the grid is group x n_slots CTAs, CTA b works on m-tile b % group of each m-group and on chunks
//    b / group, + n_slots, ...; the CTAs of one slot start a chunk together and walk its tiles in step, so W
//    comes from HBM once per m-group;
//  - round-robin (n_slots = 0; the arg max, whose chunks are single tiles): the launch's units are numbered
//    m-group by m-group, inside a group chunk by chunk, inside a chunk m-tile by m-tile, and CTA b takes units
//    b, b + grid, b + 2 grid, ...  Units cost the same, so every SM is busy until the last round whatever
//    the numbers of m-tiles and chunks, and the CTAs at work at any moment hold consecutive units - the
//    m-tiles of a group on the same few tiles of W.
struct UnitIter {
    long long u;          // round-robin: the next unit
    int mg, c, mi, slot;  // slots: m-group, chunk, m-tile in the group, slot
    __device__ __forceinline__ explicit UnitIter(const GemmParams& p)
        : u((long long)blockIdx.x), mg(0), c((int)blockIdx.x / p.group), mi((int)blockIdx.x % p.group), slot((int)blockIdx.x / p.group) {}
    __device__ __forceinline__ bool next(const GemmParams& p, Unit& un) {
        if (p.n_slots == 0) {
            if (u >= (long long)p.n_chunks * p.n_mtiles) return false;
            const long long per_group = (long long)p.n_chunks * p.group;  // units of a full m-group (only the last can be ragged)
            const int g = (int)(u / per_group);
            const int r = (int)(u - (long long)g * per_group);
            const int gm = min(p.group, p.n_mtiles - g * p.group);  // m-tiles of this group
            const int cc = r / gm;
            un.m_tile = g * p.group + (r - cc * gm);
            un.chunk = cc;
            un.box_begin = (int)((long long)cc * p.n_boxes / p.n_chunks);
            un.box_end = (int)((long long)(cc + 1) * p.n_boxes / p.n_chunks);
            u += (long long)gridDim.x;
            return true;
        }
        while (mg < p.n_groups) {
            const int m_tile = mg * p.group + mi;
            if (m_tile < p.n_mtiles && c < p.n_chunks) {
                un.m_tile = m_tile;
                un.chunk = c;
                un.box_begin = (int)((long long)c * p.n_boxes / p.n_chunks);
                un.box_end = (int)((long long)(c + 1) * p.n_boxes / p.n_chunks);
                c += p.n_slots;
                return true;
            }
            ++mg;
            c = slot;
        }
        return false;
    }
};

// The producer's view of the same order, one k-block at a time.
struct KbCursor {
    UnitIter it;
    Unit un;
    int b0, nb, kb;
    bool valid;
    __device__ __forceinline__ KbCursor(const GemmParams& p, int max_boxes) : it(p), b0(0), nb(0), kb(0), valid(false) {
        next_unit(p, max_boxes);
    }
    __device__ __forceinline__ void next_unit(const GemmParams& p, int max_boxes) {
        do {
            valid = it.next(p, un);
        } while (valid && un.box_begin >= un.box_end);
        if (valid) {
            b0 = un.box_begin;
            nb = min(max_boxes, un.box_end - b0);
            kb = 0;
        }
    }
    __device__ __forceinline__ void advance(const GemmParams& p, int max_boxes) {
        if (++kb < p.num_kb) return;
        kb = 0;
        b0 += max_boxes;
        if (b0 < un.box_end) {
            nb = min(max_boxes, un.box_end - b0);
            return;
        }
        next_unit(p, max_boxes);
    }
};

// ------------------------------------------------------------------------------------------ the kernel
// KT = capacity of the per-thread top-k list (registers); only MODE_TOPK uses it.
template <int MODE, int KT>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
head_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
                 const __grid_constant__ WMaps tmB, const GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;               // operand stages, 1024-byte aligned
    unsigned char* tiles_ptr = smem_raw + (tiles - raw);
    const int STAGES = p.stages, STAGE_BYTES = p.stage_bytes, A_BYTES = p.a_bytes;
    const int BOX_N = p.box_n, MAX_BOXES = TILE_N / p.box_n;
    // The MMA always reads a 128-row A tile; when fewer rows are loaded the rest of that window is
    // whatever follows in shared memory (rows that no output uses), so keep the window in bounds.
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + STAGES * STAGE_BYTES + p.pad_bytes);
    // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * MAX_STAGES;
    const uint32_t bar_tfull = bar_empty + 8 * MAX_STAGES;
    const uint32_t bar_tempty = bar_tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* is_last = reinterpret_cast<int*>(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool Q8 = MODE == MODE_ARGMAX_Q8;
    constexpr bool IS_ARGMAX = MODE == MODE_ARGMAX || MODE == MODE_ARGMAX_Q8;
    constexpr int KB_ELEMS = Q8 ? BLOCK_K_Q8 : BLOCK_K;  // elements of one k-block (the TMA x step)

    if (warp == 0 && lane < 6)  // the descriptors' first use would otherwise pay their fetch on the critical path
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(lane < 5 ? &tmB.m[lane] : &tmA)) : "memory");
    if (IS_ARGMAX && p.dual && warp == 0 && lane == 6) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA2)) : "memory");
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 4);
        }
        *abort_flag = 0;
        *is_last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // The whole warp walks the k-blocks in step; lanes 0..4 issue the W tile as one copy per set bit of
        // its row count (256, 128, 64, 32, 16 rows) and lanes 30 / 31 the A tiles, so the copies of a stage
        // are issued side by side instead of one after the other.
        {
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            const bool dual = IS_ARGMAX && p.dual;
            const uint32_t a_box_bytes = (uint32_t)(p.a_box_rows + (dual ? p.a2_rows : 0)) * 128u;
            const int my_rows = 256 >> lane;  // lanes 0..4: the piece size this lane copies
            // piece of `rows` (a multiple of 16, at most 256) for this lane: the rows above it come first
            auto w_piece = [&](uint32_t sa, int kb, int b0, int nb, uint32_t full) {
                const int rows = nb * BOX_N;
                if (lane < 5 && (rows & my_rows)) {
                    const int before = rows & ~(2 * my_rows - 1);
                    tma_load_2d(sa + A_BYTES + before * 128, &tmB.m[lane], kb * KB_ELEMS, b0 * BOX_N + before, full);
                }
            };
            // W is a constant of the model: fill the ring with its tiles before waiting for the kernel
            // that produces the activations, then add the A tiles of those stages.  (Not when W itself was
            // written by work that may still be running: the host then clears prefetch_w for this launch.)
            int n_pref = 0;
            for (KbCursor pre(p, MAX_BOXES); p.prefetch_w && n_pref < STAGES && pre.valid; pre.advance(p, MAX_BOXES), ++n_pref) {
                const uint32_t full = bar_full + 8 * n_pref;
                const uint32_t sa = tiles + n_pref * STAGE_BYTES;
                if (lane == 0) mbar_expect_tx(full, a_box_bytes + (uint32_t)(pre.nb * BOX_N * 128));
                __syncwarp();
                w_piece(sa, pre.kb, pre.b0, pre.nb, full);
            }
            grid_dependency_wait();
            for (KbCursor cur(p, MAX_BOXES); cur.valid; cur.advance(p, MAX_BOXES)) {
                const uint32_t full = bar_full + 8 * stage;
                const uint32_t sa = tiles + stage * STAGE_BYTES;
                if (issued >= n_pref) {
                    const bool got = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.wait_limit_ns);
                    if (!__all_sync(0xffffffffu, got)) {
                        ok = false;
                        break;
                    }
                    if (lane == 0) mbar_expect_tx(full, a_box_bytes + (uint32_t)(cur.nb * BOX_N * 128));
                    __syncwarp();
                    w_piece(sa, cur.kb, cur.b0, cur.nb, full);
                }
                if (lane == 31) tma_load_2d(sa, &tmA, cur.kb * KB_ELEMS, cur.un.m_tile * BLOCK_M, full);
                if (dual && lane == 30) tma_load_2d(sa + A_TILE_BYTES, &tmA2, cur.kb * KB_ELEMS, BLOCK_M, full);  // second m-tile
                ++issued;
                if (++stage == STAGES) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (!ok && lane == 0) {
                // Aborting: give copies already in flight a bounded chance to land before the CTA exits.
                const int pending = issued < STAGES ? (int)issued : STAGES;
                for (int i = 1; i <= pending; ++i) {
                    int s2 = stage - i;
                    uint32_t ph = phase;
                    if (s2 < 0) {
                        s2 += STAGES;
                        ph ^= 1u;
                    }
                    for (int it = 0; it < 100000; ++it)
                        if (mbar_try_wait(bar_full + 8 * s2, ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t tile = 0;
            bool ok = true;
            UnitIter it(p);
            Unit un;
            while (ok && it.next(p, un)) {
                for (int b0 = un.box_begin; b0 < un.box_end && ok; b0 += MAX_BOXES, ++tile) {
                    const int nb = min(MAX_BOXES, un.box_end - b0);
                    // dual: the tile takes both accumulator stages (one per m-tile), so tiles do not overlap
                    const bool dual = IS_ARGMAX && p.dual;
                    const uint32_t as = dual ? 0u : (tile & 1u), aphase = dual ? (tile & 1u) : ((tile >> 1) & 1u);
                    if (!mbar_wait(bar_tempty + 8 * as, aphase ^ 1u, abort_flag, p.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t idesc = Q8 ? make_idesc_e4m3(nb * BOX_N) : make_idesc_bf16(nb * BOX_N);
                    const uint32_t d_tmem = tmem_base + as * ACC_COLS;
                    for (int kb = 0; kb < p.num_kb; ++kb) {
                        if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.wait_limit_ns)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t sa = tiles + stage * STAGE_BYTES;
                        const uint64_t adesc = make_kmajor_sw128_desc(sa);
                        const uint64_t bdesc = make_kmajor_sw128_desc(sa + A_BYTES);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {  // four slices of 32 bytes (2 x 16 B) per swizzle row
                            if (Q8) tc_mma_e4m3(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                            else tc_mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                        if (dual) {  // the same W tile against the second m-tile, into the other accumulator
                            const uint64_t adesc2 = make_kmajor_sw128_desc(sa + A_TILE_BYTES);
                            // a second tile of at most 64 rows takes the M = 64 form: half the tensor work
                            const uint32_t idesc2 = p.tile2_m64 ? ((idesc & ~(0x1Fu << 24)) | ((uint32_t)(64 >> 4) << 24)) : idesc;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                if (Q8) tc_mma_e4m3(d_tmem + ACC_COLS, adesc2 + 2 * k, bdesc + 2 * k, idesc2, (kb | k) != 0 ? 1u : 0u);
                                else tc_mma_bf16(d_tmem + ACC_COLS, adesc2 + 2 * k, bdesc + 2 * k, idesc2, (kb | k) != 0 ? 1u : 0u);
                            }
                        }
                        tc_commit(bar_empty + 8 * stage);  // frees the stage once these MMAs have read it
                        if (++stage == STAGES) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (ok) tc_commit(bar_tfull + 8 * as);  // accumulator complete
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (4 warps)
        const int quad = warp & 3;
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t tile = 0;
        bool ok = true;
        grid_dependency_wait();  // the outputs and the merge scratch may still be in use by the previous kernel
        UnitIter it(p);
        Unit un;
        while (ok && it.next(p, un)) {
            const int row = un.m_tile * BLOCK_M + row_in_tile;
            // running reduction of this row over the unit's columns
            float best_v = MODE == MODE_SUMSQ ? 0.0f : -INFINITY;
            int best_i = 0x7FFFFFFF;
            const bool dual = IS_ARGMAX && p.dual;
            float best_v2 = -INFINITY;  // dual: the row of the second m-tile on this lane
            int best_i2 = 0x7FFFFFFF;
            // Sorted list, value descending, statically indexed so it stays in registers.  The k_tab live
            // entries sit at the bottom [KT - k_tab, KT); the slots above hold +inf, which nothing beats,
            // so the running threshold is always the last slot.
            float tv[KT];
            int ti[KT];
            const int k_off = KT - p.k_tab;
#pragma unroll
            for (int j = 0; j < KT; ++j) {
                tv[j] = j < k_off ? INFINITY : -INFINITY;
                ti[j] = 0x7FFFFFFF;
            }
            for (int b0 = un.box_begin; b0 < un.box_end && ok; b0 += MAX_BOXES, ++tile) {
                const int nb = min(MAX_BOXES, un.box_end - b0);
                const uint32_t as = dual ? 0u : (tile & 1u), aphase = dual ? (tile & 1u) : ((tile >> 1) & 1u);
                const int col0 = b0 * BOX_N;
                const int n_valid = min(nb * BOX_N, p.V - col0);
                // 8-bit mode: fetch the column scales of the whole tile while the tile is still being
                // computed (lane l keeps the scale of column 32 c + l for each of the eight 32-column chunks)
                float sc[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
                if (Q8) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) sc[c] = (c * 32 + lane < n_valid) ? p.col_scale[col0 + c * 32 + lane] : 0.0f;
                }
                if (!mbar_wait(bar_tfull + 8 * as, aphase, abort_flag, p.wait_limit_ns)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (IS_ARGMAX) {
                    // (the chunk loop stays rolled: it runs once per tile, and a short loop body that is
                    // fetched once beats eight copies that are each fetched cold)
                    auto sweep = [&](uint32_t acc_col, float& bv, int& bi) {
                        for (int c = 0; c * 32 < n_valid; ++c) {
                            uint32_t r[32];
                            float v[32];
                            float my_scale = sc[0];  // sc[c] by selection: keeps sc[] in registers
                            if (Q8) {
#pragma unroll
                                for (int k = 1; k < 8; ++k) my_scale = (c == k) ? sc[k] : my_scale;
                            }
                            __syncwarp();
                            tmem_ld32(lane_base + acc_col + c * 32, r);
                            tmem_wait_ld();
                            const int lim = n_valid - c * 32;  // >= 1
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                v[j] = __uint_as_float(r[j]);
                                if (Q8) v[j] *= __shfl_sync(0xffffffffu, my_scale, j);
                            }
                            if (lim < 32) {  // ragged end of the vocabulary
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = j < lim ? v[j] : -INFINITY;
                            }
                            float cv;
                            int co;
                            chunk_argmax(v, cv, co);
                            if (cv > bv) {  // earlier chunks hold lower token ids: strict
                                bv = cv;
                                bi = col0 + c * 32 + co;
                            }
                        }
                    };
                    sweep(as * ACC_COLS, best_v, best_i);
                    if (dual) sweep(ACC_COLS, best_v2, best_i2);
                }
                for (int c = 0; !IS_ARGMAX && c * 32 < n_valid; ++c) {
                    uint32_t r[32];
                    __syncwarp();
                    tmem_ld32(lane_base + as * ACC_COLS + c * 32, r);
                    tmem_wait_ld();
                    const int cbase = col0 + c * 32;
                    const int lim = n_valid - c * 32;  // >= 1
                    if (MODE == MODE_TOPK) {
                        // Almost every chunk holds nothing that beats a row's current k-th value: one maximum over the
                        // 32 columns and one vote decide that.  Otherwise the columns that some row wants are fetched
                        // again one at a time (a column address is common to the warp) and offered to every row's list;
                        // the insertion code then exists once, not once per column - 32 copies of it do not fit the
                        // instruction cache for long lists (k_tab = 10 built in 130 ms instead of 107 ms with 8).
                        float cmax = -INFINITY;
#pragma unroll
                        for (int j = 0; j < 32; ++j) cmax = fmaxf(cmax, j < lim ? __uint_as_float(r[j]) : -INFINITY);
                        if (__any_sync(0xffffffffu, cmax > tv[KT - 1])) {
                            unsigned want = 0;
#pragma unroll
                            for (int j = 0; j < 32; ++j) want |= (j < lim && __uint_as_float(r[j]) > tv[KT - 1]) ? (1u << j) : 0u;
                            unsigned cols = __reduce_or_sync(0xffffffffu, want);
                            while (cols) {  // ascending columns: equal values keep the lower token id ahead
                                const int j = __ffs(cols) - 1;
                                cols &= cols - 1;
                                const float v = __uint_as_float(tmem_ld1(lane_base + as * ACC_COLS + c * 32 + j));
                                tmem_wait_ld();
                                if (v > tv[KT - 1]) {
                                    // branch-free insertion from the bottom up: slot q takes its upper
                                    // neighbour if v also beats that one, else v itself; strict compares
                                    // keep earlier (lower) token ids ahead of equal values
                                    const int c_id = cbase + j;
#pragma unroll
                                    for (int q = KT - 1; q > 0; --q) {
                                        const bool up = v > tv[q - 1];
                                        const bool wr = v > tv[q];
                                        const float nv = up ? tv[q - 1] : v;
                                        const int ni = up ? ti[q - 1] : c_id;
                                        tv[q] = wr ? nv : tv[q];
                                        ti[q] = wr ? ni : ti[q];
                                    }
                                    if (v > tv[0]) {
                                        tv[0] = v;
                                        ti[0] = c_id;
                                    }
                                }
                            }
                        }
                    } else if (MODE == MODE_SUMSQ) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float v = __uint_as_float(r[j]);
                            if (j < lim) best_v += v * v;  // best_v doubles as the running sum (starts at 0)
                        }
                    } else {
                        if (row < p.a_rows) {
                            float* out = p.logits + (size_t)row * p.V + cbase;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (j < lim) out[j] = __uint_as_float(r[j]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * as);
            }
            if (!ok) break;
            if (dual) {
                // An M = 64 accumulator keeps row i in TMEM lane 32 (i / 16) + i % 16 (measured): the lower 16
                // lanes of each epilogue warp hold rows, the upper 16 nothing.
                const int row2 = BLOCK_M + (p.tile2_m64 ? quad * 16 + lane : row_in_tile);
                if (row2 < p.a_rows && (!p.tile2_m64 || lane < 16)) {
                    const unsigned long long key =
                        ((unsigned long long)orderable_f32(best_v2) << 32) | (unsigned long long)(~(uint32_t)best_i2);
                    atomicMax(p.keys + row2, key);
                }
            }
            if (row < p.a_rows) {
                if (IS_ARGMAX) {
                    const unsigned long long key =
                        ((unsigned long long)orderable_f32(best_v) << 32) | (unsigned long long)(~(uint32_t)best_i);
                    atomicMax(p.keys + row, key);
                } else if (MODE == MODE_SUMSQ) {
                    p.part_val[(size_t)un.chunk * p.a_rows + row] = best_v;
                } else if (MODE == MODE_TOPK) {
                    const size_t base = ((size_t)un.chunk * p.a_rows + row) * p.k_tab;
#pragma unroll
                    for (int j = 0; j < KT; ++j)
                        if (j >= k_off) {
                            p.part_val[base + j - k_off] = tv[j];
                            p.part_idx[base + j - k_off] = ti[j];
                        }
                }
            }
        }
        if (IS_ARGMAX) {
            // The CTA that finishes last turns the merged keys into the outputs and re-arms the scratch.
            // A CTA that gave up on a wait says so in the word after the ticket before it takes its
            // ticket, so the last CTA knows that the merged keys are incomplete.
            const int et = threadIdx.x - 64;
            __threadfence();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (et == 0) {
                if (*abort_flag) {
                    atomicAdd(p.ticket + 1, 1u);
                    atomicOr(p.status, SPEC_STATUS_TIMEOUT);
                    __threadfence();
                }
                const unsigned int t = atomicAdd(p.ticket, 1u);
                int last = (t == gridDim.x - 1) ? 1 : 0;
                if (last) {  // every other CTA has published by now: 2 = some CTA gave up
                    __threadfence();
                    if (*((volatile unsigned int*)(p.ticket + 1)) != 0u) last = 2;
                }
                *is_last = last;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*is_last) {
                __threadfence();
                const bool incomplete = *is_last == 2;
                for (int i = et; i < p.a_rows; i += 128) {
                    const unsigned long long key = atomicExch(p.keys + i, 0ull);
                    int idx = (int)(~(uint32_t)(key & 0xFFFFFFFFull));
                    if (idx < 0 || idx >= p.V) idx = 0;
                    if (incomplete) {  // some slice of the vocabulary is missing: no row may pass for a result
                        if (p.keys_out) p.keys_out[i] = (long long)0x8000000000000000ull;  // below every real key
                        else {
                            p.argmax[i] = -1;
                            if (p.maxv) p.maxv[i] = -INFINITY;
                        }
                        continue;
                    }
                    if (p.keys_out) {
                        // shard of the vocabulary: global token id, and the sign bit flipped so that the key
                        // orders correctly as a signed 64-bit integer (what a max all-reduce compares)
                        const unsigned long long g = (key & 0xFFFFFFFF00000000ull) | (unsigned long long)(~(uint32_t)(idx + p.idx_offset));
                        p.keys_out[i] = (long long)(g ^ 0x8000000000000000ull);
                        continue;
                    }
                    p.argmax[i] = idx;
                    if (p.maxv) p.maxv[i] = from_orderable_f32((uint32_t)(key >> 32)) * (Q8 ? p.row_scale[i] : 1.0f);
                }
                if (et == 0) {
                    p.ticket[0] = 0u;
                    p.ticket[1] = 0u;
                }
                if (p.fuse_accept && !incomplete) {
                    // the predictions are complete: greedy acceptance right here saves a kernel launch
                    __threadfence();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    for (int sq = et >> 5; sq < p.acc.S; sq += 4) accept_sequence(p.acc, sq, lane);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, SPEC_STATUS_TIMEOUT);
    if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ------------------------------------------------------------------------------------------ table merge / extension
// One thread per token x: merge the per-chunk partial lists (value descending, then token id
// ascending) into the final k_tab entries.
__global__ void merge_topk_kernel(const float* __restrict__ part_val, const int32_t* __restrict__ part_idx, int n_chunks,
                                  int rows, int k, int32_t* __restrict__ tab_idx, float* __restrict__ tab_val) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= rows) return;
    float tv[kMaxKTab];
    int ti[kMaxKTab];
    for (int j = 0; j < k; ++j) {
        tv[j] = -INFINITY;
        ti[j] = 0x7FFFFFFF;
    }
    for (int c = 0; c < n_chunks; ++c) {
        const size_t base = ((size_t)c * rows + x) * k;
        for (int j = 0; j < k; ++j) {
            const float v = part_val[base + j];
            const int i = part_idx[base + j];
            if (i == 0x7FFFFFFF) break;
            if (v > tv[k - 1] || (v == tv[k - 1] && i < ti[k - 1])) {
                int pos = k - 1;
                while (pos > 0 && (v > tv[pos - 1] || (v == tv[pos - 1] && i < ti[pos - 1]))) {
                    tv[pos] = tv[pos - 1];
                    ti[pos] = ti[pos - 1];
                    --pos;
                }
                tv[pos] = v;
                ti[pos] = i;
            } else {
                break;  // a chunk's list is sorted: nothing further in it can enter
            }
        }
    }
    for (int j = 0; j < k; ++j) {
        tab_idx[(size_t)x * k + j] = ti[j] == 0x7FFFFFFF ? 0 : ti[j];
        if (tab_val) tab_val[(size_t)x * k + j] = tv[j];
    }
}

// ext[x][r][0] = T[x][r]; ext[x][r][j+1] = T[ext[x][r][j]][0].
__global__ void extend_table_kernel(const int32_t* __restrict__ tab, int V, int k, int w, int32_t* __restrict__ ext) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)V * k) return;
    int s = tab[i];
    for (int j = 0; j < w; ++j) {
        ext[i * w + j] = s;
        s = (s >= 0 && s < V) ? tab[(size_t)s * k] : 0;
    }
}

// ------------------------------------------------------------------------------------------ host: unit shapes
struct Shape {
    int box_n, box_idx, group, n_groups, n_slots, n_chunks, grid;
    int a_box_rows, a2_rows, a_bytes, stage_bytes, pad_bytes, stages, smem, dual;
};

// Derives the shared-memory geometry from (box_n, group, n_chunks, grid).
static void finish_shape(Shape& sh, int a_rows, int V) {
    const int n_mtiles = (a_rows + BLOCK_M - 1) / BLOCK_M;
    sh.box_idx = sh.box_n == 16 ? 0 : sh.box_n == 32 ? 1 : sh.box_n == 64 ? 2 : sh.box_n == 128 ? 3 : 4;
    sh.n_groups = sh.dual ? 1 : (n_mtiles + sh.group - 1) / sh.group;
    const int n_boxes = (V + sh.box_n - 1) / sh.box_n;
    const int chunk_max = (n_boxes + sh.n_chunks - 1) / sh.n_chunks;
    const int nb_max = std::min(TILE_N / sh.box_n, chunk_max);
    sh.a_box_rows = n_mtiles == 1 ? std::min(BLOCK_M, (a_rows + 7) / 8 * 8) : BLOCK_M;
    // dual: the second m-tile is loaded only as tall as it is (a smaller stage means a deeper ring)
    sh.a2_rows = sh.dual ? std::min(BLOCK_M, (a_rows - BLOCK_M + 7) / 8 * 8) : 0;
    const int a_last_bytes = ((sh.dual ? sh.a2_rows : sh.a_box_rows) * 128 + 1023) / 1024 * 1024;
    sh.a_bytes = sh.dual ? A_TILE_BYTES + a_last_bytes : a_last_bytes;
    sh.stage_bytes = sh.a_bytes + (nb_max * sh.box_n * BLOCK_K * 2 + 1023) / 1024 * 1024;
    const int pad = A_TILE_BYTES - a_last_bytes;  // the MMA's 128-row window over the last A tile stays in bounds
    sh.stages = std::min(MAX_STAGES, (SMEM_LIMIT - SMEM_MISC - pad) / sh.stage_bytes);
    sh.pad_bytes = pad;
    sh.smem = sh.stages * sh.stage_bytes + pad + SMEM_MISC;
}

// Unit shapes.  `box_n` is the granularity in which the vocabulary is cut into chunks and tiles (a
// tile is then copied in power-of-two pieces, see the producer).  One m-tile (memory-bound): every
// SM streams its own slice of W once, cut to 32 rows so slices balance to within 32 rows.  Several
// m-tiles (tensor-bound): `group` m-tiles share each W chunk and tiles are whole 256-row blocks (one
// copy per k-block).  (Measured on B200, V=32000, d=4096, when a tile was still copied box by box:
// 32-row boxes 0.9, 64-row 1.1, 256-row 1.2 PFLOP/s; groups of 8..16 beat groups of 2..4 by 10-20%.)
// `tile_chunks`: a chunk is a single tile (the arg max is merged per row with one atomic per unit, so
// units may be as small as a tile and the round-robin then balances to within one tile); otherwise a chunk
// costs a partial result per row (top-k lists, sums of squares) and there are about #SMs / group of them.
static Shape choose_shape(int a_rows, int V, int sms, size_t max_chunks, bool allow_dual, bool tile_chunks) {
    const int n_mtiles = (a_rows + BLOCK_M - 1) / BLOCK_M;
    Shape sh{};
    if (n_mtiles == 1 || (n_mtiles == 2 && allow_dual)) {
        // (two m-tiles: still one pass over W, every CTA computes both tiles against its slice)
        sh.dual = n_mtiles == 2 ? 1 : 0;
        sh.box_n = 32;
        sh.group = 1;
        sh.n_chunks = (int)std::min<size_t>((size_t)std::min(sms, (V + 31) / 32), max_chunks);
        sh.grid = sh.n_chunks;
    } else {
        if (tile_chunks) {
            // round-robin order: neither the group nor the number of chunks has to divide the number of SMs;
            // larger groups re-stream W less often
            // (measured, V = 128256, 22 m-tiles: groups of 8 / 11 / 16 / 22 run at 1249 / 1268 / 1286 / 1290 TFLOP/s;
            // V = 32000, 72 m-tiles: groups of 16 / 24 / 36 / 72 at 1267 / 1310 / 1326 / 1206 - beyond some thirty
            // m-tiles the hidden states of a group and the tiles of W in flight no longer share the L2)
            const int n_groups = (n_mtiles + 31) / 32;
            sh.group = (n_mtiles + n_groups - 1) / n_groups;
            sh.box_n = 256;
            while (sh.box_n > 32 && (long long)((V + sh.box_n - 1) / sh.box_n) * n_mtiles < sms) sh.box_n >>= 1;
            const int n_boxes = (V + sh.box_n - 1) / sh.box_n;
            const int tiles = (int)(((long long)n_boxes * sh.box_n + TILE_N - 1) / TILE_N);  // one tile per chunk
            sh.n_chunks = (int)std::min<size_t>((size_t)std::min(tiles, n_boxes), max_chunks);
            sh.grid = (int)std::min<long long>((long long)sms, (long long)sh.n_chunks * n_mtiles);
            sh.n_slots = 0;
        } else {
            // slot order: the group (up to 16 m-tiles) that keeps most SMs busy, counting a ragged last m-group;
            // larger groups re-stream W less often
            double best = -1.0;
            for (int g = std::min(16, n_mtiles); g >= 1; --g) {
                const int slots = sms / g, groups = (n_mtiles + g - 1) / g;
                const double busy = (double)n_mtiles / (groups * g) * (double)(slots * g) / sms * (1.0 - 0.02 * (16 - g));
                if (busy > best + 1e-9) {
                    best = busy;
                    sh.group = g;
                }
            }
            const int slots = sms / sh.group;
            // 256-row boxes need one TMA issue per k-block and measured faster than better balanced chunks
            // of smaller boxes; fall back to smaller boxes only when the vocabulary is too small to give
            // every slot a chunk
            sh.box_n = 256;
            while (sh.box_n > 32 && (V + sh.box_n - 1) / sh.box_n < slots) sh.box_n >>= 1;
            const int n_boxes = (V + sh.box_n - 1) / sh.box_n;
            sh.n_chunks = (int)std::min<size_t>((size_t)std::min(slots, n_boxes), max_chunks);
            sh.n_slots = std::min(slots, sh.n_chunks);
            sh.grid = sh.group * sh.n_slots;
        }
    }
    finish_shape(sh, a_rows, V);
    return sh;
}

static Shape cached_shape(spec_ctx* ctx, int a_rows, size_t max_chunks, bool allow_dual = false, bool tile_chunks = false) {
#ifdef NGRAM_SPEC_TUNING
    // Tuning builds only: NGRAM_SPEC_SHAPE="box,group,chunks" overrides the choice (values are clamped).
    if (const char* ov = getenv("NGRAM_SPEC_SHAPE")) {
        int box = 32, g = 1, c = 1;
        if (sscanf(ov, "%d,%d,%d", &box, &g, &c) == 3 && (box == 16 || box == 32 || box == 64 || box == 128 || box == 256)) {
            const int n_mtiles = (a_rows + BLOCK_M - 1) / BLOCK_M;
            Shape s{};
            s.box_n = box;
            s.group = std::max(1, std::min(std::min(g, n_mtiles), ctx->num_sms));
            const int n_boxes = (ctx->V + box - 1) / box;
            s.n_chunks = (int)std::max<size_t>(1, std::min<size_t>(std::min<size_t>((size_t)std::max(c, 1), (size_t)n_boxes), max_chunks));
            s.grid = (int)std::min<long long>((long long)ctx->num_sms, (long long)s.n_chunks * (s.dual ? 1 : n_mtiles));
            finish_shape(s, a_rows, ctx->V);
            return s;
        }
    }
#endif
    // Process-wide table of the shapes chosen so far.
    const auto key = std::make_tuple(a_rows, ctx->V, ctx->d, ctx->num_sms, max_chunks, allow_dual, tile_chunks);
    std::lock_guard<std::mutex> lock(host_mutex());
    static std::map<std::tuple<int, int, int, int, size_t, bool, bool>, Shape> cache;
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    Shape s = choose_shape(a_rows, ctx->V, ctx->num_sms, max_chunks, allow_dual, tile_chunks);
    cache[key] = s;
#ifdef NGRAM_SPEC_TUNING
    if (getenv("NGRAM_SPEC_TRACE"))
        fprintf(stderr, "[ngram_spec] rows=%d V=%d d=%d: dual=%d box=%d group=%d groups=%d chunks=%d grid=%d a_box=%d stages=%d stage=%dB smem=%dB\n",
                a_rows, ctx->V, ctx->d, s.dual, s.box_n, s.group, s.n_groups, s.n_chunks, s.grid, s.a_box_rows, s.stages, s.stage_bytes, s.smem);
#endif
    return s;
}

// Tensor maps of the unembedding (or, for the unigram, the embedding), encoded once per context.
static int w_map(spec_ctx* ctx, const WMaps** out, bool embedding = false) {
    WMaps* maps = embedding ? &ctx->tm_e : &ctx->tm_w;
    bool& ready = embedding ? ctx->tm_e_ready : ctx->tm_w_ready;
    if (!ready) {
        int rc = make_w_maps(ctx, maps, embedding ? ctx->embed : ctx->unembed, 2);
        if (rc) return rc;
        ready = true;
    }
    *out = maps;
    return SPEC_OK;
}

template <int MODE, int KT>
static int set_smem_attr(spec_ctx* ctx) {
    static bool done[64] = {false};
    std::lock_guard<std::mutex> lock(host_mutex());
    bool& d = done[ctx->device & 63];
    if (d) return SPEC_OK;
    int rc = check_cuda(ctx, cudaFuncSetAttribute(head_gemm_kernel<MODE, KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT),
                        "head gemm: cudaFuncSetAttribute");
    if (rc == SPEC_OK) d = true;
    return rc;
}

static void fill_common(spec_ctx* ctx, GemmParams& p, int a_rows, const Shape& sh) {
    p.a_rows = a_rows;
    p.V = ctx->V;
    p.num_kb = (ctx->d + BLOCK_K - 1) / BLOCK_K;
    p.n_mtiles = sh.dual ? 1 : (a_rows + BLOCK_M - 1) / BLOCK_M;  // dual: one unit covers both m-tiles
    p.dual = sh.dual;
    p.tile2_m64 = (sh.dual && a_rows - BLOCK_M <= 64) ? 1 : 0;
    p.box_n = sh.box_n;
    p.n_boxes = (ctx->V + sh.box_n - 1) / sh.box_n;
    p.n_chunks = sh.n_chunks;
    p.group = sh.group;
    p.n_groups = sh.n_groups;
    p.n_slots = sh.n_slots;
    p.a_box_rows = sh.a_box_rows;
    p.a2_rows = sh.a2_rows;
    p.a_bytes = sh.a_bytes;
    p.stage_bytes = sh.stage_bytes;
    p.pad_bytes = sh.pad_bytes;
    p.stages = sh.stages;
    p.keys = ctx->d_keys;
    p.ticket = ctx->d_ticket;
    p.argmax = nullptr;
    p.maxv = nullptr;
    p.k_tab = 0;
    p.part_val = nullptr;
    p.part_idx = nullptr;
    p.logits = nullptr;
    p.status = ctx->d_status;
    p.fuse_accept = 0;
    p.acc = AcceptArgs{};
    p.keys_out = nullptr;
    p.idx_offset = 0;
    p.col_scale = nullptr;
    p.row_scale = nullptr;
    p.wait_limit_ns = WAIT_LIMIT_NS;
    p.prefetch_w = 1;
}

int launch_verify(spec_ctx* ctx, const void* d_hidden, int M, int32_t* d_argmax, float* d_max, cudaStream_t st,
                  const AcceptArgs* fuse, long long* d_keys_out, int idx_offset) {
    int rc = set_smem_attr<MODE_ARGMAX, 1>(ctx);
    if (rc) return rc;
    const Shape sh = cached_shape(ctx, M, (size_t)1 << 20, true, true);
    const WMaps* tmW;
    if ((rc = w_map(ctx, &tmW))) return rc;
    const CUtensorMap* tmA;
    if ((rc = a_tensor_map(ctx, &tmA, d_hidden, M, ctx->d, sh.a_box_rows))) return rc;
    const CUtensorMap* tmA2 = tmA;  // second m-tile of the two-tile pass: same matrix, a box only as tall as that tile
    if (sh.dual && (rc = a_tensor_map(ctx, &tmA2, d_hidden, M, ctx->d, sh.a2_rows))) return rc;
    GemmParams p;
    fill_common(ctx, p, M, sh);
    p.argmax = d_argmax;
    p.maxv = d_max;
    if (fuse) {
        p.fuse_accept = 1;
        p.acc = *fuse;
        p.acc.status = ctx->d_status;
    }
    p.keys_out = d_keys_out;
    p.idx_offset = idx_offset;
    cudaError_t e = launch_pdl(head_gemm_kernel<MODE_ARGMAX, 1>, dim3(sh.grid), dim3(GEMM_THREADS), (size_t)sh.smem, st, *tmA, *tmA2, *tmW, p);
    ctx->launches += 1;
    return check_cuda(ctx, e, "verify_lmhead_argmax launch");
}

// ------------------------------------------------------------------------------------------ 8-bit head
// Per-row quantisation of a bf16 matrix to E4M3 (all arithmetic fp32, round to nearest even):
//   amax = max |x|, scale = amax / 448 (1 for an all-zero row), code = e4m3(x / scale), zero stored as +0.
// One CTA per row; a thread handles 8 consecutive elements at a time.
__device__ __forceinline__ uint32_t e4m3_pair(float lo, float hi) {
    uint16_t r;  // cvt packs {hi, lo}: the first source lands in the upper byte
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    uint32_t v = r;
    if ((v & 0x007Fu) == 0u) v &= 0xFF00u;  // -0 -> +0
    if ((v & 0x7F00u) == 0u) v &= 0x00FFu;
    return v;
}

__global__ void __launch_bounds__(256) quantize_rows_e4m3_kernel(const __nv_bfloat16* __restrict__ X, int d,
                                                                 uint8_t* __restrict__ codes, float* __restrict__ scale) {
    __shared__ float warp_max[8];
    grid_dependency_wait();
    grid_launch_dependents();
    const size_t row = blockIdx.x;
    const uint4* x8 = reinterpret_cast<const uint4*>(X + row * d);  // 8 bf16 per load; d % 16 == 0
    const int n8 = d / 8;
    float amax = 0.0f;
    for (int i = threadIdx.x; i < n8; i += blockDim.x) {
        const uint4 v = x8[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            amax = fmaxf(amax, fabsf(__uint_as_float(w[j] << 16)));
            amax = fmaxf(amax, fabsf(__uint_as_float(w[j] & 0xFFFF0000u)));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = warp_max[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) amax = fmaxf(amax, warp_max[j]);
    const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
    if (threadIdx.x == 0) scale[row] = sc;
    uint2* out = reinterpret_cast<uint2*>(codes + row * d);
    for (int i = threadIdx.x; i < n8; i += blockDim.x) {
        const uint4 v = x8[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t pair[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            pair[j] = e4m3_pair(__fdiv_rn(__uint_as_float(w[j] << 16), sc), __fdiv_rn(__uint_as_float(w[j] & 0xFFFF0000u), sc));
        out[i] = make_uint2(pair[0] | (pair[1] << 16), pair[2] | (pair[3] << 16));
    }
}

int launch_quantize_rows(spec_ctx* ctx, const void* d_rows, int n_rows, uint8_t* d_codes, float* d_scale, cudaStream_t st) {
    cudaError_t e = launch_pdl(quantize_rows_e4m3_kernel, dim3(n_rows), dim3(256), 0, st, (const __nv_bfloat16*)d_rows, ctx->d,
                               d_codes, d_scale);
    ctx->launches += 1;
    return check_cuda(ctx, e, "8-bit quantisation launch");
}

int launch_verify_fp8(spec_ctx* ctx, const uint8_t* d_hq, const float* d_hscale, int M, int32_t* d_argmax, float* d_max,
                      cudaStream_t st) {
    int rc = set_smem_attr<MODE_ARGMAX_Q8, 1>(ctx);
    if (rc) return rc;
    const Shape sh = cached_shape(ctx, M, (size_t)1 << 20, true, true);
    if (!ctx->tm_q_ready) {
        if ((rc = make_w_maps(ctx, &ctx->tm_q, ctx->wq, 1))) return rc;
        ctx->tm_q_ready = true;
    }
    const CUtensorMap* tmA;
    if ((rc = a_tensor_map(ctx, &tmA, d_hq, M, ctx->d, sh.a_box_rows, 1))) return rc;
    const CUtensorMap* tmA2 = tmA;
    if (sh.dual && (rc = a_tensor_map(ctx, &tmA2, d_hq, M, ctx->d, sh.a2_rows, 1))) return rc;
    GemmParams p;
    fill_common(ctx, p, M, sh);
    p.num_kb = (ctx->d + BLOCK_K_Q8 - 1) / BLOCK_K_Q8;
    p.argmax = d_argmax;
    p.maxv = d_max;
    p.col_scale = ctx->wscale;
    p.row_scale = d_hscale;
    // The 8-bit head may have been written by a kernel of this stream that is still running (it lets its
    // dependents start early): the first verification after a head was set reads W only after the wait.
    p.prefetch_w = ctx->wq_fresh ? 0 : 1;
    ctx->wq_fresh = false;
    cudaError_t e = launch_pdl(head_gemm_kernel<MODE_ARGMAX_Q8, 1>, dim3(sh.grid), dim3(GEMM_THREADS), (size_t)sh.smem, st, *tmA, *tmA2,
                               ctx->tm_q, p);
    ctx->launches += 1;
    return check_cuda(ctx, e, "verify_lmhead_argmax_fp8 launch");
}

int launch_logits(spec_ctx* ctx, const void* d_rows, int m, float* d_logits, cudaStream_t st) {
    int rc = set_smem_attr<MODE_STORE, 1>(ctx);
    if (rc) return rc;
    const Shape sh = cached_shape(ctx, m, (size_t)1 << 20, false, true);
    const WMaps* tmW;
    if ((rc = w_map(ctx, &tmW))) return rc;
    CUtensorMap tmA;
    if ((rc = make_tensor_map(ctx, &tmA, d_rows, m, ctx->d, sh.a_box_rows))) return rc;
    GemmParams p;
    fill_common(ctx, p, m, sh);
    p.logits = d_logits;
    head_gemm_kernel<MODE_STORE, 1><<<sh.grid, GEMM_THREADS, sh.smem, st>>>(tmA, tmA, *tmW, p);
    ctx->launches += 1;
    return check_cuda(ctx, cudaGetLastError(), "spec_debug_logits launch");
}

// Table rows for the n_rows rows of A that start at d_rows (the whole matrix, or one rank's slice of it).
int launch_table(spec_ctx* ctx, const void* d_rows, int n_rows, int k_tab, int32_t* d_tab_idx, float* d_tab_val, cudaStream_t st) {
    const int kt = k_tab <= 8 ? 8 : (k_tab <= 16 ? 16 : 32);
    int rc = kt == 8 ? set_smem_attr<MODE_TOPK, 8>(ctx) : (kt == 16 ? set_smem_attr<MODE_TOPK, 16>(ctx) : set_smem_attr<MODE_TOPK, 32>(ctx));
    if (rc) return rc;
    // partial lists cost 8 bytes per entry and chunk: keep them under 256 MB
    int max_chunks = (int)std::max<long long>(1, (256ll << 20) / ((long long)n_rows * k_tab * 8));
    const Shape sh = cached_shape(ctx, n_rows, (size_t)max_chunks);
    const WMaps* tmW;
    if ((rc = w_map(ctx, &tmW))) return rc;
    CUtensorMap tmA;
    if ((rc = make_tensor_map(ctx, &tmA, d_rows, n_rows, ctx->d, sh.a_box_rows))) return rc;
    const size_t need = (size_t)sh.n_chunks * n_rows * k_tab;
    if (need > ctx->part_capacity) {
        cudaStreamSynchronize(st);
        cudaFree(ctx->d_part_val);
        cudaFree(ctx->d_part_idx);
        ctx->d_part_val = nullptr;
        ctx->d_part_idx = nullptr;
        ctx->part_capacity = 0;
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_part_val, need * sizeof(float)), "cudaMalloc(partial values)"))) return rc;
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_part_idx, need * sizeof(int32_t)), "cudaMalloc(partial ids)"))) return rc;
        ctx->part_capacity = need;
    }
    GemmParams p;
    fill_common(ctx, p, n_rows, sh);
    p.k_tab = k_tab;
    p.part_val = ctx->d_part_val;
    p.part_idx = ctx->d_part_idx;
    if (kt == 8)
        head_gemm_kernel<MODE_TOPK, 8><<<sh.grid, GEMM_THREADS, sh.smem, st>>>(tmA, tmA, *tmW, p);
    else if (kt == 16)
        head_gemm_kernel<MODE_TOPK, 16><<<sh.grid, GEMM_THREADS, sh.smem, st>>>(tmA, tmA, *tmW, p);
    else
        head_gemm_kernel<MODE_TOPK, 32><<<sh.grid, GEMM_THREADS, sh.smem, st>>>(tmA, tmA, *tmW, p);
    if ((rc = check_cuda(ctx, cudaGetLastError(), "build_model_ngram_tables launch"))) return rc;
    merge_topk_kernel<<<(n_rows + 127) / 128, 128, 0, st>>>(ctx->d_part_val, ctx->d_part_idx, sh.n_chunks, n_rows, k_tab, d_tab_idx,
                                                           d_tab_val);
    ctx->launches += 2;
    return check_cuda(ctx, cudaGetLastError(), "table merge launch");
}

int launch_extend_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, int w_ext, int32_t* d_ext, cudaStream_t st) {
    const long long n = (long long)ctx->V * k_tab;
    extend_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(d_tab_idx, ctx->V, k_tab, w_ext, d_ext);
    ctx->launches += 1;
    return check_cuda(ctx, cudaGetLastError(), "table extension launch");
}

// ------------------------------------------------------------------------------------------ bounded-wait check
// Test aid: one thread waits, with the same bounded wait the contraction uses, on an mbarrier that nobody
// ever arrives at.  The wait must give up after limit_ns, the kernel must return, and the context must
// report SPEC_STATUS_TIMEOUT.  With mark_incomplete the kernel also does what a contraction CTA does when
// it gives up: it counts itself in the word after the merge ticket, so that the next verification finds
// its merge incomplete.
__global__ void wait_probe_kernel(unsigned long long limit_ns, int* status, unsigned int* ticket, int mark_incomplete) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool got = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_ns);
        if (!got) {
            atomicOr(status, SPEC_STATUS_TIMEOUT);
            if (mark_incomplete) atomicAdd(ticket + 1, 1u);
        }
    }
}

int launch_wait_probe(spec_ctx* ctx, unsigned long long limit_ns, int mark_incomplete, cudaStream_t st) {
    wait_probe_kernel<<<1, 32, 0, st>>>(limit_ns, ctx->d_status, ctx->d_ticket, mark_incomplete);
    ctx->launches += 1;
    return check_cuda(ctx, cudaGetLastError(), "spec_debug_expire_wait launch");
}

// ------------------------------------------------------------------------------------------ vocabulary shards
// Turns merged (value, id) keys (see keys_out above) back into token ids and winning logits.
__global__ void unpack_keys_kernel(const long long* __restrict__ keys, int M, int V_total, int32_t* __restrict__ argmax,
                                   float* __restrict__ maxv) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();
    if (i >= M) return;
    const unsigned long long key = (unsigned long long)keys[i] ^ 0x8000000000000000ull;
    int idx = (int)(~(uint32_t)(key & 0xFFFFFFFFull));
    if (idx < 0 || idx >= V_total) idx = 0;
    argmax[i] = idx;
    if (maxv) maxv[i] = from_orderable_f32((uint32_t)(key >> 32));
}

int launch_unpack_keys(const long long* d_keys, int M, int V_total, int32_t* d_argmax, float* d_max, cudaStream_t st) {
    cudaError_t e = launch_pdl(unpack_keys_kernel, dim3((M + 255) / 256), dim3(256), 0, st, d_keys, M, V_total, d_argmax, d_max);
    return e == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------ model unigram
// Column sums of W in two deterministic stages: colsum[y][t] over a slab of rows, then the mean.
__global__ void unigram_colsum_kernel(const __nv_bfloat16* __restrict__ W, int V, int d, float* __restrict__ colsum) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= d) return;
    const int rows_per = (V + gridDim.y - 1) / gridDim.y;
    const int x0 = blockIdx.y * rows_per, x1 = min(V, x0 + rows_per);
    float acc = 0.0f;
    for (int x = x0; x < x1; ++x) acc += __bfloat162float(W[(size_t)x * d + t]);
    colsum[(size_t)blockIdx.y * d + t] = acc;
}
__global__ void unigram_mean_kernel(const float* __restrict__ colsum, int n_slabs, int V, int d, float* __restrict__ mean) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= d) return;
    float acc = 0.0f;
    for (int y = 0; y < n_slabs; ++y) acc += colsum[(size_t)y * d + t];
    mean[t] = acc / (float)V;
}
// centred[x][t] = bf16(W[x][t] - mean[t])
__global__ void unigram_centre_kernel(const __nv_bfloat16* __restrict__ W, const float* __restrict__ mean, size_t n, int d,
                                      __nv_bfloat16* __restrict__ out) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (; i < n; i += stride) out[i] = __float2bfloat16_rn(__bfloat162float(W[i]) - mean[i % d]);
}
// dist2[x] = sum over chunks of the partial sums, in chunk order
__global__ void unigram_sum_kernel(const float* __restrict__ part, int n_chunks, int V, float* __restrict__ dist2) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= V) return;
    float acc = 0.0f;
    for (int c = 0; c < n_chunks; ++c) acc += part[(size_t)c * V + x];
    dist2[x] = acc;
}
// The k smallest distances in ascending order, equal values by ascending token id: one CTA picks, k
// times, the smallest (value, id) key above the previous pick.
__global__ void __launch_bounds__(1024) unigram_smallest_k_kernel(const float* __restrict__ dist2, int V, int k,
                                                                  int32_t* __restrict__ idx) {
    __shared__ unsigned long long warp_min[32];
    __shared__ unsigned long long picked;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long prev = 0ull;
    bool first = true;
    for (int j = 0; j < k; ++j) {
        unsigned long long best = ~0ull;
        for (int x = tid; x < V; x += blockDim.x) {
            const unsigned long long key = ((unsigned long long)orderable_f32(dist2[x]) << 32) | (uint32_t)x;
            if ((first || key > prev) && key < best) best = key;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other < best ? other : best;
        }
        if (lane == 0) warp_min[warp] = best;
        __syncthreads();
        if (warp == 0) {
            unsigned long long b = lane < (int)(blockDim.x >> 5) ? warp_min[lane] : ~0ull;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long other = __shfl_xor_sync(0xffffffffu, b, o);
                b = other < b ? other : b;
            }
            if (lane == 0) {
                picked = b;
                idx[j] = (int32_t)(uint32_t)(b & 0xFFFFFFFFull);
            }
        }
        __syncthreads();
        prev = picked;
        first = false;
        __syncthreads();
    }
}

int launch_unigram(spec_ctx* ctx, int k_uni, int32_t* d_uni_idx, float* d_dist2, cudaStream_t st) {
    int rc = set_smem_attr<MODE_SUMSQ, 1>(ctx);
    if (rc) return rc;
    const int V = ctx->V, d = ctx->d, n_slabs = 64;
    const size_t n = (size_t)V * d;
    if (!ctx->d_centred) {
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_centred, n * 2), "cudaMalloc(centred embeddings)"))) return rc;
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_colsum, sizeof(float) * (size_t)(n_slabs + 1) * d), "cudaMalloc(column sums)")))
            return rc;
    }
    const Shape sh = cached_shape(ctx, V, (size_t)1 << 20);
    const size_t need = (size_t)sh.n_chunks * V;
    if (need > ctx->part_capacity) {
        cudaStreamSynchronize(st);
        cudaFree(ctx->d_part_val);
        cudaFree(ctx->d_part_idx);
        ctx->d_part_val = nullptr;
        ctx->d_part_idx = nullptr;
        ctx->part_capacity = 0;
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_part_val, need * sizeof(float)), "cudaMalloc(partial sums)"))) return rc;
        if ((rc = check_cuda(ctx, cudaMalloc(&ctx->d_part_idx, need * sizeof(int32_t)), "cudaMalloc(partial ids)"))) return rc;
        ctx->part_capacity = need;
    }
    float* mean = ctx->d_colsum + (size_t)n_slabs * d;
    const __nv_bfloat16* W = (const __nv_bfloat16*)ctx->unembed;
    unigram_colsum_kernel<<<dim3((d + 127) / 128, n_slabs), 128, 0, st>>>(W, V, d, ctx->d_colsum);
    unigram_mean_kernel<<<(d + 127) / 128, 128, 0, st>>>(ctx->d_colsum, n_slabs, V, d, mean);
    unigram_centre_kernel<<<ctx->num_sms * 8, 256, 0, st>>>(W, mean, n, d, (__nv_bfloat16*)ctx->d_centred);
    const WMaps* tmE;
    if ((rc = w_map(ctx, &tmE, true))) return rc;
    CUtensorMap tmA;
    if ((rc = make_tensor_map(ctx, &tmA, ctx->d_centred, V, d, sh.a_box_rows))) return rc;
    GemmParams p;
    fill_common(ctx, p, V, sh);
    p.part_val = ctx->d_part_val;
    head_gemm_kernel<MODE_SUMSQ, 1><<<sh.grid, GEMM_THREADS, sh.smem, st>>>(tmA, tmA, *tmE, p);
    unigram_sum_kernel<<<(V + 255) / 256, 256, 0, st>>>(ctx->d_part_val, sh.n_chunks, V, d_dist2);
    ctx->launches += 5;
    if (k_uni > 0) {
        unigram_smallest_k_kernel<<<1, 1024, 0, st>>>(d_dist2, V, k_uni, d_uni_idx);
        ctx->launches += 1;
    }
    return check_cuda(ctx, cudaGetLastError(), "build_model_unigram launch");
}

}  // namespace ngs

// ------------------------------------------------------------------------------------------ allocation-free verify
// Scratch of verify_lmhead_argmax_noalloc: merge keys for SPEC_NOALLOC_MAX_ROWS rows, then one 64-bit
// word holding the completion ticket and the count of CTAs that gave up, and one for the status bits.
// It lives in the library image, so every GPU that loads the library holds these ~33 KB until the
// process exits.
static __device__ __align__(256) unsigned long long g_noalloc_scratch[SPEC_NOALLOC_MAX_ROWS + 32];

namespace ngs {
struct NoAllocDevice {
    std::mutex lock;  // host-side state below; calls on one device are enqueued one at a time
    bool ready = false;
    unsigned long long* scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int num_sms = 0;
    EncodeTiledFn encode = nullptr;
    // tensor maps of the head seen last, so that a decode loop does not re-encode them on every call
    const void* w_base = nullptr;
    int w_V = 0, w_d = 0;
    WMaps tm_w;
    spec_ctx::AMap a_maps[4];
    int a_map_next = 0;
};
static NoAllocDevice g_noalloc_dev[64];
}  // namespace ngs

extern "C" int verify_lmhead_argmax_noalloc(const void* d_unembed, int V, int d, const void* d_hidden, int M,
                                            int32_t* d_argmax, float* d_max, int device, void* stream) {
    using namespace ngs;
    if (!d_unembed || !d_hidden || !d_argmax) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_noalloc: NULL pointer");
    if (!aligned16(d_unembed) || !aligned16(d_hidden))
        return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_noalloc: matrices must be 16-byte aligned");
    if (V <= 0 || d <= 0 || d % 8 != 0) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_noalloc: need V > 0, d > 0, d %% 8 == 0");
    if (M < 0 || M > SPEC_NOALLOC_MAX_ROWS)
        return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_noalloc: M = %d exceeds the built-in scratch (at most %d rows); "
                    "use verify_lmhead_argmax with a context for larger blocks", M, (int)SPEC_NOALLOC_MAX_ROWS);
    if (device < 0 || device >= 64) return fail(nullptr, SPEC_ERR_ARG, "verify_lmhead_argmax_noalloc: device %d out of range", device);
    if (M == 0) return SPEC_OK;
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return check_cuda(nullptr, e, "verify_lmhead_argmax_noalloc: cudaSetDevice");

    NoAllocDevice& nd = g_noalloc_dev[device];
    std::lock_guard<std::mutex> guard(nd.lock);
    if (!nd.ready) {
        // One-time set-up for this device (made current above).  In host code the array's name is only a
        // handle: the address a kernel can use has to be asked for, per device.
        int major = 0;
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device)) != cudaSuccess)
            return check_cuda(nullptr, e, "verify_lmhead_argmax_noalloc: cudaDeviceGetAttribute");
        if (major != 10) return fail(nullptr, SPEC_ERR_CUDA, "verify_lmhead_argmax_noalloc: device %d is not sm_100", device);
        if ((e = cudaDeviceGetAttribute(&nd.num_sms, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess)
            return check_cuda(nullptr, e, "verify_lmhead_argmax_noalloc: cudaDeviceGetAttribute");
        unsigned long long* ptr = nullptr;
        if ((e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch)) != cudaSuccess || !ptr)
            return check_cuda(nullptr, e == cudaSuccess ? cudaErrorInvalidSymbol : e, "verify_lmhead_argmax_noalloc: cudaGetSymbolAddress");
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess)
            return fail(nullptr, SPEC_ERR_CUDA, "verify_lmhead_argmax_noalloc: cuTensorMapEncodeTiled not available from the driver");
        nd.scratch = ptr;
        nd.encode = (EncodeTiledFn)fn;
        nd.ready = true;
    }

    // A context on the stack, pointing at the built-in scratch, lets the ordinary launch path run unchanged.
    spec_ctx tmp;
    tmp.device = device;
    tmp.V = V;
    tmp.d = d;
    tmp.num_sms = nd.num_sms;
    tmp.unembed = d_unembed;
    tmp.encode = nd.encode;
    tmp.d_keys = nd.scratch;
    tmp.d_ticket = reinterpret_cast<unsigned int*>(nd.scratch + SPEC_NOALLOC_MAX_ROWS);
    tmp.d_status = reinterpret_cast<int*>(nd.scratch + SPEC_NOALLOC_MAX_ROWS + 1);
    if (nd.w_base == d_unembed && nd.w_V == V && nd.w_d == d) {  // same head as last time: reuse its tensor maps
        tmp.tm_w = nd.tm_w;
        tmp.tm_w_ready = true;
        for (int i = 0; i < 4; ++i) tmp.a_maps[i] = nd.a_maps[i];
        tmp.a_map_next = nd.a_map_next;
    }
    cudaStream_t st = (cudaStream_t)stream;
    int rc = SPEC_OK;
    {
        // The scratch keeps whatever the previous call left: the keys of this call's rows, the ticket and
        // the status word must start at zero.  Outputs start at -1 so an expired wait cannot pass for a result.
        e = cudaMemsetAsync(nd.scratch, 0, sizeof(unsigned long long) * (size_t)M, st);
        if (e == cudaSuccess) e = cudaMemsetAsync(nd.scratch + SPEC_NOALLOC_MAX_ROWS, 0, 2 * sizeof(unsigned long long), st);
        if (e == cudaSuccess) e = cudaMemsetAsync(d_argmax, 0xFF, sizeof(int32_t) * (size_t)M, st);
        rc = check_cuda(&tmp, e, "verify_lmhead_argmax_noalloc: cudaMemsetAsync");
    }
    if (rc == SPEC_OK) rc = launch_verify(&tmp, d_hidden, M, d_argmax, d_max, st, nullptr, nullptr, 0);
    if (rc != SPEC_OK) return fail(nullptr, rc, "%s", tmp.err);
    nd.w_base = d_unembed;
    nd.w_V = V;
    nd.w_d = d;
    nd.tm_w = tmp.tm_w;
    for (int i = 0; i < 4; ++i) nd.a_maps[i] = tmp.a_maps[i];
    nd.a_map_next = tmp.a_map_next;
    return SPEC_OK;
}
