// Shared device/host helpers of the retrieval library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rago.h"

namespace rago {

constexpr int KSUB = 256;            // codewords per sub-space (8-bit codes)
constexpr int TOPK_CAP = 2048;       // candidate buffer of the block-level selector (keys)
constexpr int MAX_K = 1024;          // k and nprobe limit: TOPK_CAP must hold k plus one batch of pushes
constexpr int PROBE_GUARD = 8;       // extra coarse candidates re-scored exactly before the final nprobe cut
constexpr unsigned long long KEY_MAX = 0xFFFFFFFFFFFFFFFFull;

// Device-side error word (first word of every workspace).
enum : uint32_t { ERR_NONE = 0, ERR_WAIT_TIMEOUT = 1, ERR_SMEM_LAYOUT = 2 };
constexpr int ERR_TICKET_WORD = 16;  // word of the 256-byte error block (cleared by every call) that small batches use as a ticket counter

// Launch shape of the table-build + scan kernel for one index (fixed at index load).
struct ScanPlan {
    int tile_vecs;     // vectors per code tile
    int stages;        // tiles in flight per CTA
    int ctas;          // persistent CTAs (one per SM)
    size_t smem_bytes;
    // shared-memory image of a query's lookup table, as the scan variant of this index lays it out
    int lut_bytes, lut_banked, lut_copies, lut_copy_off, lut_stride;
};

// Batches of at most this many queries get their lookup tables from kernels of their own, spread over the whole
// GPU, instead of every scan CTA building the table of each query it meets.
constexpr int PREBUILT_MAX_NQ = 4096;

// Index handle.  Borrowed pointers first, then what the library owns.
struct IndexImpl {
    const void* centroids;
    int coarse_bf16;
    const float* codebooks;
    const uint8_t* codes;
    const int64_t* list_offsets;
    const int64_t* ids;
    int64_t N;
    int32_t d, nlist, M, dsub, metric;
    // owned
    float* cnorm;  // [nlist] squared centroid norms (L2 coarse ranking)
    float* cbT;    // [256][M][dsub] codebook with the codeword index outermost
    float* vterm;  // [N] per-vector term of the L2 expansion (null for inner product)
    float* cwmax;  // [M] largest codeword norm of every sub-space (bounds a table entry without building the table)
    void* cparts;  // bf16 [parts][nlist][d]: the centroids as a sum of bf16 parts (fp32 index); null for a bf16 index
    int cparts_n;  // parts of the tensor-core coarse operand: 3 (fp32 index) or 1 (bf16 index, borrowed array)
    int tc_ok;     // tensor-core coarse path available (tensor map encoded)
    int coarse_mode;  // 0 auto, 1 fp32 pipes, 2 tensor cores
    alignas(64) unsigned char tmap_b[128];  // CUtensorMap of the stacked centroid parts
    alignas(64) unsigned char tmap_b_pilot[128];  // the same, every pilot_stride-th centroid
    alignas(64) unsigned char tmap_b_half[128], tmap_b_pilot_half[128];  // both again in boxes of 128 rows (CTA pairs)
    int pilot_stride;  // 0: no pilot pass for this index
    // optional first quantiser level (borrowed; tree_n1 = 0: none).  Node i owns lists child_offsets[i] .. [i+1]-1.
    const void* tree_level1;            // [tree_n1][d], the coarse dtype
    const int32_t* tree_child_offsets;  // [tree_n1 + 1]
    int tree_n1, tree_b1;
    int tree_max_cand;                  // most candidates b1 nodes can have (sum of the b1 largest child counts)
    int tree_min_cand;                  // fewest (sum of the b1 smallest): nprobe must not exceed it
    int device, num_sms;
    ScanPlan plan;
    int profile;
    cudaEvent_t ev[RAGO_NUM_STAGES + 1];
    float last_ms[RAGO_NUM_STAGES];
    int ev_valid;
};

// ---- order-preserving float <-> uint32 ------------------------------------------------------
__host__ __device__ inline uint32_t f32_orderable(float f) {
#ifdef __CUDA_ARCH__
    uint32_t u = __float_as_uint(f);
#else
    union { float f; uint32_t u; } c; c.f = f; uint32_t u = c.u;
#endif
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__host__ __device__ inline float orderable_f32(uint32_t o) {
    uint32_t u = (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o;
#ifdef __CUDA_ARCH__
    return __uint_as_float(u);
#else
    union { float f; uint32_t u; } c; c.u = u; return c.f;
#endif
}
// the same on raw fp32 bit patterns
__host__ __device__ inline uint32_t ord_bits(uint32_t u) { return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u); }
__host__ __device__ inline uint32_t unord_bits(uint32_t o) { return (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o; }
__host__ __device__ inline unsigned long long make_key(float score_smaller_is_better, uint32_t payload) {
    return ((unsigned long long)f32_orderable(score_smaller_is_better) << 32) | payload;
}

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#ifdef __CUDACC__
// ---- shared-memory address / mbarrier / bulk-copy wrappers ----------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// try_wait that lets the hardware park the thread for up to `ns` nanoseconds before it answers.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
// Bounded wait: each poll may park the thread for up to 4 us, and the wait gives up after max_polls
// polls (2^18: about a second) or as soon as *abort_flag is set by another warp.  On give-up it raises the
// CTA abort flag and the global error word; callers keep their control flow (so CTA-wide barriers
// still match) but the data is garbage.
constexpr uint32_t MBAR_MAX_POLLS = 1u << 18;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* err_word, uint32_t backoff_ns = 0,
                                          uint32_t max_polls = MBAR_MAX_POLLS) {
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t it = 0; it < max_polls; ++it) {
        if (mbar_try_wait_hint(bar, parity, 4000u)) return true;
        if (backoff_ns) __nanosleep(backoff_ns);  // single-lane roles: leave the issue slots to the working warps
        if ((it & 15) == 15 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(err_word, (uint32_t)ERR_WAIT_TIMEOUT);
    return false;
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier.
// dst/src 16-byte aligned, bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// The same with an L2 eviction-priority hint (a policy made by l2_policy_evict_first): data that is read once should
// not push out what the next kernels will read again.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
#endif  // __CUDACC__

// ---- host-side launch bookkeeping -------------------------------------------------------------
void count_launch(int n = 1);

// ---- back-to-back kernels of one search -------------------------------------------------------------
// A kernel launched with launch_overlapped may be scheduled while the kernel before it on the stream is still
// draining; it must not touch global memory before grid_dependency_wait(), which returns once that kernel has
// completed and its writes are visible.  Every kernel of the chain waits first thing and then lets its own
// successor be scheduled, so the order of all memory accesses is the stream order; what overlaps is launch
// latency.  In a kernel launched the ordinary way both calls do nothing.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <class... P, class... A>
inline cudaError_t launch_overlapped(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, P(args)...);
}
void set_error(const char* fmt, ...);

// ---- kernel launchers (one per .cu file) ------------------------------------------------------

// coarse.cu
cudaError_t launch_centroid_norms(const void* centroids, int bf16, int nlist, int d, float* cnorm, cudaStream_t s);
bool coarse_small_applies(const IndexImpl* ix, int nq);
cudaError_t launch_coarse_scores(const IndexImpl* ix, const float* queries, int nq, float* scores, uint32_t* clear_block,
                                 cudaStream_t s);
cudaError_t launch_tree_candidates(const IndexImpl* ix, const float* queries, int nq, int S, int cap,
                                   unsigned long long* cand, int32_t* cand_cnt, uint32_t* clear_block, cudaStream_t s);
constexpr int TREE_LIMIT_B1 = 64, TREE_LIMIT_N1 = 4096;
// gemm_select.cu
constexpr int GEMM_CAP_SMALL = 512, GEMM_CAP_LARGE = 1024;  // candidate-list capacities (keys per list)
constexpr int GEMM_COL_HALVES = 2;  // a row has one candidate list per column range of the grid AND per half of a 256-column tile
struct GemmLaunch {
    const void* tmap_a;          // CUtensorMap of A: bf16 [a parts * a_part_rows][d]
    const void* tmap_b;          // CUtensorMap of B: bf16 [b parts * b_part_rows][d], boxes of 256 rows
    const void* tmap_b_half;     // the same matrix in boxes of 128 rows (mg = 3: a CTA of a pair loads half a B tile)
    int nrows; int64_t ncols; int d;
    int a_part_rows; int64_t b_part_rows;
    int nterms; int term_a[6], term_b[6];
    int mg, nsplit;              // from gemm_grid: main loop (1 single, 2 pair in a CTA, 3 CTA pair) and column ranges
    float alpha; const float* colterm; int colterm_stride;
    const float* row_tau;        // initial per-row thresholds (mode 0) or null
    int mode, nsel, cap;
    unsigned long long* cand; int32_t* cand_cnt;  // [nrows][nsplit * GEMM_COL_HALVES][cap] keys and their counts
    float* scores; uint32_t* err;
};
// Candidate lists leave the tensor-core kernel as RAW entries: low word = column, high word = fp32 bits of the
// score xor a sign word (0x80000000 when the kernel stores the accumulator value of a score = -value).  Readers
// turn an entry into the usual key with cand_key().
__host__ __device__ inline uint32_t gemm_cand_sign(float alpha, const float* colterm) { return alpha == -1.f && colterm == nullptr ? 0x80000000u : 0u; }
__host__ __device__ inline unsigned long long cand_key(unsigned long long entry, uint32_t sign) {
    return ((unsigned long long)ord_bits((uint32_t)(entry >> 32) ^ sign) << 32) | (uint32_t)entry;
}
cudaError_t gemm_select_init();
cudaError_t make_tmap_bf16(void* out_map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
                           uint64_t row_stride = 0);
// The pilot pass scores every stride-th column: 16, or more when that would still leave over 32 768 columns.
inline int gemm_pilot_stride(int64_t ncols) { const int64_t s = (ncols + 32767) / 32768; return s > 16 ? (int)s : 16; }
cudaError_t launch_row_tau(const float* scores, int nrows, int n, int nsel, float* row_tau, cudaStream_t s);
int gemm_cand_cap(int nsel);  // 0: nsel too large for the fused selection
void gemm_grid(int nrows, int64_t ncols, int d, int num_sms, int* mg, int* nsplit, int* mgroups);
void gemm_set_pairing(int mode);
cudaError_t launch_gemm_select(const GemmLaunch& L, cudaStream_t s);
cudaError_t launch_split_bf16(const float* x, size_t n, int parts, void* out, cudaStream_t s);
cudaError_t launch_selftest_wait(uint32_t* err_word, uint32_t max_polls, int with_tmem, uint32_t* observed, cudaStream_t s);
// scan.cu
bool scan_supported(int M);
cudaError_t scan_plan(const IndexImpl* ix, ScanPlan* plan);
cudaError_t launch_vector_terms(const IndexImpl* ix, float* vterm, cudaStream_t s);
cudaError_t launch_transpose_codebook(const float* cb, int M, int dsub, float* cbT, cudaStream_t s);
cudaError_t launch_plan_work(const IndexImpl* ix, const int32_t* probe_list, int npairs, int tile_vecs,
                             int32_t* pair_tiles, int64_t* work_prefix, unsigned long long* qthresh, int nq,
                             int32_t* slot_cnt, int nslots, const float* queries, uint8_t* lut_img, float* lut_inv,
                             float* lut_scale, cudaStream_t s);
cudaError_t launch_scan(const IndexImpl* ix, const ScanPlan& plan, const float* queries, const int32_t* probe_list,
                        const float* probe_term, const int64_t* work_prefix, int nq, int nprobe, int k,
                        unsigned long long* qthresh, int32_t* slot_cnt, unsigned long long* slot_keys,
                        uint32_t* err_word, const uint8_t* lut_img, const float* lut_inv, cudaStream_t s);
cudaError_t launch_codeword_norms(const float* codebooks, int M, int dsub, float* cwmax, cudaStream_t s);
cudaError_t launch_build_tables(const IndexImpl* ix, const float* queries, int nq, uint8_t* lut_img, float* lut_inv,
                                float* lut_scale, cudaStream_t s);
// no_alloc.cu
cudaError_t noalloc_prepare();  // with the index's device current: look up (and make resident) the built-in scratch array
// merge.cu
cudaError_t launch_merge(const IndexImpl* ix, const int64_t* work_prefix, int nq, int nprobe, int k, int ctas,
                         const int32_t* slot_cnt, const unsigned long long* slot_keys, const unsigned long long* qthresh,
                         const float* queries, const int32_t* probe_list, const float* probe_bias, int64_t* out_ids,
                         float* out_dists, cudaStream_t s);
cudaError_t launch_fill_u64(unsigned long long* p, size_t n, unsigned long long v, cudaStream_t s);
// flat.cu
size_t flat_workspace_bytes(int64_t N, int d, int nq, int k);
cudaError_t launch_flat_search(const void* db, int64_t N, int d, const void* queries, int nq, int k, int64_t* out_ids,
                               float* out_scores, void* workspace, cudaStream_t s);

}  // namespace rago
