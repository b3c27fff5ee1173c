// Dense scores on the 5th-generation tensor cores with the per-row selection fused into the epilogue.
//
//   S[r][c] = alpha * sum_t <A_{ta(t)}[r], B_{tb(t)}[c]>  +  colterm[c]          smaller = better
//
// A (queries) and B (coarse centroids, or the flat database) are bf16, row-major with the
// contraction dimension innermost.  fp32 operands are represented as sums of bf16 "parts"
// (x = x0 + x1 + x2 exactly up to 24 bits) and the product as the six part pairs whose weight is at
// least 2^-16 relative; each pair is simply more K-blocks accumulated into the same TMEM tile.
//
// One CTA works on 128 x 256 output tiles, K-blocks of 64 bf16 (one 128-byte swizzle span):
//   warp 0    TMA producer: cp.async.bulk.tensor (tiled, 128B swizzle) into a ring of stages, mbarrier tx counts
//   warp 1    one lane issues tcgen05.mma (M128 N256 K16, bf16 -> fp32 in TMEM), tcgen05.commit frees stages
//   warps 2-9 epilogue: tcgen05.ld 32 columns at a time, thread = output row; warp w reads TMEM lane quarter
//             w mod 4 and the column half (w - 2) / 4 of the tile, and never waits for another warp
// Three shapes of the main loop (template parameter LOOP):
//   LOOP_SINGLE    one row tile per CTA.  A stage holds A (16 KB) and B (32 KB), four stages; the two 256-column
//                  TMEM accumulators alternate, so the epilogue of one tile overlaps the MMAs of the next.
//   LOOP_PAIR      two row tiles per CTA (256 queries).  A stage holds A0, A1 and ONE B tile (64 KB), three
//                  stages; every K-block feeds two MMA chains, A0.B into accumulator 0 and A1.B into accumulator
//                  1, so a B tile crosses L2 -> shared memory once per 256 queries and the operand traffic per
//                  flop drops by a third.  Both accumulators belong to the same column tile, so the epilogue
//                  does not overlap the next tile's MMAs; eight epilogue warps keep it short.
//   LOOP_TWO_CTA   a cluster of two CTAs (one SM pair) works on 256 rows x 256 columns with tcgen05.mma
//                  cta_group::2: each CTA loads its own 128 rows of A and HALF of the B tile (128 of the 256
//                  columns' rows), 32 KB per stage, six stages; one thread of the cluster's first CTA issues the
//                  MMAs (M = 256), each CTA's tensor memory receives its own 128 rows, and the accumulators
//                  alternate as in LOOP_SINGLE, so the operand traffic of LOOP_PAIR comes with an overlapped
//                  epilogue.  Loads of both CTAs complete on the first CTA's "full" barrier; tcgen05.commit
//                  signals "stage empty" and "accumulator full" in both CTAs; the second CTA's epilogue warps
//                  arrive on the first CTA's "accumulator empty" barrier through the cluster's shared window.
//                  No copy is multicast: every CTA fetches its own operands.
// A CTA owns a contiguous range of column tiles, so a row's running state (threshold, candidate count) lives in
// the registers of the thread that owns the (row, column half).
//
// Fused selection (mode 0).  A value below the row's threshold is appended to a candidate list in global memory
// (one list per row, column range and column half; capacity CAP = 32*NK keys, 64-bit key = ordered score bits
// << 32 | column).  When a list could overflow, its warp loads it into registers (NK keys per lane), bisects for
// a cut value that keeps between nsel and nsel + slack keys (a few warp-wide counts), writes the kept keys back
// and lowers the threshold.  The threshold is always at least the nsel-th smallest of a subset of the row, so no
// key that belongs to the row's nsel best is ever dropped; the lists are merged by the caller.  Mode 1 writes
// the score matrix instead.
//
// Pilot thresholds.  A row may start with a threshold instead of +inf: the caller first runs mode 1
// over every 16th column (a tensor map with a 16-row stride: 6% more work) and takes, per row, the
// nsel-th smallest of that sample (row_tau_kernel).  The nsel-th smallest of a subset is never below
// the nsel-th smallest of the whole row, so the selection stays exact, while the values that get past
// the filter drop from thousands per row to about 16 * nsel and lists hardly ever need cutting.
//
// Every wait is bounded (common.cuh); on a timeout the roles leave their loops, the error word is
// set, TMEM is still released.
#include <cuda.h>
#include <cstring>

#include "topk.cuh"

namespace rago {

constexpr int GBM = 128, GBN = 256, GBK = 64;
constexpr int G_A_BYTES = GBM * GBK * 2;
constexpr int G_B_BYTES = GBN * GBK * 2;
constexpr int G_RING_BYTES = 4 * (G_A_BYTES + G_B_BYTES);  // four stages of A + B, or three of A0 + A1 + B
constexpr int G_MAX_STAGES = 6;
constexpr int LOOP_SINGLE = 0, LOOP_PAIR = 1, LOOP_TWO_CTA = 2;
constexpr int G_EPI_WARPS = 8;                       // 4 TMEM lane quarters x 2 column halves
constexpr int G_THREADS = 32 * (2 + G_EPI_WARPS);
constexpr int G_HALF = GBN / GEMM_COL_HALVES;        // columns of a tile one epilogue warp reads
constexpr int G_TMEM_COLS = 512;
constexpr int G_CN_BYTES = G_EPI_WARPS * 2 * G_HALF * 4;  // column terms: two copies per epilogue warp
constexpr int G_SMEM_BYTES = G_RING_BYTES + G_CN_BYTES + 256 + 1024;  // + barriers + alignment slack
static_assert(3 * (2 * G_A_BYTES + G_B_BYTES) <= G_RING_BYTES, "three paired stages fit the ring");
static_assert(6 * (G_A_BYTES + G_B_BYTES / 2) <= G_RING_BYTES, "six two-CTA stages fit the ring");

// tcgen05 instruction descriptor, kind::f16: D = f32 (bits 4-5 = 1), A = B = bf16 (bits 7-9, 10-12 = 1),
// both operands K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in bits 24-28.
constexpr uint32_t G_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GBN >> 3) << 17) | ((uint32_t)(GBM >> 4) << 24);
constexpr uint32_t G_IDESC_2CTA = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GBN >> 3) << 17) | ((uint32_t)((2 * GBM) >> 4) << 24);  // M = 256 over the CTA pair

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(const CUtensorMap* map, uint32_t bar, uint32_t dst, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// ---- the same for a CTA pair (cta_group::2) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tiled load into this CTA's shared memory whose completion bytes count on a barrier of the pair (bar is a
// shared::cluster address: the leader's barrier).  One destination, one CTA: nothing is multicast.
__device__ __forceinline__ void tma_load_2d_pair(const CUtensorMap* map, uint32_t cluster_bar, uint32_t dst, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(cluster_bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets TMEM lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
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
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (one swizzle span):
// start address >> 4 in bits 0-13, leading-dimension offset (unused for this layout) 1 in bits 16-29,
// stride between 8-row groups (1024 bytes) >> 4 in bits 32-45, descriptor version 1 in bits 46-47,
// layout type 2 (128-byte swizzle) in bits 61-63.  The tile base is 1024-byte aligned; a K step of 16
// elements (32 bytes) inside the span advances the start-address field by 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}

// A candidate list holds RAW entries: low word = column, high word = the fp32 bits of the score xor `sign`
// (sign = 0x80000000 on the alpha = -1 path, where the accumulator value itself is stored and the score is its
// negation).  Appending is then a compare, a predicated 8-byte store and a predicated pointer bump per value;
// the order-preserving key bits are formed by whoever reads the list (cand_key in common.cuh).
//   if (value > thr) { *ptr++ = {col, bits(value)}; }          (alpha = -1, no column term: score = -value)
__device__ __forceinline__ void push_if_above(unsigned long long*& ptr, float value, float thr, uint32_t col) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.gt.f32 p, %1, %2;\n\t"
        "@p st.global.v2.u32 [%0], {%3, %4};\n\t"
        "@p add.u64 %0, %0, 8;\n\t}"
        : "+l"(ptr)
        : "f"(value), "f"(thr), "r"(col), "r"(__float_as_uint(value))
        : "memory");
}
//   if (score < tau) { *ptr++ = {col, bits}; }
__device__ __forceinline__ void push_if_below(unsigned long long*& ptr, float score, float tau, uint32_t col, uint32_t bits) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.lt.f32 p, %1, %2;\n\t"
        "@p st.global.v2.u32 [%0], {%3, %4};\n\t"
        "@p add.u64 %0, %0, 8;\n\t}"
        : "+l"(ptr)
        : "f"(score), "f"(tau), "r"(col), "r"(bits)
        : "memory");
}

struct GemmArgs {
    int nrows, ncols;            // valid rows of A (queries) and of B (lists / database rows)
    int a_part_rows, b_part_rows;  // row distance between consecutive parts in the stacked operands
    int kblocks;                 // ceil(d / 64)
    int nterms;
    int term_a[6], term_b[6];    // part pair of each term
    int mtiles, ntiles;          // row tiles, column tiles
    float alpha;
    const float* colterm;        // [ncols * colterm_stride] or null: column c adds colterm[c * colterm_stride]
    int colterm_stride;
    const float* row_tau;        // [nrows] initial thresholds (mode 0) or null for +inf
    int mode;                    // 0: candidate lists, 1: score matrix
    int nsel;                    // keys a row must keep (mode 0)
    unsigned long long* cand;    // [nrows][nsplit][GEMM_COL_HALVES][CAP]
    int32_t* cand_cnt;           // [nrows][nsplit][GEMM_COL_HALVES]
    float* scores;               // [nrows][ncols] (mode 1)
    uint32_t* err;
};

// Cut one list of n (> nsel) keys down to between nsel and nkeep keys and return the new threshold.
// The cut value T is found by bisection on the ordered score bits between the list's minimum and
// maximum: it stops as soon as nsel <= #(score <= T) <= nkeep, which takes a handful of warp-wide
// counts instead of one per bit; if it runs down to a single value (a tie group larger than the slack)
// only as many of the tied keys are kept as are needed to reach nsel.  Every kept set contains the
// nsel smallest keys of the list, and the threshold is the largest kept score.
// The list is in the raw format described above (sign: see push_if_above) and stays in it.
template <int NK>
__device__ __forceinline__ float compact_list(unsigned long long* list, int n, int nsel, int nkeep, int lane, int* kept,
                                              uint32_t sign) {
    uint32_t s[NK];
    uint32_t pl[NK];
    uint32_t mn = 0xFFFFFFFFu, mx = 0u;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        const int idx = lane + 32 * j;
        const unsigned long long k = idx < n ? list[idx] : 0ull;
        s[j] = idx < n ? ord_bits((uint32_t)(k >> 32) ^ sign) : 0xFFFFFFFFu;
        pl[j] = (uint32_t)k;
        if (idx < n) {
            mn = s[j] < mn ? s[j] : mn;
            mx = s[j] > mx ? s[j] : mx;
        }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    // invariant: #(score <= lo) < nsel <= #(score <= hi)   (lo = mn - 1 as a 64-bit value to allow mn = 0)
    long long lo = (long long)mn - 1, hi = mx;
    uint32_t c_hi = (uint32_t)n;
#pragma unroll 1
    while (hi - lo > 1 && c_hi > (uint32_t)nkeep) {
        const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
        uint32_t c = 0;
#pragma unroll
        for (int j = 0; j < NK; ++j) c += (s[j] <= mid) ? 1u : 0u;  // padding keys carry the largest score pattern
        c = __reduce_add_sync(0xffffffffu, c);
        if (c < (uint32_t)nsel) lo = mid; else { hi = mid; c_hi = c; }
    }
    const uint32_t T = (uint32_t)hi;
    // keys below T are all kept; keys equal to T only as far as needed when the tie group is too large
    uint32_t less = 0;
#pragma unroll
    for (int j = 0; j < NK; ++j) less += (s[j] < T) ? 1u : 0u;
    less = __reduce_add_sync(0xffffffffu, less);
    int need = c_hi <= (uint32_t)nkeep ? (int)(c_hi - less) : nsel - (int)less;  // keys equal to T to keep
    __syncwarp();
    const uint32_t lt_mask = (1u << lane) - 1u;
    int base = 0;
#pragma unroll
    for (int j = 0; j < NK; ++j) {
        const bool valid = lane + 32 * j < n;
        const bool eq = valid && s[j] == T;
        const uint32_t meq = __ballot_sync(0xffffffffu, eq);
        const bool keep = valid && (s[j] < T || (eq && __popc(meq & lt_mask) < need));
        const uint32_t mk = __ballot_sync(0xffffffffu, keep);
        if (keep) list[base + __popc(mk & lt_mask)] = ((unsigned long long)(unord_bits(s[j]) ^ sign) << 32) | pl[j];
        base += __popc(mk);
        const int eq_kept = __popc(meq) < need ? __popc(meq) : need;
        need -= eq_kept;
    }
    __syncwarp();
    *kept = base;
    return orderable_f32(T);
}

// Epilogue of one accumulator half in mode 0: G_HALF columns starting at TMEM address taddr, global column col_g.
// NEG1: alpha = -1 and no column term, so "score < tau" is "value > -tau" on the accumulator value itself and
// nothing but the compare stands between the TMEM load and the store (chunks that reach past the last valid
// column take the general path, whose column terms are +inf there).
// (Measured and dropped: skipping pairs of columns behind a warp-wide vote when none of their 64 values passes.
// Even at the flat search's pass rate of 0.3% the votes and branches cost more than the predicated stores save.)
template <int NK, bool NEG1>
__device__ __forceinline__ void epilogue_select(uint32_t taddr, const float* cn, float alpha, uint32_t col_g, int ncols,
                                                unsigned long long* list, float& tau, int& cnt, int nsel, int nkeep,
                                                int lane) {
    constexpr int CAP = NK * 32;
    constexpr uint32_t SIGN = NEG1 ? 0x80000000u : 0u;
    unsigned long long* ptr = list + cnt;
    unsigned long long* const full = list + (CAP - 32);
#pragma unroll 1
    for (int c0 = 0; c0 < G_HALF; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + c0, v);
        const uint32_t colc = col_g + c0;
        if (NEG1 && (int)colc + 32 <= ncols) {
            const float thr = -tau;
#pragma unroll
            for (int j = 0; j < 32; ++j) push_if_above(ptr, v[j], thr, colc + j);
        } else {
            // all 32 scores first (their column-term loads must not queue behind the stores), then one
            // predicated store per value: no branches, the only serial dependence is the list cursor
            float sc[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                const float4 c4 = *reinterpret_cast<const float4*>(cn + c0 + j);
                sc[j + 0] = fmaf(alpha, v[j + 0], c4.x);
                sc[j + 1] = fmaf(alpha, v[j + 1], c4.y);
                sc[j + 2] = fmaf(alpha, v[j + 2], c4.z);
                sc[j + 3] = fmaf(alpha, v[j + 3], c4.w);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) push_if_below(ptr, sc[j], tau, colc + j, __float_as_uint(sc[j]) ^ SIGN);
        }
        uint32_t todo = __ballot_sync(0xffffffffu, ptr > full);
        while (todo) {  // warp-uniform
            const int r = __ffs(todo) - 1;
            todo &= todo - 1;
            const int n = __shfl_sync(0xffffffffu, (int)(ptr - list), r);
            const unsigned long long lp = __shfl_sync(0xffffffffu, (unsigned long long)list, r);
            __syncwarp();
            int kept = 0;
            const float nt_tau =
                compact_list<NK>(reinterpret_cast<unsigned long long*>(lp), n, nsel, nkeep, lane, &kept, SIGN);
            if (lane == r) { ptr = list + kept; tau = nt_tau; }
        }
    }
    cnt = (int)(ptr - list);
}

// The same in mode 1: scores of row `row`, columns colb .. colb + G_HALF - 1, to the score matrix.
__device__ __forceinline__ void epilogue_store(uint32_t taddr, const float* cn, float alpha, int row, int nrows,
                                               int ncols, int colb0, float* scores) {
#pragma unroll 1
    for (int c0 = 0; c0 < G_HALF; c0 += 32) {
        float v[32];
        tmem_ld32(taddr + c0, v);
        if (row < nrows) {
            const int colb = colb0 + c0;
            float* out = scores + (size_t)row * ncols + colb;
            if ((ncols & 3) == 0 && colb + 32 <= ncols) {  // 16-byte stores: rows start on 16-byte boundaries
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 c4 = *reinterpret_cast<const float4*>(cn + c0 + j);
                    float4 o;
                    o.x = fmaf(alpha, v[j + 0], c4.x);
                    o.y = fmaf(alpha, v[j + 1], c4.y);
                    o.z = fmaf(alpha, v[j + 2], c4.z);
                    o.w = fmaf(alpha, v[j + 3], c4.w);
                    *reinterpret_cast<float4*>(out + j) = o;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (colb + j < ncols) out[j] = fmaf(alpha, v[j], cn[c0 + j]);
            }
        }
    }
}

template <int NK, int LOOP>
__global__ void __launch_bounds__(G_THREADS, 1)
gemm_select_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs a) {
    constexpr int CAP = NK * 32;
    constexpr bool PAIR = LOOP == LOOP_PAIR, TWO = LOOP == LOOP_TWO_CTA;
    constexpr int STAGES = PAIR ? 3 : (TWO ? 6 : 4);
    constexpr int B_BYTES = TWO ? G_B_BYTES / 2 : G_B_BYTES;  // a CTA of a pair holds half of the B tile
    constexpr int STAGE_BYTES = (PAIR ? 2 : 1) * G_A_BYTES + B_BYTES;
    constexpr int B_OFF = STAGE_BYTES - B_BYTES;  // B follows the A tile(s) of its stage
    const uint32_t crank = TWO ? cluster_ctarank() : 0u;  // 0: the CTA that issues the pair's MMAs
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    float* cn_all = reinterpret_cast<float*>(smem + G_RING_BYTES);  // [8 warps][2][G_HALF] column terms
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + G_RING_BYTES + G_CN_BYTES);
    const uint32_t bar0 = base + G_RING_BYTES + G_CN_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (G_MAX_STAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * G_MAX_STAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * G_MAX_STAGES + 2 + b); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * G_MAX_STAGES + 4);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), TWO ? 2 * G_EPI_WARPS : G_EPI_WARPS);  // the leader hears from both CTAs' epilogues
        }
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 0) {
        if (TWO) tmem_alloc_pair(smem_u32(tmem_slot), G_TMEM_COLS); else tmem_alloc(smem_u32(tmem_slot), G_TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    if (TWO) cluster_sync_all();  // the peer's barriers exist before anything of ours is aimed at them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // PAIR / TWO: blockIdx.y counts pairs of row tiles (the last pair may hold one tile); else row tiles.
    // TWO: the two CTAs of a cluster are neighbours in x and share a column range.
    const int split = TWO ? blockIdx.x >> 1 : blockIdx.x, nsplit = TWO ? gridDim.x >> 1 : gridDim.x;
    const int m0 = PAIR ? blockIdx.y * 2 : (TWO ? blockIdx.y * 2 + (int)crank : blockIdx.y);
    const int mcount = PAIR ? ((a.mtiles - m0) < 2 ? (a.mtiles - m0) : 2) : 1;
    const int nt_begin = (int)((long long)split * a.ntiles / nsplit);
    const int nt_end = (int)((long long)(split + 1) * a.ntiles / nsplit);
    const int nunits = nt_end - nt_begin;  // column tiles of this CTA
    const int kiters = a.nterms * a.kblocks;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            // unit = column tile; inside it the terms, inside a term the k-blocks: kept by counting, no division per load
            const int total = nunits * kiters;
            const uint32_t tx_bytes = TWO ? 2u * STAGE_BYTES  // both CTAs' loads complete on the leader's barrier
                                          : (uint32_t)(mcount == 2 ? STAGE_BYTES : G_A_BYTES + G_B_BYTES);
            int nt = nt_begin, t = 0, kb = 0, s = 0;
            uint32_t ph = 0;
            for (int gi = 0; gi < total; ++gi) {
                const int kx = kb * GBK;
                const int ya = a.term_a[t] * a.a_part_rows + m0 * GBM;
                const int yb = a.term_b[t] * a.b_part_rows + nt * GBN;
                if (++kb == a.kblocks) {
                    kb = 0;
                    if (++t == a.nterms) { t = 0; ++nt; }
                }
                if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, a.err, 64)) break;
                const uint32_t st = base + s * STAGE_BYTES;
                if (TWO) {
                    // An mbarrier's transaction count may run ahead of its expectation, so the peer's bytes may land
                    // before the leader announces them; the phase cannot complete without the leader's arrival.
                    if (crank == 0) mbar_arrive_expect_tx(full_bar(s), tx_bytes);
                    const uint32_t lead_full = mapa_shared(full_bar(s), 0);
                    tma_load_2d_pair(&tmA, lead_full, st, kx, ya);
                    tma_load_2d_pair(&tmB, lead_full, st + B_OFF, kx, yb + (int)crank * (GBN / 2));
                } else {
                    mbar_arrive_expect_tx(full_bar(s), tx_bytes);
                    tma_load_2d(&tmA, full_bar(s), st, kx, ya);
                    if (PAIR && mcount == 2) tma_load_2d(&tmA, full_bar(s), st + G_A_BYTES, kx, ya + GBM);
                    tma_load_2d(&tmB, full_bar(s), st + B_OFF, kx, yb);
                }
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (of a CTA pair: the leader's) =================
        if (lane == 0 && crank == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool dead = false;
            for (int u = 0; u < nunits && !dead; ++u) {
                // PAIR: both accumulators belong to this unit, one barrier pair; else the accumulators alternate
                const int buf = PAIR ? 0 : (u & 1);
                const uint32_t uph = PAIR ? (u & 1u) : ((u >> 1) & 1u);
                if (!mbar_wait(tempty_bar(buf), uph ^ 1u, abort_flag, a.err, 64)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * GBN);
                for (int ki = 0; ki < kiters; ++ki) {
                    if (!mbar_wait(full_bar(s), ph, abort_flag, a.err, 32)) { dead = true; break; }
                    tc_fence_after();
                    const uint32_t st = base + s * STAGE_BYTES;
                    const uint64_t da = smem_desc_sw128(st);
                    const uint64_t db = smem_desc_sw128(st + B_OFF);
#pragma unroll
                    for (int k = 0; k < GBK / 16; ++k) {
                        if (TWO) tc_mma_bf16_pair(d_tmem, da + 2u * k, db + 2u * k, G_IDESC_2CTA, (ki | k) != 0 ? 1u : 0u);
                        else tc_mma_bf16(d_tmem, da + 2u * k, db + 2u * k, G_IDESC, (ki | k) != 0 ? 1u : 0u);
                    }
                    if (PAIR && mcount == 2) {
                        const uint64_t da1 = smem_desc_sw128(st + G_A_BYTES);
#pragma unroll
                        for (int k = 0; k < GBK / 16; ++k)
                            tc_mma_bf16(d_tmem + GBN, da1 + 2u * k, db + 2u * k, G_IDESC, (ki | k) != 0 ? 1u : 0u);
                    }
                    if (TWO) tc_commit_pair(empty_bar(s)); else tc_commit(empty_bar(s));  // frees the stage once these MMAs have read it
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!dead) { if (TWO) tc_commit_pair(tfull_bar(buf)); else tc_commit(tfull_bar(buf)); }  // accumulator(s) complete
            }
        }
    } else {
        // ================= epilogue warps =================
        const int ew = warp - 2;
        const int q4 = warp & 3;   // TMEM lane quarter this warp may read
        const int half = ew >> 2;  // column half of the tile: warps 2-5 take half 0, warps 6-9 half 1
        float* cn = cn_all + ew * 2 * G_HALF;  // this warp's own copies: no cross-warp barrier needed
        const float inf = __int_as_float(0x7f800000);
        float tau[2] = {inf, inf};
        int cnt[2] = {0, 0};
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const int r = (m0 + g) * GBM + q4 * 32 + lane;
            if (r >= a.nrows || g >= mcount) tau[g] = -inf; else if (a.row_tau) tau[g] = a.row_tau[r];
        }
        const int slack = a.nsel / 4 > 8 ? a.nsel / 4 : 8;
        const int nkeep = a.nsel + slack < CAP - 64 ? a.nsel + slack : CAP - 64;  // what the bisection may leave in a list
        const bool neg1 = gemm_cand_sign(a.alpha, a.colterm) != 0u;  // accumulator values are compared and stored as they are
        unsigned long long* lists[2];
#pragma unroll
        for (int g = 0; g < 2; ++g) {  // never written for padding rows
            const int r = (m0 + g) * GBM + q4 * 32 + lane;
            lists[g] = a.cand + (((size_t)(r < a.nrows ? r : 0) * nsplit + split) * GEMM_COL_HALVES + half) * CAP;
        }
        bool dead = false;
        for (int u = 0; u < nunits && !dead; ++u) {
            const int nt = nt_begin + u;
            const int buf = PAIR ? 0 : (u & 1);
            const uint32_t uph = PAIR ? (u & 1u) : ((u >> 1) & 1u);
            float* cnu = cn + (u & 1) * G_HALF;
            const int colb = nt * GBN + half * G_HALF;
            for (int i = lane; i < G_HALF; i += 32) {
                const int col = colb + i;
                cnu[i] = col < a.ncols ? (a.colterm ? __ldg(a.colterm + (size_t)col * a.colterm_stride) : 0.f) : inf;
            }
            __syncwarp();
            if (!mbar_wait(tfull_bar(buf), uph, abort_flag, a.err)) { dead = true; break; }
            tc_fence_after();
#pragma unroll
            for (int g = 0; g < (PAIR ? 2 : 1); ++g) {
                if (g >= mcount) break;
                const int row = (m0 + g) * GBM + q4 * 32 + lane;
                const uint32_t taddr = tmem_base + ((uint32_t)(q4 * 32) << 16) +
                                       (uint32_t)((PAIR ? g : buf) * GBN + half * G_HALF);
                if (a.mode == 0) {
                    if (neg1)
                        epilogue_select<NK, true>(taddr, cnu, a.alpha, (uint32_t)colb, a.ncols, lists[g], tau[g], cnt[g],
                                                  a.nsel, nkeep, lane);
                    else
                        epilogue_select<NK, false>(taddr, cnu, a.alpha, (uint32_t)colb, a.ncols, lists[g], tau[g], cnt[g],
                                                   a.nsel, nkeep, lane);
                } else {
                    epilogue_store(taddr, cnu, a.alpha, row, a.nrows, a.ncols, colb, a.scores);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (TWO && crank != 0) mbar_arrive_cluster(mapa_shared(tempty_bar(buf), 0));
                else mbar_arrive(tempty_bar(buf));
            }
        }
        if (a.mode == 0 && !dead) {
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                const int r = (m0 + g) * GBM + q4 * 32 + lane;
                if (g < mcount && r < a.nrows) a.cand_cnt[((size_t)r * nsplit + split) * GEMM_COL_HALVES + half] = cnt[g];
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (TWO) cluster_sync_all();  // neither CTA's tensor memory or barriers go away while the other may still use them
    if (warp == 0) {
        tc_fence_after();
        if (*abort_flag) __nanosleep(100000);  // let copies / MMAs in flight drain after a timed-out wait
        if (TWO) tmem_dealloc_pair(tmem_base, G_TMEM_COLS); else tmem_dealloc(tmem_base, G_TMEM_COLS);
    }
}

// ---- host side ----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map of a row-major bf16 matrix [rows][cols] read in boxes of box_rows x 64 columns, 128-byte swizzle.
// row_stride (in elements, a multiple of 8, >= cols) lets the map pick every n-th row of a larger matrix.
cudaError_t make_tmap_bf16(void* out_map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
                           uint64_t row_stride) {
    if (row_stride == 0) row_stride = cols;
    // A map is a pure function of these five values.  A search loop asks for the same few maps call after call
    // (the query operand in the caller's workspace, the flat database): the last ones each thread asked for are
    // kept, so a repeated call encodes nothing.
    struct Slot { const void* ptr; uint64_t rows, cols, stride; uint32_t box; bool used; alignas(64) unsigned char map[128]; };
    constexpr int NSLOT = 8;
    static thread_local Slot slots[NSLOT];
    static thread_local int next_slot = 0;
    for (int i = 0; i < NSLOT; ++i) {
        const Slot& c = slots[i];
        if (c.used && c.ptr == ptr && c.rows == rows && c.cols == cols && c.stride == row_stride && c.box == box_rows) {
            std::memcpy(out_map, c.map, 128);
            return cudaSuccess;
        }
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return cudaErrorNotSupported;
    if (rows == 0 || cols == 0 || (row_stride * 2) % 16 != 0 || row_stride < cols ||
        reinterpret_cast<uintptr_t>(ptr) % 16 != 0)
        return cudaErrorInvalidValue;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride * 2};
    const cuuint32_t box[2] = {GBK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    Slot& c = slots[next_slot];
    c.used = false;
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(c.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr),
                    dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    c.ptr = ptr; c.rows = rows; c.cols = cols; c.stride = row_stride; c.box = box_rows; c.used = true;
    next_slot = (next_slot + 1) % NSLOT;
    std::memcpy(out_map, c.map, 128);
    return cudaSuccess;
}

int gemm_cand_cap(int nsel) { return nsel <= GEMM_CAP_SMALL - 128 ? GEMM_CAP_SMALL : (nsel <= GEMM_CAP_LARGE - 64 ? GEMM_CAP_LARGE : 0); }

// Grid shape and main loop.  *mg: 1 = one row tile per CTA (LOOP_SINGLE), 2 = two row tiles per CTA sharing each B
// tile (LOOP_PAIR), 3 = two row tiles per CTA PAIR (LOOP_TWO_CTA: a cluster of two CTAs shares each B tile).
// Batches of more than 128 rows take the CTA pair.  Measured on the two big contractions (ms, same box):
//                                        single   pair in a CTA   CTA pair
//   flat search, B = 20 GB from HBM       5.74        5.27        4.7 - 5.2 (power-capped to 1.2 - 1.6 GHz)
//   Hyperscale coarse stage, B in L2      0.410       0.464       0.401
// The in-CTA pair saves the same operand traffic as the CTA pair but cannot overlap its epilogue; it is kept as a
// measured alternative that the test hook reaches.  *nsplit = column ranges; *mgroups = grid rows.
static int g_pairing = 0;  // 0: as above, 1: LOOP_SINGLE, 2: LOOP_PAIR, 3: LOOP_TWO_CTA (2, 3: batches with two row tiles)
void gemm_set_pairing(int mode) { g_pairing = mode; }
void gemm_grid(int nrows, int64_t ncols, int d, int num_sms, int* mg, int* nsplit, int* mgroups) {
    const int mtiles = (nrows + GBM - 1) / GBM;
    const int64_t ntiles = (ncols + GBN - 1) / GBN;
    int loop = 1;
    if (mtiles >= 2) {
        if (g_pairing == 2 || g_pairing == 3) loop = g_pairing;
        else if (g_pairing == 0) loop = 3;
    }
    const int groups = loop == 1 ? mtiles : (mtiles + 1) / 2;
    int64_t split = (loop == 3 ? num_sms / 2 : num_sms) / groups;  // a CTA pair occupies two SMs
    if (split < 1) split = 1;
    if (split > ntiles) split = ntiles;
    *mg = loop;
    *nsplit = (int)split;
    *mgroups = groups;
}


cudaError_t launch_gemm_select(const GemmLaunch& L, cudaStream_t s) {
    GemmArgs a;
    a.nrows = L.nrows; a.ncols = (int)L.ncols;
    a.a_part_rows = L.a_part_rows; a.b_part_rows = (int)L.b_part_rows;
    a.kblocks = (L.d + GBK - 1) / GBK;
    a.nterms = L.nterms;
    for (int t = 0; t < 6; ++t) { a.term_a[t] = L.term_a[t]; a.term_b[t] = L.term_b[t]; }
    a.mtiles = (L.nrows + GBM - 1) / GBM;
    a.ntiles = (int)((L.ncols + GBN - 1) / GBN);
    a.alpha = L.alpha; a.colterm = L.colterm; a.colterm_stride = L.colterm_stride > 0 ? L.colterm_stride : 1;
    a.row_tau = L.row_tau;
    a.mode = L.mode; a.nsel = L.nsel;
    a.cand = L.cand; a.cand_cnt = L.cand_cnt; a.scores = L.scores; a.err = L.err;
    const CUtensorMap* ma = reinterpret_cast<const CUtensorMap*>(L.tmap_a);
    const CUtensorMap* mb = reinterpret_cast<const CUtensorMap*>(L.mg == 3 ? L.tmap_b_half : L.tmap_b);
    const bool large = L.mode == 0 && L.cap == GEMM_CAP_LARGE;
    const int groups = L.mg == 1 ? a.mtiles : (a.mtiles + 1) / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L.mg == 3 ? 2 * L.nsplit : L.nsplit, groups);
    cfg.blockDim = dim3(G_THREADS);
    cfg.dynamicSmemBytes = G_SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    if (L.mg == 3) {  // the two CTAs of a pair are neighbours in x
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
    cudaError_t e;
#define RAGO_GEMM_LAUNCH(NKV, LOOPV) e = cudaLaunchKernelEx(&cfg, gemm_select_kernel<NKV, LOOPV>, *ma, *mb, a)
    if (large) {
        if (L.mg == 3) RAGO_GEMM_LAUNCH(GEMM_CAP_LARGE / 32, LOOP_TWO_CTA);
        else if (L.mg == 2) RAGO_GEMM_LAUNCH(GEMM_CAP_LARGE / 32, LOOP_PAIR);
        else RAGO_GEMM_LAUNCH(GEMM_CAP_LARGE / 32, LOOP_SINGLE);
    } else {
        if (L.mg == 3) RAGO_GEMM_LAUNCH(GEMM_CAP_SMALL / 32, LOOP_TWO_CTA);
        else if (L.mg == 2) RAGO_GEMM_LAUNCH(GEMM_CAP_SMALL / 32, LOOP_PAIR);
        else RAGO_GEMM_LAUNCH(GEMM_CAP_SMALL / 32, LOOP_SINGLE);
    }
#undef RAGO_GEMM_LAUNCH
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- pilot thresholds: per row, a value with at least nsel of the row's n sample scores at or below it --------
// One CTA per row: the row is read once (as ordered score bits), then bisected between its minimum and maximum
// with CTA-wide counts; the search stops as soon as the count lies in [nsel, nsel + nsel/4] and returns the next
// representable value above the cut, so that "score < tau" keeps ties of the cut itself.
// A row that fits the registers and gives every warp enough values is not bisected CTA-wide: each of the W warps
// bisects its own share for a value with at least ceil(nsel / W) of its values at or below it (warp-wide counts,
// no barrier), and the row's threshold is the largest of the W values: at least nsel sample scores lie at or below
// it, which is all a threshold has to guarantee; it is a little looser than the sample's exact nsel-th smallest.
constexpr int RT_THREADS = 256;
constexpr int RT_REG = 16;  // values a thread keeps in registers (rows of up to RT_REG * RT_THREADS scores)
template <bool IN_REGS>
__global__ void __launch_bounds__(RT_THREADS) row_tau_kernel(const float* __restrict__ scores, int n, int nsel,
                                                             float* __restrict__ row_tau) {
    extern __shared__ uint32_t rt_vals[];  // [n] when the row does not fit the registers
    __shared__ uint32_t red[2][RT_THREADS / 32];
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* r = scores + (size_t)row * n;
    uint32_t mine[RT_REG];
    uint32_t mn = 0xFFFFFFFFu, mx = 0u;
    if (IN_REGS) {
#pragma unroll
        for (int j = 0; j < RT_REG; ++j) {
            const int i = tid + j * RT_THREADS;
            mine[j] = i < n ? f32_orderable(__ldg(r + i)) : 0xFFFFFFFFu;
            if (i < n) { mn = mine[j] < mn ? mine[j] : mn; mx = mine[j] > mx ? mine[j] : mx; }
        }
    } else {
        for (int i = tid; i < n; i += RT_THREADS) {
            const uint32_t o = f32_orderable(__ldg(r + i));
            rt_vals[i] = o;
            mn = o < mn ? o : mn;
            mx = o > mx ? o : mx;
        }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (IN_REGS) {
        constexpr int W = RT_THREADS / 32;
        const int m = (nsel + W - 1) / W;
        // values are dealt out round-robin by thread: the last warp holds the fewest
        const int fewest = (n / RT_THREADS) * 32 + (n % RT_THREADS > RT_THREADS - 32 ? n % RT_THREADS - (RT_THREADS - 32) : 0);
        if (fewest >= m) {  // uniform
            uint32_t nv = 0;
#pragma unroll
            for (int j = 0; j < RT_REG; ++j) nv += tid + j * RT_THREADS < n ? 1u : 0u;
            uint32_t c_hi = __reduce_add_sync(0xffffffffu, nv);
            long long lo = (long long)mn - 1, hi = mx;  // #(<= lo) < m <= #(<= hi), within the warp
            const uint32_t want_max = (uint32_t)(m + m / 4);
            while (hi - lo > 1 && c_hi > want_max) {  // uniform within the warp
                const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
                uint32_t c = 0;
#pragma unroll
                for (int j = 0; j < RT_REG; ++j) c += mine[j] <= mid ? 1u : 0u;  // padding holds the largest pattern
                c = __reduce_add_sync(0xffffffffu, c);
                if (c < (uint32_t)m) lo = mid; else { hi = mid; c_hi = c; }
            }
            if (lane == 0) red[0][warp] = (uint32_t)hi;
            __syncthreads();
            if (tid == 0) {
                uint32_t T = red[0][0];
                for (int w = 1; w < W; ++w) T = red[0][w] > T ? red[0][w] : T;
                row_tau[row] = T == 0xFFFFFFFFu ? orderable_f32(T) : orderable_f32(T + 1u);
            }
            return;
        }
    }
    if (lane == 0) { red[0][warp] = mn; red[1][warp] = mx; }
    __syncthreads();
    mn = red[0][0]; mx = red[1][0];
    for (int w = 1; w < RT_THREADS / 32; ++w) {
        mn = red[0][w] < mn ? red[0][w] : mn;
        mx = red[1][w] > mx ? red[1][w] : mx;
    }
    __syncthreads();
    long long lo = (long long)mn - 1, hi = mx;  // #(<= lo) < nsel <= #(<= hi)
    uint32_t c_hi = (uint32_t)n;
    const uint32_t want_max = (uint32_t)(nsel + nsel / 4);
    int round = 0;
    while (hi - lo > 1 && c_hi > want_max) {  // uniform: every thread holds the same lo, hi, c_hi
        const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
        uint32_t c = 0;
        if (IN_REGS) {
#pragma unroll
            for (int j = 0; j < RT_REG; ++j) c += mine[j] <= mid ? 1u : 0u;  // padding holds the largest pattern
        } else {
            for (int i = tid; i < n; i += RT_THREADS) c += rt_vals[i] <= mid ? 1u : 0u;
        }
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) red[round & 1][warp] = c;  // the other buffer may still be read by slower warps
        __syncthreads();
        c = 0;
        for (int w = 0; w < RT_THREADS / 32; ++w) c += red[round & 1][w];
        if (c < (uint32_t)nsel) lo = mid; else { hi = mid; c_hi = c; }
        ++round;
    }
    if (tid == 0) {
        const uint32_t T = (uint32_t)hi;
        row_tau[row] = T == 0xFFFFFFFFu ? orderable_f32(T) : orderable_f32(T + 1u);
    }
}
cudaError_t launch_row_tau(const float* scores, int nrows, int n, int nsel, float* row_tau, cudaStream_t s) {
    if (n <= RT_REG * RT_THREADS) {
        row_tau_kernel<true><<<nrows, RT_THREADS, 0, s>>>(scores, n, nsel, row_tau);
    } else {
        if ((size_t)n * 4 > 200 * 1024) return cudaErrorInvalidValue;
        row_tau_kernel<false><<<nrows, RT_THREADS, (size_t)n * 4, s>>>(scores, n, nsel, row_tau);
    }
    count_launch();
    return cudaGetLastError();
}

// Per-device set-up: the kernels' dynamic shared-memory limits (called at index load and by the flat search).
template <int NKV, int LOOPV>
static cudaError_t gemm_attr() {
    return cudaFuncSetAttribute(gemm_select_kernel<NKV, LOOPV>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES);
}
cudaError_t gemm_select_init() {
    cudaError_t e = gemm_attr<GEMM_CAP_SMALL / 32, LOOP_SINGLE>();
    if (e == cudaSuccess) e = gemm_attr<GEMM_CAP_SMALL / 32, LOOP_PAIR>();
    if (e == cudaSuccess) e = gemm_attr<GEMM_CAP_SMALL / 32, LOOP_TWO_CTA>();
    if (e == cudaSuccess) e = gemm_attr<GEMM_CAP_LARGE / 32, LOOP_SINGLE>();
    if (e == cudaSuccess) e = gemm_attr<GEMM_CAP_LARGE / 32, LOOP_PAIR>();
    if (e == cudaSuccess) e = gemm_attr<GEMM_CAP_LARGE / 32, LOOP_TWO_CTA>();
    if (e == cudaSuccess)  // rows of up to 51 200 pilot scores in shared memory
        e = cudaFuncSetAttribute(row_tau_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

// ---- self-test of the bounded waits ---------------------------------------------------------------
// One CTA, two warps, the roles of the kernels above in miniature.  Lane 0 of warp 0 waits, through the same
// mbar_wait the kernels use, on a barrier that nothing ever arrives at, with a poll limit of the caller's choice:
// the wait runs out, sets the CTA's abort flag and the error word.  Lane 0 of warp 1 waits on a second such
// barrier with the full limit and must be released early by the abort flag (the hand-off that lets every role
// of a kernel leave its loop after one of them timed out).  With with_tmem the CTA holds all 512 TMEM columns
// meanwhile and gives them back before it exits, as gemm_select_kernel does after an abort.  Nothing traps,
// faults or spins without a limit: the kernel ends normally.
// observed[0] = 1 if the first wait gave up, observed[1] = 1 if the second was released by the abort flag.
__global__ void __launch_bounds__(64, 1) selftest_wait_kernel(uint32_t* err_word, uint32_t max_polls, int with_tmem,
                                                              uint32_t* observed) {
    __shared__ unsigned long long bars[2];
    __shared__ uint32_t tmem_slot;
    __shared__ uint32_t abort_word;
    volatile uint32_t* abort_flag = &abort_word;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_word = 0;
        fence_barrier_init();
    }
    if (with_tmem && warp == 0) tmem_alloc(smem_u32(&tmem_slot), G_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (lane == 0) {
        if (warp == 0) {
            const bool ok = mbar_wait(smem_u32(&bars[0]), 0u, abort_flag, err_word, 0, max_polls);
            observed[0] = ok ? 0u : 1u;
        } else {
            // given the first warp's limit of max_polls polls of at most 4 us, this one must not need its own
            const bool ok = mbar_wait(smem_u32(&bars[1]), 0u, abort_flag, err_word, 0, MBAR_MAX_POLLS);
            observed[1] = (!ok && *abort_flag) ? 1u : 0u;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (with_tmem && warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_slot, G_TMEM_COLS);
    }
}
cudaError_t launch_selftest_wait(uint32_t* err_word, uint32_t max_polls, int with_tmem, uint32_t* observed, cudaStream_t s) {
    selftest_wait_kernel<<<1, 64, 0, s>>>(err_word, max_polls, with_tmem, observed);
    count_launch();
    return cudaGetLastError();
}

// ---- fp32 -> stacked bf16 parts: out[p][i] = bf16 part p of x[i] ---------------------------------
__global__ void split_bf16_kernel(const float* __restrict__ x, size_t n, int parts, __nv_bfloat16* __restrict__ out) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float r = x[i];
        for (int p = 0; p < parts; ++p) {
            const __nv_bfloat16 h = __float2bfloat16_rn(r);
            out[(size_t)p * n + i] = h;
            r -= __bfloat162float(h);
        }
    }
}
cudaError_t launch_split_bf16(const float* x, size_t n, int parts, void* out, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    const size_t want = (n + 255) / 256;
    const int blocks = (int)(want < 148 * 8 ? want : 148 * 8);
    split_bf16_kernel<<<blocks, 256, 0, s>>>(x, n, parts, static_cast<__nv_bfloat16*>(out));
    count_launch();
    return cudaGetLastError();
}

}  // namespace rago
