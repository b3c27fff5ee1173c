// Lookup-table construction + asymmetric-distance scan of the probed inverted lists.
//
// One persistent CTA per SM walks a contiguous, equally sized share of the batch's code tiles
// (pairs (query, probed list) in probe order, each list cut into tiles of TV vectors).  A producer
// warp streams code tiles global -> shared with 1-D bulk copies (cp.async.bulk + mbarrier, a ring of
// S tiles in flight, the tiles two steps further down the list prefetched into L2); consumer warps
// build the lookup table of the current QUERY in shared memory (or, for small batches, fetch the
// image a kernel before the scan has built), then every lane owns one (virtual) code row of the tile
// and sums table entries.
//
// Score, smaller is better for both metrics:
//   inner product:  -<q, c_p>  +  sum_m -<q_m, cw_m>
//   squared L2:     ||q - c_p||^2  +  (||r||^2 + 2<c_p, r>)  +  sum_m -2<q_m, cw_m>      (r = decoded residual)
// i.e. bias(q, list) + term(vector) + sum of entries of a table that depends on the query only, so a
// table is rebuilt when the query changes, not at every probed list.  The expansion costs a few ulps
// of the largest term (see vector_terms_kernel); results agree with the direct form to ~1e-6 relative
// on data whose residuals are not tiny against the centroid distances.  The per-vector terms of a tile
// travel with it (a second bulk copy on the same barrier).
//
// Shared-memory access pattern.  A code row is read as 32-bit words; at step (blk, il, t) lane L
// reads word  blk*G + (il ^ a(L))  and uses byte  t ^ b(L)  of it, so that within any one
// instruction the 32 lanes touch 32 different banks both for the code words (rows are M bytes
// apart) and for the table (bank = table column mod 32).  Rows wider than 32*odd bytes are split
// into R "virtual rows" handled by adjacent lanes and summed with a shuffle; sub-space counts that
// are 16 mod 32 keep two table copies so lanes L and L^4 never collide.
//
// Table addressing.  Per code byte the inner loop spends one byte-permute, one shared load and one
// add: the table is stored as 64-column banks of 256 rows x 256 bytes that start at a shared-memory
// address which is a multiple of 64 KB, so the load address  (bank << 16) | (code << 8) | column*4
// is assembled by a single PRMT from the code word and a per-lane constant.  Tables wider than two
// banks (M = 80 with its two copies) fall back to a multiply-add address.
//
// Fixed-point table.  Entries are stored as 32-bit integers scaled by a per-query power of two chosen
// so that a sum of M entries cannot overflow (|sum| < 2^30): the scan then adds two entries per
// instruction (a three-input integer add) and the sum is exact, so it does not depend on the order of
// the additions; it is converted back to fp32 once per vector.  The quantisation step is
// max|entry| * M / 2^30, i.e. an absolute error below max|entry| * M^2 / 2^31 per vector (2e-5 for
// M = 96 and entries of size 5), far inside the 1e-4 relative bar.
//
// Candidates better than the running threshold go to a shared buffer (topk.cuh).  The producer warp
// watches the buffer count and marks a tile "cut first" when the tiles in flight could overflow it; a
// cut is a CTA-wide bisection on the ordered score bits that keeps the k best keys and a few more (one
// barrier per step), and the exact k best are sorted once, when the CTA leaves the query.  The
// threshold of a query is shared between CTAs through global memory, which only ever removes keys that
// cannot be among the k best, so the result does not depend on timing.
//
// A warp works on RGW row groups of 32 (virtual) rows per tile, unrolled, so that several independent
// chains code word -> address -> table entry are in flight per warp; with R lanes per vector one
// epilogue (term, bias, key, push) serves R row groups.
#include <type_traits>

#include "topk.cuh"
#include "plan.cuh"

namespace rago {

constexpr int MAX_STAGES = 4;
constexpr int SCAN_PF = 2;                  // tiles ahead of the one being copied that are prefetched into L2 (measured: 1-2 best)
// Prefetch of a contiguous global range into L2 (16-byte aligned start, size a multiple of 16 bytes).
__device__ __forceinline__ void l2_prefetch(const void* g, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(g), "r"(bytes) : "memory");
}
constexpr int SMEM_OPTIN = 227 * 1024;          // dynamic shared memory asked for (the sm_100 per-block limit)
constexpr uint32_t SMEM_BASE_EXPECTED = 1024;   // shared-window address of dynamic shared memory when the kernel has no static part
constexpr int CTRL_BYTES = 1024;

struct TileDesc {
    int32_t pair;      // index into probe_list (query * nprobe + rank)
    float term;        // the pair's (query, list) term of the score
    uint32_t pos0;     // storage position of the tile's first vector
    int32_t nvec;      // vectors in this tile
    int32_t newpair;   // bit 0: first tile of this pair inside this CTA; bit 1: cut the candidate buffer before this tile
    int32_t vrem;      // index of the first vector's term inside the staged term block (0..3)
    uint32_t tile_addr;  // shared address of the stage's code tile
    uint32_t vt_addr;    // shared address of the stage's per-vector terms
};

struct ScanArgs {
    const uint8_t* codes;
    const int64_t* list_offsets;
    const int32_t* probe_list;
    const float* probe_term;
    const float* queries;
    const float* cbT;
    const float* vterm;  // [N + 4] per-vector term (L2), null for inner product
    const int64_t* work_prefix;
    unsigned long long* qthresh;
    int32_t* slot_cnt;
    unsigned long long* slot_keys;
    uint32_t* err;
    const uint8_t* lut_img;  // [nq][LUT_BYTES] tables built ahead of the scan (small batches), or null
    const float* lut_inv;    // [nq] fp32 value of one integer unit of each such table
    int32_t npairs, nprobe, d, dsub, metric, k, stages;
    int32_t stream_once;     // the batch is small: code tiles are fetched with an evict-first hint, so that the centroid
                             // table the next search's coarse step reads stays in L2
    uint32_t dyn_bytes;
};

template <int WV, int G, int R, int NCW_, int RGW_>
struct Cfg {
    static constexpr int NCW = NCW_;                    // consumer warps
    static constexpr int NCT = NCW * 32;                // consumer threads
    static constexpr int THREADS = NCT + 32;            // + one producer warp
    static constexpr int MV = WV * 4;                   // bytes per virtual row
    static constexpr int M = MV * R;                    // code bytes per vector
    static constexpr int NBLK = WV / G;                 // blocks of G words per virtual row
    static constexpr int COPIES = G == 4 ? 2 : 1;
    static constexpr int COPY_OFF = COPIES == 1 ? 0 : (M == 16 ? 16 : (M == 48 ? 80 : M));  // 16 mod 32
    static constexpr int NCOLS = COPIES == 1 ? M : COPY_OFF + M;
    static constexpr bool BANKED = NCOLS <= 128;        // PRMT addressing
    static constexpr int NBANK = (NCOLS + 63) / 64;
    static constexpr int LSTRIDE = NCOLS;               // words per table row (multiply-add addressing)
    static constexpr int LUT_BYTES = BANKED ? NBANK * 65536 : KSUB * LSTRIDE * 4;
    static constexpr int RGW = RGW_;                    // 32-row groups per warp per tile (unrolled: independent work in flight)
    static constexpr int TILE_VROWS = NCW * 32 * RGW;
    static constexpr int TV = TILE_VROWS / R;           // vectors per tile
    static constexpr int TILE_BYTES = TILE_VROWS * MV;
    static constexpr int VT_BYTES = (TV + 4) * 4;       // staged per-vector terms (start rounded down to 16 bytes)
    static constexpr int KCAP = LUT_BYTES <= 65536 ? 2 * TOPK_CAP : TOPK_CAP;  // keys of the CTA's candidate buffer
    // Banked tables start at this absolute shared address (a multiple of 64 KB).  Two tiles of more than 48 KB do not
    // fit above a table at 64 KB, so configurations with such tiles keep their tiles below a table at 128 KB.
    static constexpr uint32_t LUT_WINDOW = (NBANK == 1 && TILE_BYTES > 48 * 1024) ? 0x20000u : 0x10000u;
    static_assert(WV % G == 0, "virtual rows are whole blocks");
    static_assert(TILE_VROWS % R == 0, "tile must hold whole vectors");
    static_assert(RGW % (R < RGW ? R : RGW) == 0, "row groups are taken min(R, RGW) at a time");
    // The producer asks for a cut of the candidate buffer when the count it sees plus everything the tiles in
    // flight can still push would not fit; SMAX bounds the ring depth so that this leaves room to work in.
    static constexpr int SMAX = KCAP / TV / 2 < MAX_STAGES ? KCAP / TV / 2 : MAX_STAGES;
    static_assert(SMAX >= 2, "two tiles in flight must fit the candidate buffer twice over");
    static_assert(MAX_K + SMAX * TV <= KCAP, "k kept keys plus the pushes of all tiles in flight must fit");
    static_assert(COPY_OFF % 32 == (COPIES == 2 ? 16 : 0), "second copy must sit 16 banks away");
    static_assert(LSTRIDE % 32 == 0 || BANKED, "table rows must keep bank = column mod 32");
    static_assert(VT_BYTES % 16 == 0 && TILE_BYTES % 16 == 0, "bulk-copy destinations are 16-byte granular");
    // banked addressing: the columns one lane touches in one block stay inside one 64-column bank
    __host__ __device__ static constexpr bool banked_ok() {
        for (int copy = 0; copy < COPIES; ++copy)
            for (int sr = 0; sr < R; ++sr)
                for (int blk = 0; blk < NBLK; ++blk) {
                    const int cb = copy * COPY_OFF + sr * MV;
                    if ((cb % 64) + ((blk * 4 * G) % 64) + 4 * G > 64) return false;
                }
        return true;
    }
    static_assert(!BANKED || banked_ok(), "a lane's columns of one block straddle two banks");
    // address of table entry (code j, column col) relative to the table's start
    __host__ __device__ static constexpr uint32_t lut_off(int j, int col) {
        return BANKED ? (uint32_t)(col / 64) * 65536u + (uint32_t)j * 256u + (uint32_t)(col % 64) * 4u
                      : ((uint32_t)j * LSTRIDE + (uint32_t)col) * 4u;
    }
    // immediate added for block blk (banked addressing)
    __host__ __device__ static constexpr uint32_t blk_imm(int blk) {
        return (uint32_t)((blk * 4 * G) / 64) * 65536u + (uint32_t)((blk * 4 * G) % 64) * 4u;
    }
};

// Absolute shared-memory addresses of everything the kernel keeps there.  The same function runs on
// the host (to choose the number of stages, with the expected window base) and in the kernel (with
// the real base); a plan that does not fit makes the kernel report an error and return.
struct SmemPlan {
    uint32_t lut, ctrl, keys, rT, vt[MAX_STAGES], tile[MAX_STAGES];
    int ok;
};

template <class C>
__host__ __device__ inline SmemPlan plan_smem(uint32_t base, uint32_t dyn_bytes, int d, int stages, bool need_vt) {
    SmemPlan p;
    p.ok = 1;
    const uint32_t end = base + dyn_bytes;
    uint32_t lo_cur, lo_end, hi_cur;
    if (C::BANKED) {
        p.lut = C::LUT_WINDOW;
        if (base > C::LUT_WINDOW) p.ok = 0;
        lo_cur = base; lo_end = C::LUT_WINDOW; hi_cur = C::LUT_WINDOW + C::LUT_BYTES;
    } else {
        p.lut = (base + 127u) & ~127u;
        lo_cur = lo_end = 0; hi_cur = p.lut + C::LUT_BYTES;
    }
    if (hi_cur > end) p.ok = 0;
    auto take = [&](uint32_t bytes, uint32_t align) -> uint32_t {
        uint32_t a = (lo_cur + align - 1) & ~(align - 1);
        if (a + bytes <= lo_end) { lo_cur = a + bytes; return a; }
        a = (hi_cur + align - 1) & ~(align - 1);
        if (a + bytes <= end) { hi_cur = a + bytes; return a; }
        p.ok = 0;
        return base;
    };
    // largest pieces first, each below the table if it fits there, else above it
    for (int s = 0; s < MAX_STAGES; ++s) p.tile[s] = s < stages ? take(C::TILE_BYTES, 128) : base;
    p.keys = take(C::KCAP * 8, 16);
    for (int s = 0; s < MAX_STAGES; ++s) p.vt[s] = (s < stages && need_vt) ? take(C::VT_BYTES, 16) : base;
    // The scaled, transposed query is only alive while a table is built, when the candidate buffer is empty: it
    // shares the buffer's space when it fits there.
    p.rT = (uint32_t)d * 4 <= (uint32_t)C::KCAP * 8 ? p.keys : take((uint32_t)d * 4, 16);
    p.ctrl = take(CTRL_BYTES, 16);
    return p;
}

// Control block.
constexpr int WARP_CUT_MAX = 1024;  // buffer cuts of at most this many keys, for k of at most WARP_CUT_K, are made by one warp
constexpr int WARP_CUT_K = 32;      // (a larger k needs bisection rounds, which the whole CTA does faster)
struct Ctrl {
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long cbar;  // consumer barrier
    unsigned long long lutbar;  // a prebuilt table has landed
    TileDesc desc[MAX_STAGES];
    int cnt;
    uint32_t abort_flag;
    float red[32];  // per-warp maxima of the table build
    uint32_t redu[2][32];  // per-warp minima / maxima / counts of the buffer cut
};
static_assert(sizeof(Ctrl) <= CTRL_BYTES, "control block too large");

template <int IMM>
__device__ __forceinline__ float lds_f32_imm(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(IMM));
    return v;
}
template <int IMM>
__device__ __forceinline__ uint32_t lds_u32_imm(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(IMM));
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Table construction by the consumer threads.  Entry e = j * M + m of the transposed codebook is
// DSUB contiguous floats; consecutive threads take consecutive entries (coalesced loads, and table
// stores that walk the banks).  UNR entries per thread are loaded before any is used so that enough
// requests are in flight to cover the L2 latency.
template <class C, int D4>
__device__ __forceinline__ float build_table(const float* __restrict__ cbT, const float* rT, uint32_t lut, int ctid) {
    float mx = 0.f;
    constexpr int UNR = D4 >= 3 ? 4 : 8;
    constexpr int TOTAL = KSUB * C::M;
    for (int e0 = ctid; e0 < TOTAL; e0 += C::NCT * UNR) {
        float4 cv[UNR][D4];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int e = e0 + u * C::NCT;
#pragma unroll
            for (int i = 0; i < D4; ++i)
                cv[u][i] = e < TOTAL ? __ldg(reinterpret_cast<const float4*>(cbT + (size_t)e * (D4 * 4)) + i)
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int e = e0 + u * C::NCT;
            if (e >= TOTAL) break;
            const int j = e / C::M, m = e - j * C::M;
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < D4; ++i) {
                acc = fmaf(rT[(4 * i + 0) * C::M + m], cv[u][i].x, acc);
                acc = fmaf(rT[(4 * i + 1) * C::M + m], cv[u][i].y, acc);
                acc = fmaf(rT[(4 * i + 2) * C::M + m], cv[u][i].z, acc);
                acc = fmaf(rT[(4 * i + 3) * C::M + m], cv[u][i].w, acc);
            }
            sts_f32(lut + C::lut_off(j, m), acc);
            mx = fmaxf(mx, fabsf(acc));
        }
    }
    return mx;
}
template <class C>
__device__ __forceinline__ float build_table_any(const float* __restrict__ cbT, const float* rT, uint32_t lut,
                                                int ctid, int dsub) {
    float mx = 0.f;
    for (int e = ctid; e < KSUB * C::M; e += C::NCT) {
        const int j = e / C::M, m = e - j * C::M;
        float acc = 0.f;
        for (int t = 0; t < dsub; ++t) acc = fmaf(rT[t * C::M + m], __ldg(cbT + (size_t)e * dsub + t), acc);
        sts_f32(lut + C::lut_off(j, m), acc);
        mx = fmaxf(mx, fabsf(acc));
    }
    return mx;
}
// Second pass of the table build: every thread turns the fp32 entries it wrote itself into scaled
// integers (and fills the second copy where the layout keeps one).
template <class C>
__device__ __forceinline__ void quantise_table(uint32_t lut, int ctid, float scale) {
    for (int e = ctid; e < KSUB * C::M; e += C::NCT) {
        const int j = e / C::M, m = e - j * C::M;
        const uint32_t addr = lut + C::lut_off(j, m);
        const int q = __float2int_rn(lds_f32(addr) * scale);
        sts_f32(addr, __int_as_float(q));
        if (C::COPIES == 2) sts_f32(lut + C::lut_off(j, C::COPY_OFF + m), __int_as_float(q));
    }
}

// Code words of one virtual row, all loaded before the first look-up (look-up addresses depend on them,
// so loading block by block would expose the shared-memory latency once per block).
// wa[il] is the lane's address of word (il ^ a(L)) of its row in the tile's first row group of this warp; OFF is
// the byte offset of the row group being read, a compile-time constant that ends up in the load's immediate.
template <class C, int G, int BLK, int OFF>
struct LoadWords {
    __device__ __forceinline__ static void run(const uint32_t (&wa)[G], uint32_t (&x)[C::NBLK][G]) {
#pragma unroll
        for (int il = 0; il < G; ++il) x[BLK][il] = lds_u32_imm<OFF + BLK * G * 4>(wa[il]);
        if constexpr (BLK + 1 < C::NBLK) LoadWords<C, G, BLK + 1, OFF>::run(wa, x);
    }
};

// One block (G code words = 4G sub-spaces) of one virtual row: 4G look-ups, written as three passes over
// half a block (all addresses, all loads, all adds).
template <class C, int G, int BLK>
__device__ __forceinline__ void scan_block(const uint32_t (&x)[G], const uint32_t (&cc)[G][2], const uint32_t (&sel)[4],
                                           const uint32_t (&lo)[G][4], uint32_t lut, int (&acc)[4]) {
    constexpr int H = G / 2;
#pragma unroll
    for (int h0 = 0; h0 < G; h0 += H) {
        uint32_t ad[H][4];
        uint32_t vv[H][4];
#pragma unroll
        for (int i = 0; i < H; ++i)
#pragma unroll
            for (int t = 0; t < 4; ++t)
                ad[i][t] = C::BANKED ? __byte_perm(x[h0 + i], cc[h0 + i][t >> 1], sel[t])
                                     : lut + __byte_perm(x[h0 + i], 0u, sel[t]) * (uint32_t)(C::LSTRIDE * 4) + lo[h0 + i][t];
#pragma unroll
        for (int i = 0; i < H; ++i)
#pragma unroll
            for (int t = 0; t < 4; ++t)
                vv[i][t] = C::BANKED ? lds_u32_imm<(int)C::blk_imm(BLK)>(ad[i][t]) : lds_u32_imm<BLK * G * 16>(ad[i][t]);
#pragma unroll
        for (int i = 0; i < H; i += 2)  // two entries per add
#pragma unroll
            for (int t = 0; t < 4; ++t) acc[t] = acc[t] + (int)vv[i][t] + (int)vv[i + 1][t];
    }
}
template <class C, int G, int BLK>
struct ScanBlocks {
    __device__ __forceinline__ static void run(const uint32_t (&x)[C::NBLK][G], const uint32_t (&cc)[G][2],
                                               const uint32_t (&sel)[4], const uint32_t (&lo)[G][4], uint32_t lut,
                                               int (&acc)[4]) {
        scan_block<C, G, BLK>(x[BLK], cc, sel, lo, lut, acc);
        if constexpr (BLK + 1 < C::NBLK) ScanBlocks<C, G, BLK + 1>::run(x, cc, sel, lo, lut, acc);
    }
};

template <int WV, int G, int R, int NCW_, int RGW_>
__global__ void __launch_bounds__(Cfg<WV, G, R, NCW_, RGW_>::THREADS, 1) scan_kernel(const ScanArgs a) {
    using C = Cfg<WV, G, R, NCW_, RGW_>;
    constexpr int NCW = C::NCW, NCT = C::NCT;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = a.stages;
    const uint32_t base = smem_u32(smem);
    const SmemPlan P = plan_smem<C>(base, a.dyn_bytes, a.d, S, a.vterm != nullptr);
    if (!P.ok) {  // uniform: every thread sees the same plan
        if (tid == 0) atomicExch(a.err, (uint32_t)ERR_SMEM_LAYOUT);
        return;
    }
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + (P.ctrl - base));
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem + (P.keys - base));
    float* rT = reinterpret_cast<float*>(smem + (P.rT - base));
    volatile uint32_t* abort_flag = &ctrl->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), NCW);
        }
        mbar_init(smem_u32(&ctrl->cbar), NCW);
        mbar_init(smem_u32(&ctrl->lutbar), 1);
        ctrl->cnt = 0;
        ctrl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    __syncthreads();

    // Everything above touched shared memory and kernel arguments only; from here on the kernel reads what the
    // kernels before it wrote.
    grid_dependency_wait();
    grid_dependents_may_launch();
    // A batch of a few queries is latency-bound, and most of a CTA's start-up would be a chain of dependent reads
    // (total, binary search for the first pair, the pair's list, the list's offset) before its first tile can be
    // asked for.  With at most 32 pairs lane i of every warp reads pair i's first unit beside the total, so the
    // first pair follows from one vote; the producer warp reads the rest of every pair's description in the same
    // round trip (the offsets in a second one), and the consumers know their first query without the producer.
    const bool few_pairs = a.npairs <= 32;
    const long long pw = few_pairs ? a.work_prefix[lane < a.npairs ? lane : a.npairs] : 0;  // >= npairs: the total
    int c_list = 0; long long c_off = 0, c_len = 0, c_ws = 0, c_we = 0; float c_term = 0.f;  // producer: lane i's cached pair
    if (few_pairs && warp == NCW && lane < a.npairs) {
        c_list = a.probe_list[lane];
        c_term = a.probe_term[lane];
        c_we = a.work_prefix[lane + 1];
        c_off = a.list_offsets[c_list];
        c_len = a.list_offsets[c_list + 1] - c_off;
    }
    // This CTA's share of the work units (tiles).
    const long long W = a.work_prefix[a.npairs];
    const long long u_begin = (long long)blockIdx.x * W / gridDim.x;
    const long long u_end = (long long)(blockIdx.x + 1) * W / gridDim.x;
    const int T = (int)(u_end - u_begin);
    if (T <= 0) return;
    // few pairs: the pair whose range contains u_begin = the largest p with work_prefix[p] <= u_begin
    const int first_pair = few_pairs ? __popc(__ballot_sync(0xffffffffu, pw <= u_begin)) - 1 : -1;

    if (warp == NCW) {
        // ================= producer warp =================
        // first pair whose range contains u_begin: largest p with work_prefix[p] <= u_begin
        int lo = 0, hi = a.npairs;  // invariant: work_prefix[lo] <= u_begin < work_prefix[hi]
        while (!few_pairs && hi - lo > 1) {  // 32 probes per step, evenly spaced: lane i looks at lo + (i + 1) * step
            const int step = (hi - lo + 31) / 32;
            const int pp = lo + (lane + 1) * step;
            const bool le = pp < hi && a.work_prefix[pp] <= u_begin;
            const int c = __popc(__ballot_sync(0xffffffffu, le));  // the prefix is monotone: the first c probes pass
            const int nhi = lo + (c + 1) * step;
            lo += c * step;
            hi = nhi < hi ? nhi : hi;
        }
        int cache_base = few_pairs ? 0 : lo;  // lane i caches pair cache_base + i
        if (few_pairs) {
            c_ws = pw;
            if (lane >= a.npairs) { c_ws = c_we = W; }
        }
        auto fill = [&]() {
            const int p = cache_base + lane;
            if (p < a.npairs) {
                c_list = a.probe_list[p];
                c_off = a.list_offsets[c_list];
                c_len = a.list_offsets[c_list + 1] - c_off;
                c_ws = a.work_prefix[p];
                c_we = a.work_prefix[p + 1];
                c_term = a.probe_term[p];
            } else {
                c_list = 0; c_off = 0; c_len = 0; c_ws = c_we = W; c_term = 0.f;
            }
        };
        if (!few_pairs) fill();
        int cur = few_pairs ? first_pair : 0;
        const uint64_t once_policy = l2_policy_evict_first();
        long long u = u_begin;
        bool dead = false;
        int issued = 0;
        int pst = 0;          // n % S, kept by counting (S is a run-time value: no division per tile)
        uint32_t pround = 0;  // n / S
        for (int n = 0; n < T && !dead; ++n, ++u) {
            const int st = pst;
            const uint32_t round = pround;
            if (++pst == S) { pst = 0; ++pround; }
            // advance to the pair that owns unit u (skips empty pairs); all of this before the wait for the
            // stage, so that as little as possible stands between a stage coming free and its refill
            for (;;) {
                const long long we = __shfl_sync(0xffffffffu, c_we, cur);
                if (u < we) break;
                if (++cur == 32) { cache_base += 32; fill(); cur = 0; }
            }
            const long long ws = __shfl_sync(0xffffffffu, c_ws, cur);
            const long long off = __shfl_sync(0xffffffffu, c_off, cur);
            const long long len = __shfl_sync(0xffffffffu, c_len, cur);
            const float term = __shfl_sync(0xffffffffu, c_term, cur);
            if (round > 0) dead = !mbar_wait(smem_u32(&ctrl->empty[st]), (round - 1) & 1, abort_flag, a.err);
            if (dead) break;
            if (lane == 0) {
                const long long t_in_pair = u - ws;
                const long long v0 = t_in_pair * C::TV;
                long long nvec = len - v0;
                if (nvec > C::TV) nvec = C::TV;
                const uint32_t pos0 = (uint32_t)(off + v0);
                TileDesc& D = ctrl->desc[st];
                D.pair = cache_base + cur;
                D.term = term;
                D.pos0 = pos0;
                D.nvec = (int32_t)nvec;
                // everything tiles n-S+1 .. n can still push must fit behind what is in the buffer now
                const int cnt_seen = *reinterpret_cast<volatile int*>(&ctrl->cnt);
                const int cut = cnt_seen + (S + 1) * C::TV > C::KCAP ? 2 : 0;
                D.newpair = ((n == 0 || t_in_pair == 0) ? 1 : 0) | cut;
                D.vrem = (int32_t)(pos0 & 3u);
                D.tile_addr = P.tile[st];
                D.vt_addr = P.vt[st];
                const uint32_t bytes = (uint32_t)nvec * C::M;
                // per-vector terms: start rounded down to a 16-byte boundary, length rounded up
                const uint32_t vbytes = a.vterm ? (((pos0 & 3u) + (uint32_t)nvec) * 4u + 15u) & ~15u : 0u;
                const uint32_t bar = smem_u32(&ctrl->full[st]);
                mbar_arrive_expect_tx(bar, bytes + vbytes);
                if (a.stream_once) {  // small batch: the codes are read once and should leave L2 first
                    bulk_g2s_hint(P.tile[st], a.codes + (size_t)pos0 * C::M, bytes, bar, once_policy);
                    if (vbytes) bulk_g2s_hint(P.vt[st], a.vterm + (pos0 & ~3u), vbytes, bar, once_policy);
                } else {
                    bulk_g2s(P.tile[st], a.codes + (size_t)pos0 * C::M, bytes, bar);
                    if (vbytes) bulk_g2s(P.vt[st], a.vterm + (pos0 & ~3u), vbytes, bar);
                }
                // pull the tiles a few steps ahead in this list into L2, so that their copies find them there
                for (int ahead = (t_in_pair == 0 ? 1 : SCAN_PF); ahead <= SCAN_PF; ++ahead) {
                    const long long vp = v0 + (long long)ahead * C::TV;
                    if (vp >= len) break;
                    long long np = len - vp;
                    if (np > C::TV) np = C::TV;
                    l2_prefetch(a.codes + (size_t)(off + vp) * C::M, (uint32_t)np * C::M);
                }
            }
            issued = n + 1;
        }
        if (dead && lane == 0) {
            // let copies already in flight land before the CTA's shared memory goes away
            for (int n = issued > S ? issued - S : 0; n < issued; ++n) {
                const uint32_t bar = smem_u32(&ctrl->full[n % S]);
                for (int it = 0; it < (1 << 16) && !mbar_try_wait(bar, (n / S) & 1); ++it) __nanosleep(64);
            }
        }
        return;
    }

    // ================= consumer warps =================
    const int ctid = tid;  // 0 .. NCT-1
    uint32_t cphase = 0, lphase = 0;
    bool dead = false;
    auto csync = [&]() {
        if (dead) return;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->cbar));
        dead = !mbar_wait(smem_u32(&ctrl->cbar), cphase, abort_flag, a.err);
        cphase ^= 1;
    };

    // lane constants of the access pattern
    const int xa = G == 8 ? (lane >> 2) : (lane >> 3);  // word xor
    const int xb = lane & 3;                            // byte xor
    const int copy = G == 4 ? ((lane >> 2) & 1) : 0;
    const int sr = lane % R;                            // which slice of the vector this lane sums
    const int colbase = copy * C::COPY_OFF + sr * C::MV;
    uint32_t xo[G], cc[G][2], lo[G][4], sel[4];
#pragma unroll
    for (int il = 0; il < G; ++il) {
        xo[il] = (uint32_t)(warp * C::RGW * 32 + lane) * C::MV + 4u * (uint32_t)(il ^ xa);  // offset in a tile of the lane's word il of the warp's first row group
#pragma unroll
        for (int t = 0; t < 4; ++t)
            lo[il][t] = C::BANKED ? 0u : 4u * (uint32_t)(colbase + 4 * (il ^ xa) + (t ^ xb));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            // bytes: column*4 for t = 2h, column*4 for t = 2h+1, table bank, 0
            const uint32_t c0 = 4u * (uint32_t)((colbase % 64) + 4 * (il ^ xa) + ((2 * h) ^ xb));
            const uint32_t c1 = 4u * (uint32_t)((colbase % 64) + 4 * (il ^ xa) + ((2 * h + 1) ^ xb));
            cc[il][h] = c0 | (c1 << 8) | (((P.lut >> 16) + (uint32_t)(colbase / 64)) << 16);
        }
    }
#pragma unroll
    for (int t = 0; t < 4; ++t)
        sel[t] = C::BANKED ? ((uint32_t)(4 + (t & 1)) | ((uint32_t)(t ^ xb) << 4) | 0x7600u)
                           : (0x4440u | (uint32_t)(t ^ xb));

    int cur_q = -1;
    unsigned long long tau = KEY_MAX;
    float bias = 0.f;
    const int k = a.k;
    const bool ip = a.metric == RAGO_IP;
    const float lut_scale = ip ? -1.f : -2.f;
    float inv_scale = 1.f;  // fp32 value of one unit of the current query's integer table

    // Cut the candidate buffer (more than k keys, count stable, called by all consumer threads after a csync and
    // followed by another before the buffer or its count is used again):
    // every thread takes its share of the keys into registers, the CTA bisects on the ordered score bits for a
    // value T with between k and k + k/4 keys at or below it (one barrier per step instead of the ~66 of a full
    // sort), and the keys up to T are pushed back.  All keys of the k best are kept; T bounds the k-th best.
    auto cut_buffer = [&]() {
        constexpr int KPT = (C::KCAP + NCT - 1) / NCT;
        const int n = ctrl->cnt < C::KCAP ? ctrl->cnt : C::KCAP;
        if (n <= WARP_CUT_MAX && k <= WARP_CUT_K) {  // uniform
            // A short buffer and a small k (small batches, mostly): warp 0 alone finds the cut and compacts the buffer in place,
            // with no barrier and no atomic on the way; the others wait once.  For k <= 32 the cut is the k-th
            // smallest of the 32 lanes' minima: at least k keys lie at or below it, about 1.5 k on keys in no
            // particular order.  Otherwise (or if ties leave too many) it is bisected, the score words re-read from
            // shared memory in every round.
            if (warp == 0) {
                const uint32_t* kw = reinterpret_cast<const uint32_t*>(keys);  // score word of key i: kw[2 i + 1]
                uint32_t lmn = 0xFFFFFFFFu, wmx = 0u;  // this lane's smallest score word, the largest of all
#pragma unroll 4
                for (int i = lane; i < n; i += 32) {
                    const uint32_t o = kw[2 * i + 1];
                    lmn = o < lmn ? o : lmn;
                    wmx = o > wmx ? o : wmx;
                }
                const uint32_t wmn = __reduce_min_sync(0xffffffffu, lmn);
                wmx = __reduce_max_sync(0xffffffffu, wmx);
                long long lo = (long long)wmn - 1, hi = wmx;  // #(score <= lo) < k <= #(score <= hi)
                uint32_t want_max = (uint32_t)(k + (k >> 2) + 8);
                if (want_max < (uint32_t)WARP_SORT_MAX) want_max = WARP_SORT_MAX;  // what one warp sorts afterwards
                const bool quick = k <= 32 && n >= 32;
                uint32_t c_hi = (uint32_t)n;
                if (quick) {  // the count at the quick cut comes out of the compaction
                    hi = __shfl_sync(0xffffffffu, warp_sort_u32(lmn, lane), k - 1);
                    c_hi = 0;
                }
                const uint32_t lt_mask = (1u << lane) - 1u;
                int nn = n;
                for (int attempt = 0; attempt < 2; ++attempt) {
                    while (hi - lo > 1 && c_hi > want_max) {
                        const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
                        uint32_t c = 0;
#pragma unroll 4
                        for (int i = lane; i < nn; i += 32) c += kw[2 * i + 1] <= mid ? 1u : 0u;
                        c = __reduce_add_sync(0xffffffffu, c);
                        if (c < (uint32_t)k) lo = mid; else { hi = mid; c_hi = c; }
                    }
                    const uint32_t Tw = (uint32_t)hi;
                    int base = 0;
                    for (int i0 = 0; i0 < nn; i0 += 128) {  // four rows of 32 keys at a time: their loads overlap
                        unsigned long long key[4];
                        uint32_t m[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int i = i0 + 32 * u + lane;
                            key[u] = i < nn ? keys[i] : KEY_MAX;
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            m[u] = __ballot_sync(0xffffffffu, i0 + 32 * u + lane < nn && (uint32_t)(key[u] >> 32) <= Tw);
                        __syncwarp();  // a key moves to a position at or before its own, and these 128 have been read
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if ((m[u] >> lane) & 1u) keys[base + __popc(m[u] & lt_mask)] = key[u];
                            base += __popc(m[u]);
                        }
                    }
                    __syncwarp();
                    nn = base;
                    c_hi = (uint32_t)base;
                    if (!quick || attempt == 1 || c_hi <= want_max) break;
                }
                if (lane == 0) { ctrl->redu[0][1] = (uint32_t)nn; ctrl->redu[0][0] = (uint32_t)hi; }
            }
            csync();
            if (dead) return;
            // the count changes only now that every thread has taken this branch on the old one; nobody reads or
            // adds to it before the barrier the callers follow this call with
            if (ctid == 0) ctrl->cnt = (int)ctrl->redu[0][1];
            const unsigned long long bound = ((unsigned long long)ctrl->redu[0][0] << 32) | 0xFFFFFFFFull;  // >= the k-th best key
            if (bound < tau) tau = bound;
            if (ctid == 0) atomicMin(&a.qthresh[cur_q], bound);
            return;
        }
        unsigned long long mine[KPT];
        uint32_t mn = 0xFFFFFFFFu, mx = 0u;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int i = ctid + j * NCT;
            mine[j] = i < n ? keys[i] : KEY_MAX;
            if (i < n) {
                const uint32_t o = (uint32_t)(mine[j] >> 32);
                mn = o < mn ? o : mn;
                mx = o > mx ? o : mx;
            }
        }
        mn = __reduce_min_sync(0xffffffffu, mn);
        mx = __reduce_max_sync(0xffffffffu, mx);
        if (lane == 0) { ctrl->redu[0][warp] = mn; ctrl->redu[1][warp] = mx; }
        csync();
        if (dead) return;
        for (int w = 0; w < NCW; ++w) {
            mn = ctrl->redu[0][w] < mn ? ctrl->redu[0][w] : mn;
            mx = ctrl->redu[1][w] > mx ? ctrl->redu[1][w] : mx;
        }
        csync();  // the minima / maxima have been read; redu is free for the counts
        if (dead) return;
        long long lo = (long long)mn - 1, hi = mx;  // #(score <= lo) < k <= #(score <= hi)
        uint32_t c_hi = (uint32_t)n;
        const uint32_t want_max = (uint32_t)(k + (k >> 2) + 8);
        int round = 0;
        while (hi - lo > 1 && c_hi > want_max) {  // uniform across the CTA
            const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
            uint32_t c = 0;
#pragma unroll
            for (int j = 0; j < KPT; ++j) c += (mine[j] != KEY_MAX && (uint32_t)(mine[j] >> 32) <= mid) ? 1u : 0u;
            c = __reduce_add_sync(0xffffffffu, c);
            if (lane == 0) ctrl->redu[round & 1][warp] = c;
            csync();
            if (dead) return;
            c = 0;
            for (int w = 0; w < NCW; ++w) c += ctrl->redu[round & 1][w];
            if (c < (uint32_t)k) lo = mid; else { hi = mid; c_hi = c; }
            ++round;
        }
        const uint32_t T = (uint32_t)hi;
        if (ctid == 0) ctrl->cnt = 0;  // every thread holds its keys in registers since the first barrier above
        csync();
        if (dead) return;
#pragma unroll
        for (int j = 0; j < KPT; ++j)
            warp_push(keys, &ctrl->cnt, mine[j] != KEY_MAX && (uint32_t)(mine[j] >> 32) <= T, mine[j], C::KCAP);
        const unsigned long long bound = ((unsigned long long)T << 32) | 0xFFFFFFFFull;  // >= the k-th best key
        if (bound < tau) tau = bound;
        if (ctid == 0) atomicMin(&a.qthresh[cur_q], bound);
    };

    // Close the current query's candidate buffer: keep at most k keys and park them in this CTA's slot.
    auto finalize = [&]() {
        csync();
        if (dead) return;
        int kept = ctrl->cnt;
        // a long buffer: bisect down to about k keys first, then sort only those.  A cut pays when it makes the sort
        // smaller: for small k down to what one warp sorts, otherwise below the next power of two.
        if (k <= 32 ? kept > WARP_SORT_MAX : kept > 2 * k + 64) {
            cut_buffer();
            if (dead) return;
            csync();
            if (dead) return;
            kept = ctrl->cnt;
        }
        if (kept > 1) {  // the slot is left in ascending order, which the merge relies on
            kept = block_select_short(keys, &ctrl->cnt, k, ctid, NCT, csync, C::KCAP);  // few keys: one warp, one barrier
            if (dead) return;
        }
        if (kept == k && ctid == 0) atomicMin(&a.qthresh[cur_q], keys[k - 1]);
        const size_t slot = (size_t)cur_q + blockIdx.x;
        for (int i = ctid; i < kept; i += NCT) a.slot_keys[slot * k + i] = keys[i];
        if (ctid == 0) a.slot_cnt[slot] = kept;
        csync();
    };

    // Table of a query: entry (j, m) = lut_scale * <q_m, codeword j of sub-space m>.
    // Small k: once the first tiles of a query have put a hundred-odd keys into the buffer it is cut at once (cheap at
    // that length), so that the tiles that follow are pushed against a threshold instead of in full.
    bool early = false;
    auto begin_query = [&](int q) {
        cur_q = q;
        early = k <= 32;
        if (a.lut_img != nullptr) {  // the table was built ahead of the scan: fetch its shared-memory image
            // One thread asks the copy engine for the image (bulk copies, completion counted on a barrier): the 64 or
            // 128 KB arrive at the rate of the L2 -> shared-memory path instead of a few 16-byte loads per thread
            // and round trip.  Every consumer is past its last look-up in the old table (the barrier that ended the
            // previous query); the fence orders those reads before the copies' writes.
            if (ctid == 0) {
                ctrl->cnt = 0;
                fence_proxy_async();
                const uint8_t* src = a.lut_img + (size_t)q * C::LUT_BYTES;
                const uint32_t bar = smem_u32(&ctrl->lutbar);
                mbar_arrive_expect_tx(bar, (uint32_t)C::LUT_BYTES);
                constexpr uint32_t PIECE = 32768;
                for (uint32_t o = 0; o < (uint32_t)C::LUT_BYTES; o += PIECE)
                    bulk_g2s(P.lut + o, src + o, (uint32_t)C::LUT_BYTES - o < PIECE ? (uint32_t)C::LUT_BYTES - o : PIECE, bar);
            }
            inv_scale = __ldg(a.lut_inv + q);
            tau = *reinterpret_cast<volatile unsigned long long*>(&a.qthresh[q]);
            dead = dead || !mbar_wait(smem_u32(&ctrl->lutbar), lphase, abort_flag, a.err);
            lphase ^= 1u;
            csync();
            return;
        }
        const float* qrow = a.queries + (size_t)q * a.d;
        for (int j = ctid; j < a.d; j += NCT) rT[(j % a.dsub) * C::M + j / a.dsub] = lut_scale * qrow[j];
        if (ctid == 0) ctrl->cnt = 0;
        csync();
        if (dead) return;
        float mx;
        switch (a.dsub) {
            case 4: mx = build_table<C, 1>(a.cbT, rT, P.lut, ctid); break;
            case 8: mx = build_table<C, 2>(a.cbT, rT, P.lut, ctid); break;
            case 12: mx = build_table<C, 3>(a.cbT, rT, P.lut, ctid); break;
            case 16: mx = build_table<C, 4>(a.cbT, rT, P.lut, ctid); break;
            default: mx = build_table_any<C>(a.cbT, rT, P.lut, ctid, a.dsub); break;
        }
        // per-query scale: the largest power of two that keeps a sum of M entries below 2^30
        mx = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(mx)));  // non-negative floats order like their bits
        if (lane == 0) ctrl->red[warp] = mx;
        csync();
        if (dead) return;
        for (int w = 0; w < NCW; ++w) mx = fmaxf(mx, ctrl->red[w]);
        int ex = 0;
        if (mx > 0.f && mx < 3.0e38f) frexpf(mx * (float)C::M, &ex);  // mx * M < 2^ex
        ex = ex < -90 ? -90 : (ex > 120 ? 120 : ex);
        quantise_table<C>(P.lut, ctid, ldexpf(1.f, 30 - ex));
        inv_scale = ldexpf(1.f, ex - 30);
        tau = *reinterpret_cast<volatile unsigned long long*>(&a.qthresh[q]);
        csync();
    };

    // few pairs: the first query is known without the producer, so its table is fetched while the first tile is
    // still on its way (the tile loop finds cur_q set and goes straight to the scan)
    if (few_pairs) begin_query(first_pair / a.nprobe);
    int cst = 0;            // n % S and the parity of n / S, kept by counting
    uint32_t cparity = 0;
    for (int n = 0; n < T && !dead; ++n) {
        const int st = cst;
        const uint32_t parity = cparity;
        if (++cst == S) { cst = 0; cparity ^= 1u; }
        dead = dead || !mbar_wait(smem_u32(&ctrl->full[st]), parity, abort_flag, a.err);
        if (dead) break;
        const TileDesc D = ctrl->desc[st];
        if (D.newpair & 1) {
            const int q = D.pair / a.nprobe;
            if (q != cur_q) {
                if (cur_q >= 0) finalize();
                if (dead) break;
                begin_query(q);
                if (dead) break;
            }
            bias = ip ? -D.term : D.term;
        }
        // the producer saw the buffer filling up, or (small k) this is the query's second tile in this CTA: keep the
        // best k (or a few more), lower the threshold.  One site for both, so that the cut is in the loop once.
        const bool full_cut = (D.newpair & 2) != 0;
        if (full_cut || (early && !(D.newpair & 1))) {
            csync();
            if (dead) break;
            if (ctrl->cnt > (full_cut ? k : 2 * WARP_SORT_MAX)) {  // uniform: nothing is pushed between the two barriers
                cut_buffer();
                early = false;
            }
            if (dead) break;
            const unsigned long long g = *reinterpret_cast<volatile unsigned long long*>(&a.qthresh[cur_q]);
            if (g < tau) tau = g;
            csync();
            if (dead) break;
        }

        // ---- scan this tile: warp w owns row groups w*RGW .. w*RGW+RGW-1 ----
        const int nvr = D.nvec * R;
        const uint32_t tile_base = D.tile_addr;
        const uint32_t vt_base = D.vt_addr + (uint32_t)D.vrem * 4u;
        // Row groups are taken MERGE at a time: with R lanes per vector every lane of an R-group ends up with
        // the vector's sum, so lane slice g finishes row group g and one epilogue serves MERGE row groups.
        constexpr int MERGE = R < C::RGW ? R : C::RGW;
        bool released = false;
        uint32_t wa[G];  // this lane's word addresses in the warp's first row group of the tile
#pragma unroll
        for (int il = 0; il < G; ++il) wa[il] = tile_base + xo[il];
        // One pass: MERGE row groups and their shared epilogue.  RG is a type carrying the first row group's index,
        // so that every shared-memory offset below is a compile-time constant.  Returns false when the tile ended.
        auto pass = [&](auto RG) -> bool {
            constexpr int rg = decltype(RG)::value;
            const int vr0 = (warp * C::RGW + rg) * 32;
            if (vr0 >= nvr) return false;
            int mine = 0;
            auto group = [&](auto GI) {
                constexpr int g = decltype(GI)::value;
                int acc[4] = {0, 0, 0, 0};
                uint32_t x[C::NBLK][G];
                LoadWords<C, G, 0, (rg + g) * 32 * C::MV>::run(wa, x);
                ScanBlocks<C, G, 0>::run(x, cc, sel, lo, P.lut, acc);
                int si = (acc[0] + acc[1]) + (acc[2] + acc[3]);
                if (R >= 2) si += __shfl_xor_sync(0xffffffffu, si, 1);
                if (R >= 4) si += __shfl_xor_sync(0xffffffffu, si, 2);
                if (MERGE == 1 || sr == g) mine = si;
            };
            group(std::integral_constant<int, 0>{});
            if constexpr (MERGE >= 2) group(std::integral_constant<int, 1>{});
            if constexpr (MERGE >= 3) group(std::integral_constant<int, 2>{});
            if constexpr (MERGE >= 4) group(std::integral_constant<int, 3>{});
            const int vr = vr0 + (MERGE == 1 ? 0 : sr * 32) + lane;  // the virtual row whose vector this lane finishes
            const float s = (float)mine * inv_scale;
            // per-vector term of the L2 expansion (0 for inner product); rows past the tile's end read
            // stale but in-bounds shared memory and are never pushed
            const float vt = a.vterm != nullptr ? lds_f32(vt_base + (uint32_t)(vr / R) * 4u) : 0.f;
            // In the last pass over the tile that was this warp's last read of the stage: hand the stage back
            // before the rest of the epilogue, so that the refill starts that much earlier (M = 96: -1%).
            if constexpr (rg + MERGE >= C::RGW) {
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[st]));
                released = true;
            }
            const float score = (bias + vt) + s;  // smaller is better for both metrics
            const unsigned long long key = make_key(score, D.pos0 + (uint32_t)(vr / R));
            const bool owner = MERGE == 1 ? sr == 0 : sr < MERGE;
            warp_push(keys, &ctrl->cnt, vr < nvr && owner && key < tau, key, C::KCAP);
            return true;
        };
        static_assert(C::RGW / MERGE <= 4, "passes are written out below");
        bool more = pass(std::integral_constant<int, 0>{});
        if constexpr (C::RGW > MERGE) more = more && pass(std::integral_constant<int, MERGE>{});
        if constexpr (C::RGW > 2 * MERGE) more = more && pass(std::integral_constant<int, 2 * MERGE>{});
        if constexpr (C::RGW > 3 * MERGE) more = more && pass(std::integral_constant<int, 3 * MERGE>{});
        if (!released) {  // a warp that left the loop early: no rows of this tile are its own
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[st]));
        }
    }
    if (!dead && cur_q >= 0) finalize();
}

// ---- host side ----------------------------------------------------------------------------------
struct Variant {
    int M;
    void (*kernel)(const ScanArgs);
    int threads, tile_vecs;
    int (*stages_for)(int d, bool need_vt);
    int lut_bytes, lut_banked, lut_copies, lut_copy_off, lut_stride;
};
template <class C>
static int stages_for(int d, bool need_vt) {
    for (int s = C::SMAX; s >= 2; --s)
        if (plan_smem<C>(SMEM_BASE_EXPECTED, SMEM_OPTIN, d, s, need_vt).ok) return s;
    return 0;
}
#define RAGO_VARIANT(WV, G, R, NCW, RGW) \
    { Cfg<WV, G, R, NCW, RGW>::M, scan_kernel<WV, G, R, NCW, RGW>, Cfg<WV, G, R, NCW, RGW>::THREADS, \
      Cfg<WV, G, R, NCW, RGW>::TV, stages_for<Cfg<WV, G, R, NCW, RGW>>, Cfg<WV, G, R, NCW, RGW>::LUT_BYTES, \
      Cfg<WV, G, R, NCW, RGW>::BANKED ? 1 : 0, Cfg<WV, G, R, NCW, RGW>::COPIES, Cfg<WV, G, R, NCW, RGW>::COPY_OFF, \
      Cfg<WV, G, R, NCW, RGW>::LSTRIDE }
// Warps x unrolled row groups per warp were chosen by measurement: independent row groups in flight inside a warp
// hide the look-up latency better than more warps do (M = 64: 16 x 2 -> 12 x 4 gave +30%), and 15 consumer warps
// (four warps on every scheduler, the producer included) beat 12, 14 and 16 wherever their tiles fit (M = 32: +3%,
// M = 48: +6%, M = 64: +4.5%).  Where a code size has two entries the first one whose shared-memory plan fits the
// index (dimension, metric) is taken.
static const Variant kVariants[] = {
    RAGO_VARIANT(4, 4, 1, 16, 2),   // M = 16
    RAGO_VARIANT(8, 8, 1, 15, 2),   // M = 32
    RAGO_VARIANT(12, 4, 1, 15, 1),  // M = 48 (two table copies: 128 KB, a 2 048-key buffer, tiles of at most 512 vectors)
    RAGO_VARIANT(8, 8, 2, 15, 4),   // M = 64: 15 + 1 warps fill the four schedulers evenly; two 60 KB tiles below the table
    RAGO_VARIANT(8, 8, 2, 12, 4),   // M = 64 where those do not fit
    RAGO_VARIANT(20, 4, 1, 8, 1),   // M = 80
    RAGO_VARIANT(24, 8, 1, 12, 1),  // M = 96
    RAGO_VARIANT(8, 8, 4, 12, 3),   // M = 128
};

static const Variant* find_variant(int M, int d, bool need_vt) {
    for (const Variant& v : kVariants)
        if (v.M == M && v.stages_for(d, need_vt) >= 2) return &v;
    return nullptr;
}

bool scan_supported(int M) {
    for (const Variant& v : kVariants)
        if (v.M == M) return true;
    return false;
}

cudaError_t scan_plan(const IndexImpl* ix, ScanPlan* plan) {
    const Variant* v = find_variant(ix->M, ix->d, ix->metric != RAGO_IP);
    if (!v) return cudaErrorInvalidValue;
    const int stages = v->stages_for(ix->d, ix->metric != RAGO_IP);
    plan->tile_vecs = v->tile_vecs;
    plan->stages = stages;
    plan->ctas = ix->num_sms;
    plan->smem_bytes = SMEM_OPTIN;
    plan->lut_bytes = v->lut_bytes; plan->lut_banked = v->lut_banked; plan->lut_copies = v->lut_copies;
    plan->lut_copy_off = v->lut_copy_off; plan->lut_stride = v->lut_stride;
    return cudaFuncSetAttribute(v->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_OPTIN);
}

cudaError_t launch_scan(const IndexImpl* ix, const ScanPlan& plan, const float* queries, const int32_t* probe_list,
                        const float* probe_term, const int64_t* work_prefix, int nq, int nprobe, int k,
                        unsigned long long* qthresh, int32_t* slot_cnt, unsigned long long* slot_keys,
                        uint32_t* err_word, const uint8_t* lut_img, const float* lut_inv, cudaStream_t s) {
    const Variant* v = find_variant(ix->M, ix->d, ix->metric != RAGO_IP);
    if (!v) return cudaErrorInvalidValue;
    ScanArgs a;
    a.codes = ix->codes; a.list_offsets = ix->list_offsets; a.probe_list = probe_list; a.probe_term = probe_term;
    a.queries = queries; a.cbT = ix->cbT; a.work_prefix = work_prefix;
    a.vterm = ix->vterm;
    a.qthresh = qthresh; a.slot_cnt = slot_cnt; a.slot_keys = slot_keys; a.err = err_word;
    a.lut_img = lut_img; a.lut_inv = lut_inv;
    a.npairs = nq * nprobe; a.nprobe = nprobe; a.d = ix->d; a.dsub = ix->dsub;
    a.metric = ix->metric; a.k = k; a.stages = plan.stages; a.dyn_bytes = (uint32_t)plan.smem_bytes;
    a.stream_once = nq <= 64 ? 1 : 0;
    const cudaError_t e = launch_overlapped(v->kernel, dim3(plan.ctas), dim3(v->threads), plan.smem_bytes, s, a);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- lookup tables of a small batch, built ahead of the scan ---------------------------------------
// With few queries every scan CTA would build the same handful of tables, each reading the whole codebook; here
// the tables are built once, by many CTAs per query, and stored as the exact shared-memory image the scan variant
// uses (padding included), so a scan CTA fetches a table with one linear copy.
//
// The fixed-point scale cannot wait for the largest entry (the CTAs of a query do not meet), so it comes from a
// bound: |entry(j, m)| = |s <q_m, cw_mj>| <= |s| ||q_m|| max_j ||cw_mj||.  The bound costs a bit or two of the 30
// the sum may use, which leaves the quantisation error far below the tolerance.
__global__ void codeword_norms_kernel(const float* __restrict__ cb, int dsub, float* __restrict__ cwmax) {
    __shared__ float red[KSUB / 32];
    const int m = blockIdx.x, j = threadIdx.x;  // KSUB threads: one codeword each
    float n2 = 0.f;
    for (int t = 0; t < dsub; ++t) { const float v = cb[((size_t)m * KSUB + j) * dsub + t]; n2 = fmaf(v, v, n2); }
    float n = sqrtf(n2);
    for (int o = 16; o; o >>= 1) n = fmaxf(n, __shfl_xor_sync(0xffffffffu, n, o));
    if ((j & 31) == 0) red[j >> 5] = n;
    __syncthreads();
    if (j == 0) {
        for (int w = 1; w < KSUB / 32; ++w) n = fmaxf(n, red[w]);
        cwmax[m] = n;
    }
}
cudaError_t launch_codeword_norms(const float* codebooks, int M, int dsub, float* cwmax, cudaStream_t s) {
    codeword_norms_kernel<<<M, KSUB, 0, s>>>(codebooks, dsub, cwmax);
    count_launch();
    return cudaGetLastError();
}

constexpr int BT_THREADS = 256;
__global__ void __launch_bounds__(BT_THREADS) build_tables_kernel(const TableArgs t) {
    extern __shared__ float bt_smem[];
    build_table_part(t, blockIdx.y, blockIdx.x, gridDim.x, bt_smem);
}
static TableArgs table_args(const IndexImpl* ix, const float* queries, uint8_t* lut_img, float* lut_inv) {
    const ScanPlan& pl = ix->plan;
    TableArgs t;
    t.queries = queries; t.cbT = ix->cbT; t.cwmax = ix->cwmax;
    t.d = ix->d; t.dsub = ix->dsub; t.M = ix->M; t.metric = ix->metric;
    t.lut_bytes = pl.lut_bytes; t.banked = pl.lut_banked; t.copies = pl.lut_copies; t.copy_off = pl.lut_copy_off;
    t.lstride = pl.lut_stride; t.lut_img = lut_img; t.lut_inv = lut_inv;
    return t;
}
static int table_parts(const IndexImpl* ix, int nq) {
    const int parts = 2 * ix->num_sms / nq;
    return parts < 1 ? 1 : (parts > 64 ? 64 : parts);
}
// Large batches.  One CTA per (range of code values, chunk of queries): every thread keeps the codewords of its EPT
// entries in registers and walks the chunk's queries, so the codebook crosses L2 once per chunk of queries
// instead of once per query.  The scale of each query (same bound as above) comes from a kernel of
// its own, because a CTA sees only a slice of the sub-spaces.
__global__ void __launch_bounds__(128) table_scales_kernel(const float* __restrict__ queries,
                                                            const float* __restrict__ cwmax, int d, int dsub, int M,
                                                            float* __restrict__ lut_scale, float* __restrict__ lut_inv) {
    __shared__ float red[4];
    const int q = blockIdx.x, tid = threadIdx.x;
    const float* qrow = queries + (size_t)q * d;
    float mx = 0.f;
    for (int m = tid; m < M; m += 128) {
        float n2 = 0.f;
        for (int u = 0; u < dsub; ++u) { const float v = qrow[m * dsub + u]; n2 = fmaf(v, v, n2); }
        mx = fmaxf(mx, 2.0002f * sqrtf(n2) * cwmax[m]);
    }
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((tid & 31) == 0) red[tid >> 5] = mx;
    __syncthreads();
    if (tid == 0) {
        mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
        int ex = 0;
        if (mx > 0.f && mx < 3.0e38f) frexpf(mx * (float)M, &ex);
        ex = ex < -90 ? -90 : (ex > 120 ? 120 : ex);
        lut_scale[q] = ldexpf(1.f, 30 - ex);
        lut_inv[q] = ldexpf(1.f, ex - 30);
    }
}

constexpr int BTB_CW_FLOATS = 96;  // codeword floats a thread keeps in registers
// blockDim.x = M * G: thread (m, g) owns sub-space m of the code values j = j0 + g + G i, i < EPT, so everything it
// needs of a query is the DSUB values of one sub-space, fetched straight into registers (the next query's while the
// current one is multiplied): no shared memory and no barrier.  Threads with consecutive m read consecutive
// codewords and write consecutive table columns.
template <int DSUB>
__global__ void __launch_bounds__(256) build_tables_batch_kernel(const TableArgs t, const float* __restrict__ lut_scale,
                                                                  int nq, int qchunk) {
    constexpr int EPT = BTB_CW_FLOATS / DSUB;  // entries per thread
    const int d = t.d, M = t.M, tid = threadIdx.x;
    const int G = blockDim.x / M;
    const int m = tid % M, g = tid / M;
    const int j0 = blockIdx.x * (G * EPT);
    float cw[EPT][DSUB];
    uint32_t off[EPT];  // byte offset of the entry in a table image, 0xFFFFFFFF for an unused slot
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
        const int j = j0 + g + G * i;
        off[i] = 0xFFFFFFFFu;
#pragma unroll
        for (int u = 0; u < DSUB; ++u) cw[i][u] = 0.f;
        if (j < KSUB) {
            off[i] = t.banked ? (uint32_t)(m / 64) * 65536u + (uint32_t)j * 256u + (uint32_t)(m % 64) * 4u
                              : ((uint32_t)j * t.lstride + (uint32_t)m) * 4u;
            const float* src = t.cbT + ((size_t)j * M + m) * DSUB;
#pragma unroll
            for (int u = 0; u < DSUB; u += 4) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(src + u));
                cw[i][u] = v.x; cw[i][u + 1] = v.y; cw[i][u + 2] = v.z; cw[i][u + 3] = v.w;
            }
        }
    }
    // second copy of a column (layouts that keep one), as a byte distance inside the image
    const uint32_t copy_delta = t.copies == 2
        ? (t.banked ? (uint32_t)((t.copy_off / 64) * 65536 + (t.copy_off % 64) * 4) : (uint32_t)t.copy_off * 4u) : 0u;
    const float lut_s = t.metric == RAGO_IP ? -1.f : -2.f;
    const int q0 = blockIdx.y * qchunk;
    const int q1 = q0 + qchunk < nq ? q0 + qchunk : nq;
    float qn[DSUB];
    auto fetch = [&](int q) {
        const float* src = t.queries + (size_t)q * d + m * DSUB;
#pragma unroll
        for (int u = 0; u < DSUB; u += 4) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(src + u));
            qn[u] = v.x; qn[u + 1] = v.y; qn[u + 2] = v.z; qn[u + 3] = v.w;
        }
    };
    if (q0 < q1) fetch(q0);
    for (int q = q0; q < q1; ++q) {
        float qv[DSUB];
#pragma unroll
        for (int u = 0; u < DSUB; ++u) qv[u] = lut_s * qn[u];
        if (q + 1 < q1) fetch(q + 1);
        const float scale = __ldg(lut_scale + q);
        uint8_t* img = t.lut_img + (size_t)q * t.lut_bytes;
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            float acc = 0.f;
#pragma unroll
            for (int u = 0; u < DSUB; ++u) acc = fmaf(qv[u], cw[i][u], acc);
            if (off[i] != 0xFFFFFFFFu) {
                const int v = __float2int_rn(acc * scale);
                *reinterpret_cast<int*>(img + off[i]) = v;
                if (copy_delta) *reinterpret_cast<int*>(img + off[i] + copy_delta) = v;
            }
        }
    }
}

cudaError_t launch_build_tables(const IndexImpl* ix, const float* queries, int nq, uint8_t* lut_img, float* lut_inv,
                                float* lut_scale, cudaStream_t s) {
    const int dsub = ix->dsub;
    const TableArgs t = table_args(ix, queries, lut_img, lut_inv);
    if (nq > 64 && lut_scale && (dsub == 4 || dsub == 8 || dsub == 12 || dsub == 16)) {
        table_scales_kernel<<<nq, 128, 0, s>>>(queries, ix->cwmax, ix->d, dsub, ix->M, lut_scale, lut_inv);
        const int ept = BTB_CW_FLOATS / dsub;
        const int G = 256 / ix->M;  // >= 2: the scan supports M <= 128
        const int threads = ix->M * G;
        const int parts = (KSUB + G * ept - 1) / (G * ept);
        int qchunk = (int)(((long long)nq * parts + 4 * ix->num_sms - 1) / (4 * ix->num_sms));
        if (qchunk < 1) qchunk = 1;
        const dim3 grid(parts, (nq + qchunk - 1) / qchunk);
        switch (dsub) {
            case 4: build_tables_batch_kernel<4><<<grid, threads, 0, s>>>(t, lut_scale, nq, qchunk); break;
            case 8: build_tables_batch_kernel<8><<<grid, threads, 0, s>>>(t, lut_scale, nq, qchunk); break;
            case 12: build_tables_batch_kernel<12><<<grid, threads, 0, s>>>(t, lut_scale, nq, qchunk); break;
            default: build_tables_batch_kernel<16><<<grid, threads, 0, s>>>(t, lut_scale, nq, qchunk); break;
        }
        count_launch(2);
        return cudaGetLastError();
    }
    build_tables_kernel<<<dim3(table_parts(ix, nq), nq), BT_THREADS, (size_t)(ix->d + ix->M) * 4, s>>>(t);
    count_launch();
    return cudaGetLastError();
}

// ---- codebook transpose: cb[m][j][t] -> cbT[j][m][t] -------------------------------------------
__global__ void transpose_codebook_kernel(const float* __restrict__ cb, int M, int dsub, float* __restrict__ cbT) {
    const int total = M * KSUB * dsub;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int t = i % dsub, jm = i / dsub, m = jm % M, j = jm / M;
        cbT[i] = cb[((size_t)m * KSUB + j) * dsub + t];
    }
}
cudaError_t launch_transpose_codebook(const float* cb, int M, int dsub, float* cbT, cudaStream_t s) {
    transpose_codebook_kernel<<<256, 256, 0, s>>>(cb, M, dsub, cbT);
    count_launch();
    return cudaGetLastError();
}

// ---- per-vector term of the squared-L2 expansion ------------------------------------------------
// ||q - (c + r)||^2 = ||q - c||^2 + (||r||^2 + 2<c, r>) - 2<q, r>,  r = decoded residual of the vector.
// The middle term depends on the stored vector only; it is computed once per index, in double, one
// warp per vector (lanes over sub-spaces), and rounded to float once.
template <bool BF16>
__global__ void vector_terms_kernel(const uint8_t* __restrict__ codes, const int64_t* __restrict__ offsets,
                                    const void* __restrict__ centroids, const float* __restrict__ cb, long long N,
                                    int nlist, int d, int M, int dsub, float* __restrict__ vterm) {
    const int lane = threadIdx.x & 31;
    const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long pos = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; pos < N; pos += warps) {
        int lo = 0, hi = nlist;  // offsets[lo] <= pos < offsets[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (offsets[mid] <= pos) lo = mid; else hi = mid;
        }
        double acc = 0.0;
        for (int m = lane; m < M; m += 32) {
            const int code = codes[pos * M + m];
            const float* cw = cb + ((size_t)m * KSUB + code) * dsub;
            for (int t = 0; t < dsub; ++t) {
                const size_t ci = (size_t)lo * d + m * dsub + t;
                const double c = BF16 ? (double)__bfloat162float(static_cast<const __nv_bfloat16*>(centroids)[ci])
                                      : (double)static_cast<const float*>(centroids)[ci];
                const double r = (double)cw[t];
                acc += r * (r + 2.0 * c);
            }
        }
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) vterm[pos] = (float)acc;
    }
}

cudaError_t launch_vector_terms(const IndexImpl* ix, float* vterm, cudaStream_t s) {
    if (ix->N == 0) return cudaSuccess;
    const long long want = (ix->N * 32 + 255) / 256;
    const int blocks = (int)(want < 148LL * 64 ? want : 148LL * 64);
    if (ix->coarse_bf16)
        vector_terms_kernel<true><<<blocks, 256, 0, s>>>(ix->codes, ix->list_offsets, ix->centroids, ix->codebooks,
                                                         ix->N, ix->nlist, ix->d, ix->M, ix->dsub, vterm);
    else
        vector_terms_kernel<false><<<blocks, 256, 0, s>>>(ix->codes, ix->list_offsets, ix->centroids, ix->codebooks,
                                                          ix->N, ix->nlist, ix->d, ix->M, ix->dsub, vterm);
    count_launch();
    return cudaGetLastError();
}

// ---- work planning: tiles per pair and their exclusive prefix sum ------------------------------
// Three small launches: (1) tiles per pair with a CTA-local exclusive scan and one total per CTA,
// (2) one CTA scans the totals, (3) every CTA adds its offset.
constexpr int PT_THREADS = 256;
__global__ void __launch_bounds__(PT_THREADS) pair_tiles_kernel(const int32_t* __restrict__ probe_list,
                                                                const int64_t* __restrict__ offsets, int npairs,
                                                                int tile_vecs, int64_t* __restrict__ prefix,
                                                                long long* __restrict__ block_sums) {
    __shared__ long long warp_sums[PT_THREADS / 32];
    const int p = blockIdx.x * PT_THREADS + threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long v = 0;
    if (p < npairs) {
        const int l = probe_list[p];
        v = (offsets[l + 1] - offsets[l] + tile_vecs - 1) / tile_vecs;
    }
    long long incl = v;
    for (int o = 1; o < 32; o <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    long long before = incl - v;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (p < npairs) prefix[p] = before;
    if (threadIdx.x == PT_THREADS - 1) block_sums[blockIdx.x] = before + v;
}

// In-place exclusive scan of n totals by one CTA; the grand total goes to *total_out.
__global__ void __launch_bounds__(PFX_THREADS) scan_totals_kernel(long long* __restrict__ sums, int n,
                                                                  int64_t* __restrict__ total_out) {
    __shared__ long long warp_sums[32];
    __shared__ long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    for (int base = 0; base < n; base += PFX_THREADS) {
        const int i = base + tid;
        const long long v = i < n ? sums[i] : 0;
        long long incl = v;
        for (int o = 1; o < 32; o <<= 1) {
            const long long y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            long long w = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) {
                const long long y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;  // inclusive over warps
        }
        __syncthreads();
        const long long before = carry_s + (warp ? warp_sums[warp - 1] : 0) + incl - v;
        if (i < n) sums[i] = before;
        __syncthreads();
        if (tid == PFX_THREADS - 1) carry_s = before + v;
        __syncthreads();
    }
    if (tid == 0) *total_out = carry_s;
}

__global__ void __launch_bounds__(PT_THREADS) add_offsets_kernel(int64_t* __restrict__ prefix, int npairs,
                                                                 const long long* __restrict__ block_sums) {
    const int p = blockIdx.x * PT_THREADS + threadIdx.x;
    if (p < npairs) prefix[p] += block_sums[blockIdx.x];
}

// Small batches: one CTA does the whole preparation of a search (tiles per pair, their prefix sum,
// threshold and slot-counter reset), which would otherwise be four launches of a few microseconds each.
// With table_parts > 0 the CTAs after the first build the batch's lookup tables meanwhile (the tables depend on the
// queries only, so nothing orders them against the planning).
__global__ void __launch_bounds__(PFX_THREADS) plan_small_kernel(const int32_t* __restrict__ probe_list,
                                                                 const int64_t* __restrict__ offsets, int npairs,
                                                                 int tile_vecs, int64_t* __restrict__ prefix,
                                                                 unsigned long long* __restrict__ qthresh, int nq,
                                                                 int32_t* __restrict__ slot_cnt, int nslots,
                                                                 const TableArgs tables, int table_parts) {
    extern __shared__ float bt_smem[];
    grid_dependency_wait();
    grid_dependents_may_launch();
    if (blockIdx.x > 0) {
        const int b = blockIdx.x - 1;
        build_table_part(tables, b / table_parts, b % table_parts, table_parts, bt_smem);
        return;
    }
    __shared__ long long warp_sums[32];
    plan_pairs_cta(probe_list, offsets, npairs, tile_vecs, prefix, qthresh, nq, slot_cnt, nslots, warp_sums);
}

// Small batches whose probe selection plans the scan itself (see FusedPlan): what that kernel needs, or false when
// the batch does not qualify (tables not prebuilt, too many pairs for one CTA, more than 64 queries).
bool fused_plan_args(const IndexImpl* ix, int nq, int npairs, const float* queries, uint8_t* lut_img, float* lut_inv,
                     int64_t* work_prefix, unsigned long long* qthresh, int32_t* slot_cnt, int nslots, uint32_t* ticket,
                     FusedPlan* fp) {
    fp->enabled = 0;
    if (!lut_img || npairs > PLAN_SMALL_MAX || nq > 64) return false;
    fp->enabled = 1;
    fp->nq = nq;
    fp->ticket = ticket;
    fp->offsets = ix->list_offsets;
    fp->tile_vecs = ix->plan.tile_vecs;
    fp->prefix = work_prefix;
    fp->qthresh = qthresh;
    fp->slot_cnt = slot_cnt;
    fp->nslots = nslots;
    fp->tables = table_args(ix, queries, lut_img, lut_inv);
    fp->table_parts = table_parts(ix, nq);
    return true;
}

cudaError_t launch_plan_work(const IndexImpl* ix, const int32_t* probe_list, int npairs, int tile_vecs,
                             int32_t* pair_tiles, int64_t* work_prefix, unsigned long long* qthresh, int nq,
                             int32_t* slot_cnt, int nslots, const float* queries, uint8_t* lut_img, float* lut_inv,
                             float* lut_scale, cudaStream_t s) {
    const bool fused_tables = lut_img && npairs <= PLAN_SMALL_MAX && nq <= 64;
    if (lut_img && !fused_tables) {
        const cudaError_t et = launch_build_tables(ix, queries, nq, lut_img, lut_inv, lut_scale, s);
        if (et != cudaSuccess) return et;
    }
    if (npairs <= PLAN_SMALL_MAX) {
        const int parts = fused_tables ? table_parts(ix, nq) : 0;
        launch_overlapped(plan_small_kernel, dim3(1 + parts * nq), dim3(PFX_THREADS),
                          parts ? (size_t)(ix->d + ix->M) * 4 : 0, s,
            probe_list, ix->list_offsets, npairs, tile_vecs, work_prefix, qthresh, nq, slot_cnt, nslots,
            table_args(ix, queries, lut_img, lut_inv), parts);
        count_launch();
        return cudaGetLastError();
    }
    // pair_tiles (npairs int32 of scratch) holds the per-CTA totals: one 64-bit word per 256 pairs
    const int nblocks = (npairs + PT_THREADS - 1) / PT_THREADS;
    long long* block_sums = reinterpret_cast<long long*>(pair_tiles);
    pair_tiles_kernel<<<nblocks, PT_THREADS, 0, s>>>(probe_list, ix->list_offsets, npairs, tile_vecs, work_prefix,
                                                    block_sums);
    scan_totals_kernel<<<1, PFX_THREADS, 0, s>>>(block_sums, nblocks, work_prefix + npairs);
    add_offsets_kernel<<<nblocks, PT_THREADS, 0, s>>>(work_prefix, npairs, block_sums);
    count_launch(3);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = launch_fill_u64(qthresh, (size_t)nq, KEY_MAX, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(slot_cnt, 0, (size_t)nslots * 4, s);
    return e;
}

}  // namespace rago
