// Preparation of a scan that more than one kernel can run: a query's lookup table (one part of it per CTA) and
// the work plan of a small batch (tiles per (query, list) pair, their prefix sum, threshold and slot-counter reset).
// The planning launch of scan.cu runs both; for batches of a few queries the probe-selection kernel runs them at its
// own end, which saves a launch on the latency-bound path.
#pragma once
#include "common.cuh"

namespace rago {

constexpr int PFX_THREADS = 1024;
constexpr int PLAN_PER_THREAD = 4;       // pairs per thread of the single-CTA planning code
constexpr int PLAN_SMALL_MAX = PFX_THREADS * PLAN_PER_THREAD;

struct TableArgs {
    const float* queries; const float* cbT; const float* cwmax;
    int d, dsub, M, metric, lut_bytes, banked, copies, copy_off, lstride;
    uint8_t* lut_img; float* lut_inv;
};

// What the probe-selection kernel needs to plan the scan of a small batch itself (enabled = 0: it does not).
// The CTAs after the first nq build the lookup tables; the CTA that finishes its query last plans.
struct FusedPlan {
    int enabled;
    int nq;                      // queries of the batch = selection CTAs of the launch
    uint32_t* ticket;            // zero before the launch; the planning CTA leaves it zero again
    const int64_t* offsets;      // [nlist + 1]
    int tile_vecs;
    int64_t* prefix;             // [npairs + 1]
    unsigned long long* qthresh; // [nq]
    int32_t* slot_cnt;
    int nslots;
    TableArgs tables;
    int table_parts;             // CTAs per query's table
};

// coarse.cu (fp may be null: selection only)
cudaError_t launch_select_probes(const IndexImpl* ix, const float* queries, const float* scores, int nq, int nprobe,
                                 int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan* fp,
                                 cudaStream_t s);
cudaError_t launch_select_probes_cand(const IndexImpl* ix, const float* queries, const unsigned long long* cand,
                                      const int32_t* cand_cnt, uint32_t cand_sign, int nsplit, int cap, int nq, int nprobe,
                                      int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan* fp,
                                      cudaStream_t s);
// scan.cu
bool fused_plan_args(const IndexImpl* ix, int nq, int npairs, const float* queries, uint8_t* lut_img, float* lut_inv,
                     int64_t* work_prefix, unsigned long long* qthresh, int32_t* slot_cnt, int nslots, uint32_t* ticket,
                     FusedPlan* fp);

#ifdef __CUDACC__
// Part `part` of `parts` of query q's table, by all threads of the CTA.  sm: d + M floats of shared memory.
__device__ __forceinline__ void build_table_part(const TableArgs& t, int q, int part, int parts, float* sm) {
    const int d = t.d, dsub = t.dsub, M = t.M, tid = threadIdx.x, nthreads = blockDim.x;
    float* rT = sm;       // the scaled query with the sub-space index innermost
    float* bnd = sm + d;  // bound of the entries of every sub-space
    const float lut_scale = t.metric == RAGO_IP ? -1.f : -2.f;
    const float* qrow = t.queries + (size_t)q * d;
    for (int j = tid; j < d; j += nthreads) rT[(j % dsub) * M + j / dsub] = lut_scale * qrow[j];
    for (int m = tid; m < M; m += nthreads) {
        float n2 = 0.f;
        for (int u = 0; u < dsub; ++u) { const float v = qrow[m * dsub + u]; n2 = fmaf(v, v, n2); }
        bnd[m] = 2.0002f * sqrtf(n2) * t.cwmax[m];  // |s| <= 2, and a margin for the rounding of the norms
    }
    __syncthreads();
    float mx = 0.f;
    for (int m = 0; m < M; ++m) mx = fmaxf(mx, bnd[m]);
    int ex = 0;
    if (mx > 0.f && mx < 3.0e38f) frexpf(mx * (float)M, &ex);  // mx * M < 2^ex
    ex = ex < -90 ? -90 : (ex > 120 ? 120 : ex);
    const float scale = ldexpf(1.f, 30 - ex);
    if (part == 0 && tid == 0) t.lut_inv[q] = ldexpf(1.f, ex - 30);
    uint8_t* img = t.lut_img + (size_t)q * t.lut_bytes;
    auto off = [&](int j, int col) -> uint32_t {
        return t.banked ? (uint32_t)(col / 64) * 65536u + (uint32_t)j * 256u + (uint32_t)(col % 64) * 4u
                        : ((uint32_t)j * t.lstride + (uint32_t)col) * 4u;
    };
    const int total = KSUB * M;
    const int per = (total + parts - 1) / parts;
    const int e1 = (part + 1) * per < total ? (part + 1) * per : total;
    // entry e = (code value j, sub-space m), m fastest; (j, m) follow e by counting, not by dividing per entry
    const int step_j = nthreads / M, step_m = nthreads - step_j * M;
    int e = part * per + tid;
    int j = e / M, m = e - j * M;
    for (; e < e1; e += nthreads) {
        float acc = 0.f;
        for (int u = 0; u < dsub; ++u) acc = fmaf(rT[u * M + m], __ldg(t.cbT + (size_t)e * dsub + u), acc);
        const int v = __float2int_rn(acc * scale);
        *reinterpret_cast<int*>(img + off(j, m)) = v;
        if (t.copies == 2) *reinterpret_cast<int*>(img + off(j, t.copy_off + m)) = v;
        j += step_j;
        m += step_m;
        if (m >= M) { m -= M; ++j; }
    }
}

// The work plan of up to PLAN_SMALL_MAX pairs by one CTA of PFX_THREADS threads: tiles per pair, their exclusive
// prefix sum (prefix[npairs] = total), thresholds and slot counters back to their start values.  warp_sums: 32 words
// of shared memory.  The probe lists may have been written by other CTAs of the same launch (the caller has ordered
// those writes before this call): they are read past the L1 cache.
__device__ __forceinline__ void plan_pairs_cta(const int32_t* probe_list, const int64_t* __restrict__ offsets, int npairs,
                                               int tile_vecs, int64_t* __restrict__ prefix,
                                               unsigned long long* __restrict__ qthresh, int nq,
                                               int32_t* __restrict__ slot_cnt, int nslots, long long* warp_sums) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // thread t owns pairs PLAN_PER_THREAD * t .. + PLAN_PER_THREAD - 1
    long long mine[PLAN_PER_THREAD];
    long long v = 0;
#pragma unroll
    for (int j = 0; j < PLAN_PER_THREAD; ++j) {
        const int p = tid * PLAN_PER_THREAD + j;
        mine[j] = 0;
        if (p < npairs) {
            const int l = __ldcg(probe_list + p);
            mine[j] = (offsets[l + 1] - offsets[l] + tile_vecs - 1) / tile_vecs;
        }
        v += mine[j];
    }
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
        warp_sums[lane] = w;
    }
    __syncthreads();
    long long before = (warp ? warp_sums[warp - 1] : 0) + incl - v;
#pragma unroll
    for (int j = 0; j < PLAN_PER_THREAD; ++j) {
        const int p = tid * PLAN_PER_THREAD + j;
        if (p < npairs) prefix[p] = before;
        before += mine[j];
        if (p == npairs - 1) prefix[npairs] = before;
    }
    for (int i = tid; i < nq; i += PFX_THREADS) qthresh[i] = KEY_MAX;
    for (int i = tid; i < nslots; i += PFX_THREADS) slot_cnt[i] = 0;
}
#endif  // __CUDACC__

}  // namespace rago
