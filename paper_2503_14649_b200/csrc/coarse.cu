// Coarse quantiser: query x centroid scores and per-query nprobe selection.
//
// Ranking score, smaller is better:  L2: ||c||^2 - 2<q,c>  (same order as ||q-c||^2),  IP: -<q,c>.
// The nprobe + PROBE_GUARD best lists by that score are re-scored exactly (sum of (q-c)^2, or <q,c>)
// before the final cut, so the probe order follows the plain definition up to fp32 rounding.
// With a bf16 coarse quantiser the query is rounded to bf16 first (coarse step only).
#include "topk.cuh"

namespace rago {

__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

template <bool BF16>
__device__ __forceinline__ float load_c(const void* base, size_t idx) {
    if (BF16) return __bfloat162float(static_cast<const __nv_bfloat16*>(base)[idx]);
    return static_cast<const float*>(base)[idx];
}

// ---- squared centroid norms -------------------------------------------------------------------
template <bool BF16>
__global__ void centroid_norms_kernel(const void* __restrict__ cen, int nlist, int d, float* __restrict__ out) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= nlist) return;
    float acc = 0.f;
    for (int j = lane; j < d; j += 32) {
        const float c = load_c<BF16>(cen, (size_t)warp * d + j);
        acc = fmaf(c, c, acc);
    }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[warp] = acc;
}

cudaError_t launch_centroid_norms(const void* centroids, int bf16, int nlist, int d, float* cnorm, cudaStream_t s) {
    const int threads = 256, warps_per_block = threads / 32;
    const int blocks = (nlist + warps_per_block - 1) / warps_per_block;
    if (bf16)
        centroid_norms_kernel<true><<<blocks, threads, 0, s>>>(centroids, nlist, d, cnorm);
    else
        centroid_norms_kernel<false><<<blocks, threads, 0, s>>>(centroids, nlist, d, cnorm);
    count_launch();
    return cudaGetLastError();
}

// ---- score matrix on the fp32 pipes (64x64x16 tiles, 4x4 per thread) ---------------------------
constexpr int BM = 64, BN = 64, BK = 16;

template <bool BF16>
__global__ void __launch_bounds__(256) coarse_scores_kernel(const float* __restrict__ Q, const void* __restrict__ C,
                                                            const float* __restrict__ cnorm, int nq, int nlist, int d,
                                                            int metric, float* __restrict__ scores) {
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int row0 = blockIdx.y * BM, col0 = blockIdx.x * BN;
    const int lr = tid >> 2, lk = (tid & 3) * 4;  // this thread stages row lr, k-offset lk of both tiles
    const int ty = tid >> 4, tx = tid & 15;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < d; k0 += BK) {
        float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
        if (row0 + lr < nq) {
            const float4 v = *reinterpret_cast<const float4*>(Q + (size_t)(row0 + lr) * d + k0 + lk);
            a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
            if (BF16) {
#pragma unroll
                for (int i = 0; i < 4; ++i) a[i] = round_bf16(a[i]);
            }
        }
        if (col0 + lr < nlist) {
#pragma unroll
            for (int i = 0; i < 4; ++i) b[i] = load_c<BF16>(C, (size_t)(col0 + lr) * d + k0 + lk + i);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk + i][lr] = a[i];
            Bs[lk + i][lr] = b[i];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = row0 + ty * 4 + i;
        if (r >= nq) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = col0 + tx * 4 + j;
            if (c >= nlist) continue;
            scores[(size_t)r * nlist + c] = metric == RAGO_L2 ? fmaf(-2.f, acc[i][j], cnorm[c]) : -acc[i][j];
        }
    }
}

cudaError_t launch_coarse_scores(const IndexImpl* ix, const float* queries, int nq, float* scores, cudaStream_t s) {
    dim3 grid((ix->nlist + BN - 1) / BN, (nq + BM - 1) / BM);
    if (ix->coarse_bf16)
        coarse_scores_kernel<true><<<grid, 256, 0, s>>>(queries, ix->centroids, ix->cnorm, nq, ix->nlist, ix->d,
                                                        ix->metric, scores);
    else
        coarse_scores_kernel<false><<<grid, 256, 0, s>>>(queries, ix->centroids, ix->cnorm, nq, ix->nlist, ix->d,
                                                         ix->metric, scores);
    count_launch();
    return cudaGetLastError();
}

// ---- per-query selection of the nprobe best lists ----------------------------------------------
constexpr int SEL_THREADS = 256;

// Candidates come either from a score row (scores != null: all nlist lists) or from the candidate
// lists the tensor-core kernel left behind (cand[q][split][cap] keys with counts cand_cnt[q][split]).
template <bool BF16>
__global__ void __launch_bounds__(SEL_THREADS) select_probes_kernel(
    const float* __restrict__ Q, const void* __restrict__ C, const float* __restrict__ scores,
    const unsigned long long* __restrict__ cand, const int32_t* __restrict__ cand_cnt, int nsplit, int cap, int nlist,
    int d, int metric, int nprobe, int32_t* __restrict__ probe_list, float* __restrict__ probe_term,
    float* __restrict__ probe_bias) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ unsigned long long keys2[MAX_K + PROBE_GUARD];
    __shared__ int cnt;
    const int q = blockIdx.x, tid = threadIdx.x;
    auto sync = [] { __syncthreads(); };
    int nsel = nprobe + PROBE_GUARD;
    if (nsel > nlist) nsel = nlist;
    if (tid == 0) cnt = 0;
    __syncthreads();
    unsigned long long tau = KEY_MAX;
    int ub = 0;  // upper bound of cnt, identical in every thread
    const float* srow = scores ? scores + (size_t)q * nlist : nullptr;
    const int nitems = scores ? nlist : nsplit * cap;
    for (int l0 = 0; l0 < nitems; l0 += SEL_THREADS) {
        const int l = l0 + tid;
        unsigned long long key = KEY_MAX;
        if (l < nitems) {
            if (scores) {
                key = make_key(srow[l], (uint32_t)l);
            } else {
                const int sp = l / cap, i = l - sp * cap;
                if (i < cand_cnt[(size_t)q * nsplit + sp]) key = cand[((size_t)q * nsplit + sp) * cap + i];
            }
        }
        warp_push(keys, &cnt, key < tau, key);
        ub += SEL_THREADS;
        if (ub + SEL_THREADS > TOPK_CAP) {
            __syncthreads();
            const int kept = block_select(keys, &cnt, nsel, tid, SEL_THREADS, sync);
            if (kept == nsel) tau = keys[nsel - 1];
            ub = kept;
            __syncthreads();
        }
    }
    __syncthreads();
    const int kept = block_select(keys, &cnt, nsel, tid, SEL_THREADS, sync);  // kept == nsel (nsel <= nlist)
    // exact re-score of the survivors, one warp per candidate
    const int warp = tid >> 5, lane = tid & 31;
    const float* qrow = Q + (size_t)q * d;
    for (int i = warp; i < kept; i += SEL_THREADS / 32) {
        const uint32_t l = (uint32_t)(keys[i] & 0xFFFFFFFFull);
        float acc = 0.f;
        for (int j = lane; j < d; j += 32) {
            float qv = qrow[j];
            if (BF16) qv = round_bf16(qv);
            const float c = load_c<BF16>(C, (size_t)l * d + j);
            if (metric == RAGO_L2) {
                const float t = qv - c;
                acc = fmaf(t, t, acc);
            } else {
                acc = fmaf(qv, c, acc);
            }
        }
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) keys2[i] = make_key(metric == RAGO_L2 ? acc : -acc, l);
    }
    __syncthreads();
    for (int i = tid; i < TOPK_CAP; i += SEL_THREADS) keys[i] = i < kept ? keys2[i] : KEY_MAX;
    __syncthreads();
    int n2 = 2;
    while (n2 < kept) n2 <<= 1;
    block_bitonic_sort(keys, n2, tid, SEL_THREADS, sync);
    for (int i = tid; i < nprobe; i += SEL_THREADS) {
        const unsigned long long key = keys[i];
        const float sc = orderable_f32((uint32_t)(key >> 32));
        probe_list[(size_t)q * nprobe + i] = (int32_t)(key & 0xFFFFFFFFull);
        probe_term[(size_t)q * nprobe + i] = metric == RAGO_L2 ? sc : -sc;
        if (!(BF16 && metric == RAGO_L2)) probe_bias[(size_t)q * nprobe + i] = metric == RAGO_L2 ? sc : -sc;
    }
    // The scan's L2 expansion needs ||q - c||^2 for the UNROUNDED query; with a bf16 coarse quantiser
    // that differs from the coarse distance above, so it is computed separately for the chosen lists.
    if (BF16 && metric == RAGO_L2) {
        for (int i = warp; i < nprobe; i += SEL_THREADS / 32) {
            const uint32_t l = (uint32_t)(keys[i] & 0xFFFFFFFFull);
            float acc = 0.f;
            for (int j = lane; j < d; j += 32) {
                const float t = qrow[j] - load_c<BF16>(C, (size_t)l * d + j);
                acc = fmaf(t, t, acc);
            }
            for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) probe_bias[(size_t)q * nprobe + i] = acc;
        }
    }
}

static cudaError_t launch_select_any(const IndexImpl* ix, const float* queries, const float* scores,
                                     const unsigned long long* cand, const int32_t* cand_cnt, int nsplit, int cap, int nq,
                                     int nprobe, int32_t* probe_list, float* probe_term, float* probe_bias,
                                     cudaStream_t s) {
    if (ix->coarse_bf16)
        select_probes_kernel<true><<<nq, SEL_THREADS, 0, s>>>(queries, ix->centroids, scores, cand, cand_cnt, nsplit, cap,
                                                              ix->nlist, ix->d, ix->metric, nprobe, probe_list,
                                                              probe_term, probe_bias);
    else
        select_probes_kernel<false><<<nq, SEL_THREADS, 0, s>>>(queries, ix->centroids, scores, cand, cand_cnt, nsplit,
                                                               cap, ix->nlist, ix->d, ix->metric, nprobe, probe_list,
                                                               probe_term, probe_bias);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_select_probes(const IndexImpl* ix, const float* queries, const float* scores, int nq, int nprobe,
                                 int32_t* probe_list, float* probe_term, float* probe_bias, cudaStream_t s) {
    return launch_select_any(ix, queries, scores, nullptr, nullptr, 0, 0, nq, nprobe, probe_list, probe_term,
                             probe_bias, s);
}

cudaError_t launch_select_probes_cand(const IndexImpl* ix, const float* queries, const unsigned long long* cand,
                                      const int32_t* cand_cnt, int nsplit, int cap, int nq, int nprobe,
                                      int32_t* probe_list, float* probe_term, float* probe_bias, cudaStream_t s) {
    return launch_select_any(ix, queries, nullptr, cand, cand_cnt, nsplit, cap, nq, nprobe, probe_list, probe_term,
                             probe_bias, s);
}

}  // namespace rago
