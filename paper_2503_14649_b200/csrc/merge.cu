// Final top-k per query: merge the partial candidate lists the scan CTAs left behind, sort, map
// storage positions to caller ids, and write results best-first.
#include "topk.cuh"

namespace rago {

constexpr int MERGE_THREADS = 256;

// Slot numbering: CTA b working on query q writes slot q + b.  Along the CTAs' contiguous walk over the
// batch that number strictly increases, so the slots of one query form one range (unused numbers in
// between have count 0).
__device__ __forceinline__ long long cta_of_unit(long long u, long long W, int ctas) {
    // CTA b owns units [b*W/ctas, (b+1)*W/ctas): the largest b with floor(b*W/ctas) <= u
    return ((u + 1) * ctas - 1) / W;
}

__global__ void __launch_bounds__(MERGE_THREADS) merge_kernel(
    const int64_t* __restrict__ work_prefix, const int64_t* __restrict__ ids, int npairs, int nprobe, int k, int ctas,
    int metric, const int32_t* __restrict__ slot_cnt, const unsigned long long* __restrict__ slot_keys,
    const unsigned long long* __restrict__ qthresh,
    int64_t* __restrict__ out_ids, float* __restrict__ out_dists) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    const int q = blockIdx.x, tid = threadIdx.x;
    auto sync = [] { __syncthreads(); };
    if (tid == 0) cnt = 0;
    __syncthreads();
    const long long W = work_prefix[npairs];
    const long long u0 = work_prefix[(size_t)q * nprobe], u1 = work_prefix[(size_t)(q + 1) * nprobe];
    // a key above the threshold the scan CTAs agreed on is not among the k best (it is some CTA's k-th key)
    unsigned long long tau = qthresh[q];
    if (tau != KEY_MAX) ++tau;  // the threshold key itself is a result
    if (u1 > u0) {
        const long long s0 = (long long)q + cta_of_unit(u0, W, ctas);
        const long long s1 = (long long)q + cta_of_unit(u1 - 1, W, ctas);
        // all slots of the query side by side: entry e = (slot, i); empty entries are skipped
        const long long total = (s1 - s0 + 1) * (long long)k;
        // entries are fetched MERGE_BATCH per thread at a time (independent loads in flight), then pushed
        constexpr int MERGE_BATCH = 8;
        for (long long e0 = 0; e0 < total; e0 += (long long)MERGE_THREADS * MERGE_BATCH) {
            unsigned long long mine[MERGE_BATCH];
#pragma unroll
            for (int j = 0; j < MERGE_BATCH; ++j) {
                const long long e = e0 + (long long)j * MERGE_THREADS + tid;
                mine[j] = KEY_MAX;
                if (e < total) {
                    const long long s = s0 + e / k;
                    const int i = (int)(e % k);
                    if (i < slot_cnt[s]) mine[j] = slot_keys[(size_t)s * k + i];
                }
            }
#pragma unroll
            for (int j = 0; j < MERGE_BATCH; ++j) {
                warp_push(keys, &cnt, mine[j] < tau, mine[j]);
                __syncthreads();
                if (cnt + MERGE_THREADS > TOPK_CAP) {  // uniform: cnt is stable between the barriers
                    const int kept = block_select(keys, &cnt, k, tid, MERGE_THREADS, sync);
                    if (kept == k) tau = keys[k - 1];
                }
                __syncthreads();
            }
        }
    }
    __syncthreads();
    const int kept = block_select(keys, &cnt, k, tid, MERGE_THREADS, sync);
    for (int i = tid; i < k; i += MERGE_THREADS) {
        int64_t id = -1;
        float dist = metric == RAGO_L2 ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
        if (i < kept) {
            const unsigned long long key = keys[i];
            id = ids[(uint32_t)(key & 0xFFFFFFFFull)];
            const float sc = orderable_f32((uint32_t)(key >> 32));
            dist = metric == RAGO_L2 ? sc : -sc;
        }
        out_ids[(size_t)q * k + i] = id;
        out_dists[(size_t)q * k + i] = dist;
    }
}

cudaError_t launch_merge(const IndexImpl* ix, const int64_t* work_prefix, int nq, int nprobe, int k, int ctas,
                         const int32_t* slot_cnt, const unsigned long long* slot_keys, const unsigned long long* qthresh,
                         int64_t* out_ids, float* out_dists, cudaStream_t s) {
    merge_kernel<<<nq, MERGE_THREADS, 0, s>>>(work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas, ix->metric,
                                              slot_cnt, slot_keys, qthresh, out_ids, out_dists);
    count_launch();
    return cudaGetLastError();
}

__global__ void fill_u64_kernel(unsigned long long* p, size_t n, unsigned long long v) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        p[i] = v;
}
cudaError_t launch_fill_u64(unsigned long long* p, size_t n, unsigned long long v, cudaStream_t s) {
    if (n == 0) return cudaSuccess;
    const int blocks = (int)((n + 255) / 256 < 1024 ? (n + 255) / 256 : 1024);
    fill_u64_kernel<<<blocks, 256, 0, s>>>(p, n, v);
    count_launch();
    return cudaGetLastError();
}

}  // namespace rago
