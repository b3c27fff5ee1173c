// Final top-k per query: merge the partial candidate lists the scan CTAs left behind, sort, map
// storage positions to caller ids, and write results best-first.
#include "topk.cuh"

namespace rago {

// Slot numbering: CTA b working on query q writes slot q + b.  Along the CTAs' contiguous walk over the
// batch that number strictly increases, so the slots of one query form one range (unused numbers in
// between have count 0).
__device__ __forceinline__ long long cta_of_unit(long long u, long long W, int ctas) {
    // CTA b owns units [b*W/ctas, (b+1)*W/ctas): the largest b with floor(b*W/ctas) <= u
    return ((u + 1) * ctas - 1) / W;
}

// One CTA per query.  Small batches use wide CTAs (few queries, each with a slot from almost every scan
// CTA), large batches narrow ones.
template <int THREADS>
__global__ void __launch_bounds__(THREADS) merge_kernel(
    const int64_t* __restrict__ work_prefix, const int64_t* __restrict__ ids, int npairs, int nprobe, int k, int ctas,
    int metric, const int32_t* __restrict__ slot_cnt, const unsigned long long* __restrict__ slot_keys,
    const unsigned long long* __restrict__ qthresh,
    int64_t* __restrict__ out_ids, float* __restrict__ out_dists) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    const int q = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto sync = [] { __syncthreads(); };
    grid_dependency_wait();
    grid_dependents_may_launch();
    if (tid == 0) cnt = 0;
    __syncthreads();
    const long long W = work_prefix[npairs];
    const long long u0 = work_prefix[(size_t)q * nprobe], u1 = work_prefix[(size_t)(q + 1) * nprobe];
    // a key above the threshold the scan CTAs agreed on is not among the k best (it is some CTA's k-th key)
    unsigned long long tau = qthresh[q];
    if (tau != KEY_MAX) ++tau;  // the threshold key itself is a result
    if (u1 > u0) {
        const long long s0 = (long long)q + cta_of_unit(u0, W, ctas);
        const int nslots = (int)((long long)q + cta_of_unit(u1 - 1, W, ctas) - s0) + 1;
        // Slot s holds slot_cnt[s] keys in ascending order.  First the leading m keys of every slot, about 2k keys
        // in all: the k-th smallest of them bounds the k-th smallest overall, and because every slot is a random
        // part of the query's work the bound is nearly tight.  Then the rest of the slots against that bound.
        int m = (2 * k + nslots - 1) / nslots;
        if (m > k) m = k;
        if ((long long)m * nslots > TOPK_CAP) m = TOPK_CAP / nslots;
        const int total_a = nslots * m;
        for (int e0 = 0; e0 < total_a; e0 += THREADS) {  // whole warps stay in the loop for warp_push
            const int e = e0 + tid;
            unsigned long long key = KEY_MAX;
            if (e < total_a) {
                const long long s = s0 + e / m;
                const int i = e % m;
                if (i < slot_cnt[s]) key = slot_keys[(size_t)s * k + i];
            }
            warp_push(keys, &cnt, key < tau, key);
        }
        __syncthreads();
        if (m < k) {
            if (cnt >= k) {
                block_select(keys, &cnt, k, tid, THREADS, sync);
                tau = keys[k - 1];
            }
            const int rem = k - m, total_b = nslots * rem;  // at most (scan CTAs + 1) * MAX_K entries
            // The rest of every slot against that bound, one warp per slot: the slot ascends, so the warp stops at
            // the first key that fails.  Usually a handful pass and one sort finishes the query; if they overflow
            // the buffer, the pass is abandoned and redone with intermediate selections.
            const int cnt_a = cnt;
            __syncthreads();
            for (int sl = warp; sl < nslots; sl += THREADS / 32) {
                const long long s = s0 + sl;
                const int c = slot_cnt[s];
                for (int i0 = m; i0 < c; i0 += 32) {
                    const int i = i0 + lane;
                    const unsigned long long key = i < c ? slot_keys[(size_t)s * k + i] : KEY_MAX;
                    warp_push(keys, &cnt, key < tau, key);
                    if (!__all_sync(0xffffffffu, key < tau)) break;
                }
            }
            __syncthreads();
            if (cnt > TOPK_CAP) {  // uniform; pushes beyond the buffer were dropped, the first cnt_a keys are intact
                __syncthreads();
                if (tid == 0) cnt = cnt_a;
                __syncthreads();
                // entries are fetched MERGE_BATCH per thread at a time (independent loads in flight), then pushed
                constexpr int MERGE_BATCH = 8;
                for (int e0 = 0; e0 < total_b; e0 += THREADS * MERGE_BATCH) {
                    unsigned long long mine[MERGE_BATCH];
#pragma unroll
                    for (int j = 0; j < MERGE_BATCH; ++j) {
                        const int e = e0 + j * THREADS + tid;
                        mine[j] = KEY_MAX;
                        if (e < total_b) {
                            const long long s = s0 + e / rem;
                            const int i = m + e % rem;
                            if (i < slot_cnt[s]) mine[j] = slot_keys[(size_t)s * k + i];
                        }
                    }
#pragma unroll
                    for (int j = 0; j < MERGE_BATCH; ++j) {
                        warp_push(keys, &cnt, mine[j] < tau, mine[j]);
                        __syncthreads();
                        if (cnt + THREADS > TOPK_CAP) {  // uniform: cnt is stable between the barriers
                            const int kept = block_select(keys, &cnt, k, tid, THREADS, sync);
                            if (kept == k) tau = keys[k - 1];
                        }
                        __syncthreads();
                    }
                }
            }
        }
    }
    __syncthreads();
    const int kept = block_select(keys, &cnt, k, tid, THREADS, sync);
    for (int i = tid; i < k; i += THREADS) {
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
    if (nq <= 64)
        launch_overlapped(merge_kernel<1024>, dim3(nq), dim3(1024), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, out_ids, out_dists);
    else
        launch_overlapped(merge_kernel<256>, dim3(nq), dim3(256), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, out_ids, out_dists);
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
