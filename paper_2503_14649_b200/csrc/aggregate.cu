// rago_merge_results: aggregation of the answers of independently indexed database shards.
// Every shard has searched the same query batch; for each query the best k_out entries of the union
// of the shards' result lists are selected and written best first.
#include "topk.cuh"

namespace rago {

constexpr int AGG_THREADS = 256;

// One CTA per query.  Entry e = (part e / k_in, rank e % k_in); its key is (score, e), so equal scores
// keep the order (part, rank).  Padding entries (id < 0) are skipped.
__global__ void __launch_bounds__(AGG_THREADS) aggregate_kernel(
    const int64_t* __restrict__ part_ids, const float* __restrict__ part_dists, int nparts, long long part_stride,
    int k_in, int k_out, int metric, int64_t* __restrict__ out_ids, float* __restrict__ out_dists) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    const int q = blockIdx.x, tid = threadIdx.x;
    auto sync = [] { __syncthreads(); };
    if (tid == 0) cnt = 0;
    __syncthreads();
    const int total = nparts * k_in;
    const size_t row = (size_t)q * k_in;
    unsigned long long tau = KEY_MAX;
    for (int e0 = 0; e0 < total; e0 += AGG_THREADS) {
        const int e = e0 + tid;
        unsigned long long key = KEY_MAX;
        bool pred = false;
        if (e < total) {
            const size_t off = (size_t)(e / k_in) * part_stride + row + (e % k_in);
            if (part_ids[off] >= 0) {
                const float d = part_dists[off];
                key = make_key(metric == RAGO_L2 ? d : -d, (uint32_t)e);
                pred = key < tau;
            }
        }
        warp_push(keys, &cnt, pred, key);
        __syncthreads();
        if (cnt + AGG_THREADS > TOPK_CAP) {  // uniform: cnt is stable between the barriers
            const int kept = block_select(keys, &cnt, k_out, tid, AGG_THREADS, sync);
            if (kept == k_out) tau = keys[k_out - 1];
        }
        __syncthreads();
    }
    const int kept = block_select(keys, &cnt, k_out, tid, AGG_THREADS, sync);
    for (int i = tid; i < k_out; i += AGG_THREADS) {
        int64_t id = -1;
        float dist = metric == RAGO_L2 ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
        if (i < kept) {
            const int e = (int)(uint32_t)(keys[i] & 0xFFFFFFFFull);
            const size_t off = (size_t)(e / k_in) * part_stride + row + (e % k_in);
            id = part_ids[off];
            dist = part_dists[off];
        }
        out_ids[(size_t)q * k_out + i] = id;
        out_dists[(size_t)q * k_out + i] = dist;
    }
}

}  // namespace rago

using namespace rago;

extern "C" rago_status rago_merge_results(const int64_t* part_ids, const float* part_dists, int32_t nparts,
                                          int64_t part_stride, int32_t nq, int32_t k_in, int32_t k_out,
                                          int32_t metric, int64_t* out_ids, float* out_dists, void* cuda_stream) {
    if (nparts < 1 || k_in < 1 || k_out < 1 || nq < 0) {
        set_error("nparts = %d, k_in = %d, k_out = %d must be >= 1 and nq = %d >= 0", nparts, k_in, k_out, nq);
        return RAGO_EINVAL;
    }
    if (metric != RAGO_L2 && metric != RAGO_IP) { set_error("metric = %d is neither L2 nor IP", metric); return RAGO_EINVAL; }
    if (k_out > MAX_K) { set_error("k_out = %d exceeds %d", k_out, MAX_K); return RAGO_EUNSUPPORTED; }
    if ((long long)nparts * k_in > 0x7fffffffLL) {
        set_error("nparts * k_in = %lld exceeds 2^31 - 1", (long long)nparts * k_in);
        return RAGO_EUNSUPPORTED;
    }
    if (part_stride < (int64_t)nq * k_in) {
        set_error("part_stride = %lld is smaller than nq * k_in = %lld", (long long)part_stride, (long long)nq * k_in);
        return RAGO_EINVAL;
    }
    if (nq == 0) return RAGO_OK;
    if (!part_ids || !part_dists || !out_ids || !out_dists) { set_error("null pointer"); return RAGO_EINVAL; }
    aggregate_kernel<<<nq, AGG_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        part_ids, part_dists, nparts, (long long)part_stride, k_in, k_out, metric, out_ids, out_dists);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("aggregate kernel: %s", cudaGetErrorString(e)); return RAGO_ECUDA; }
    return RAGO_OK;
}
