// Final top-k per query: merge the partial candidate lists the scan CTAs left behind, sort, map
// storage positions to caller ids, and write results best-first.
//
// Squared-L2 results whose terms cancel are re-scored before they are written.  The scan ranks candidates with
// the expanded form  bias + term + sum  =  ||q-c||^2 + (||r||^2 + 2<c,r>) - 2<q,r>,  whose rounding error is a
// few ulps of its LARGEST term T: harmless for ranking, but for a query that almost coincides with a stored
// vector the terms (tens to thousands) cancel to a distance of 1e-3 or less and the relative error of the sum
// becomes large.  A winner whose value is below T / 32 (relative error of the expanded form possibly above
// ~1e-5; T is known at this point from the list's bias and the vector's stored term) is therefore scored again
// in the direct form  sum_j ((q_j - c_j) - cw_j)^2  (all terms non-negative: relative error about sqrt(d) ulps),
// and the winners are re-ordered if any value changed.  On ordinary data no winner qualifies and the check costs
// one 4-byte load per winner.
#include "topk.cuh"

namespace rago {

struct RescoreArgs {
    int enabled;                 // squared L2 only
    const float* queries;        // [nq][d]
    const void* centroids;       // [nlist][d] fp32 or bf16
    int coarse_bf16;
    const float* cbT;            // [256][M][dsub]: the library's own copy of the codebook, codeword index outermost
    const uint8_t* codes;        // [N][M]
    const int64_t* list_offsets; // [nlist + 1]
    const int32_t* probe_list;   // [nq][nprobe]: a result lies in one of the lists its query probed
    const float* probe_bias;     // [nq][nprobe]: ||q - c||^2 of those lists (the scan's per-list term)
    const float* vterm;          // [N]: the scan's per-vector term
    int nlist, d, M, dsub;
};

// ||q - (c_list + decoded codewords)||^2 of the vector at storage position pos, which lies in inverted list
// `list`, by one warp (d a multiple of 4).  All of a lane's loads are independent of each other except the
// codeword, which follows its code byte.
__device__ __forceinline__ float direct_l2(const RescoreArgs& r, const float* qrow, uint32_t pos, int list, int lane) {
    const uint8_t* code = r.codes + (size_t)pos * r.M;
    float acc = 0.f;
    for (int j = lane * 4; j < r.d; j += 128) {
        const float4 qv = *reinterpret_cast<const float4*>(qrow + j);
        float c[4], cw[4];
        if (r.coarse_bf16) {
            const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(r.centroids) + (size_t)list * r.d + j);
            c[0] = __uint_as_float(raw.x << 16); c[1] = __uint_as_float(raw.x & 0xFFFF0000u);
            c[2] = __uint_as_float(raw.y << 16); c[3] = __uint_as_float(raw.y & 0xFFFF0000u);
        } else {
            const float4 cv = *reinterpret_cast<const float4*>(static_cast<const float*>(r.centroids) + (size_t)list * r.d + j);
            c[0] = cv.x; c[1] = cv.y; c[2] = cv.z; c[3] = cv.w;
        }
        if ((r.dsub & 3) == 0) {  // the four dimensions share a sub-space: one code byte, one 16-byte codeword load
            const int m = j / r.dsub, t = j - m * r.dsub;
            const float4 w = __ldg(reinterpret_cast<const float4*>(r.cbT + ((size_t)code[m] * r.M + m) * r.dsub + t));
            cw[0] = w.x; cw[1] = w.y; cw[2] = w.z; cw[3] = w.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int jj = j + i, m = jj / r.dsub, t = jj - m * r.dsub;
                cw[i] = __ldg(r.cbT + ((size_t)code[m] * r.M + m) * r.dsub + t);
            }
        }
        const float qq[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float e = (qq[i] - c[i]) - cw[i];  // residual first, as the definition forms it
            acc = fmaf(e, e, acc);
        }
    }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

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
    const unsigned long long* __restrict__ qthresh, const RescoreArgs rs,
    int64_t* __restrict__ out_ids, float* __restrict__ out_dists) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    __shared__ int p_list[MAX_K];          // re-scoring: the query's probed lists and their storage ranges
    __shared__ uint32_t p_lo[MAX_K], p_hi[MAX_K];
    __shared__ int redo[MAX_K], redo_list[MAX_K];  // winners to score again (index into keys) and their lists
    __shared__ int nredo;
    const int q = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto sync = [] { __syncthreads(); };
    grid_dependency_wait();
    grid_dependents_may_launch();
    if (tid == 0) { cnt = 0; nredo = 0; }
    if (rs.enabled) {
        for (int i = tid; i < nprobe; i += THREADS) {
            const int l = rs.probe_list[(size_t)q * nprobe + i];
            p_list[i] = l;
            p_lo[i] = (uint32_t)rs.list_offsets[l];
            p_hi[i] = (uint32_t)rs.list_offsets[l + 1];
        }
    }
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
                block_select_short(keys, &cnt, k, tid, THREADS, sync);
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
    int kept = block_select_short(keys, &cnt, k, tid, THREADS, sync);
    if (rs.enabled && kept > 0) {  // uniform
        // which winners lost too many bits to cancellation: one thread per winner
        for (int i = tid; i < kept; i += THREADS) {
            const uint32_t pos = (uint32_t)(keys[i] & 0xFFFFFFFFull);
            int p = 0;
            while (p < nprobe && !(pos >= p_lo[p] && pos < p_hi[p])) ++p;
            if (p == nprobe) continue;  // cannot happen: every candidate comes from a probed list
            const float dist = orderable_f32((uint32_t)(keys[i] >> 32));
            const float bias = rs.probe_bias[(size_t)q * nprobe + p], vt = rs.vterm[pos];
            const float T = fmaxf(fmaxf(bias, fabsf(vt)), fabsf(dist - (bias + vt)));
            if (dist < T * (1.f / 32.f)) {
                const int at = atomicAdd(&nredo, 1);
                redo[at] = i;
                redo_list[at] = p_list[p];
            }
        }
        __syncthreads();
        const int nr = nredo;
        if (nr > 0) {  // uniform
            const float* qrow = rs.queries + (size_t)q * rs.d;
            for (int e = warp; e < nr; e += THREADS / 32) {
                const int i = redo[e];
                const uint32_t pos = (uint32_t)(keys[i] & 0xFFFFFFFFull);
                const float dist = direct_l2(rs, qrow, pos, redo_list[e], lane);
                __syncwarp();
                if (lane == 0) keys[i] = make_key(dist, pos);
            }
            __syncthreads();
            if (tid == 0) cnt = kept;
            __syncthreads();
            kept = block_select_short(keys, &cnt, k, tid, THREADS, sync);  // order by the new values
        }
    }
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

// Small batches (latency): the same result by a shorter chain of dependent memory accesses.  A query's slots are
// consecutive in memory, so the CTA's 1024 threads fetch ALL of their keys (at most KPT each) and the slot counts in
// one round trip, keep them in registers, find a cut with between k and k + k/4 + 8 keys at or below it by a counting
// bisection on the 64-bit keys (distinct, so it always ends), and only the keys up to the cut go to shared memory to
// be sorted.  The ids of the winners are fetched together with the values the cancellation check needs.
template <int KPT>
__global__ void __launch_bounds__(1024) merge_small_kernel(
    const int64_t* __restrict__ work_prefix, const int64_t* __restrict__ ids, int npairs, int nprobe, int k, int ctas,
    int metric, const int32_t* __restrict__ slot_cnt, const unsigned long long* __restrict__ slot_keys,
    const unsigned long long* __restrict__ qthresh, const RescoreArgs rs,
    int64_t* __restrict__ out_ids, float* __restrict__ out_dists) {
    constexpr int THREADS = 1024, BUF = 2 * MAX_K;
    __shared__ unsigned long long keys[BUF];
    __shared__ int cnt;
    __shared__ unsigned long long s_mn, s_mx;
    __shared__ uint32_t s_nv, s_round[3];
    __shared__ int p_list[MAX_K];
    __shared__ uint32_t p_lo[MAX_K], p_hi[MAX_K];
    __shared__ int redo[MAX_K], redo_list[MAX_K];
    __shared__ int nredo;
    const int q = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto sync = [] { __syncthreads(); };
    grid_dependency_wait();
    grid_dependents_may_launch();
    if (tid == 0) { cnt = 0; nredo = 0; s_mn = KEY_MAX; s_mx = 0ull; s_nv = 0u; s_round[0] = s_round[1] = s_round[2] = 0u; }
    const long long W = work_prefix[npairs];
    const long long u0 = work_prefix[(size_t)q * nprobe], u1 = work_prefix[(size_t)(q + 1) * nprobe];
    unsigned long long tau = qthresh[q];
    if (tau != KEY_MAX) ++tau;  // the threshold key itself is a result
    if (rs.enabled) {
        for (int i = tid; i < nprobe; i += THREADS) {
            const int l = rs.probe_list[(size_t)q * nprobe + i];
            p_list[i] = l;
            p_lo[i] = (uint32_t)rs.list_offsets[l];
            p_hi[i] = (uint32_t)rs.list_offsets[l + 1];
        }
    }
    unsigned long long mine[KPT];
#pragma unroll
    for (int j = 0; j < KPT; ++j) mine[j] = KEY_MAX;
    if (u1 > u0) {
        const long long s0 = (long long)q + cta_of_unit(u0, W, ctas);
        const int nslots = (int)((long long)q + cta_of_unit(u1 - 1, W, ctas) - s0) + 1;
        const int total = nslots * k;  // at most KPT * THREADS: the launcher checked (ctas + 1) * k
        const unsigned long long* src = slot_keys + (size_t)s0 * k;
        const int32_t* csrc = slot_cnt + s0;
#pragma unroll
        for (int j = 0; j < KPT; ++j) {
            const int e = tid + j * THREADS;
            if (e < total) {
                const int sl = e / k, i = e - sl * k;
                const int c = csrc[sl];
                const unsigned long long key = src[e];  // entries past a slot's count are stale, never out of bounds
                if (i < c && key < tau) mine[j] = key;
            }
        }
    }
    unsigned long long mn = KEY_MAX, mx = 0ull;
    uint32_t nv = 0;
#pragma unroll
    for (int j = 0; j < KPT; ++j)
        if (mine[j] != KEY_MAX) { mn = mine[j] < mn ? mine[j] : mn; mx = mine[j] > mx ? mine[j] : mx; ++nv; }
    __syncthreads();  // the shared words are initialised
    nv = __reduce_add_sync(0xffffffffu, nv);
    if (nv) {  // uniform within the warp
        for (int o = 16; o; o >>= 1) {
            const unsigned long long a = shfl_xor_u64(mn, o), b = shfl_xor_u64(mx, o);
            mn = a < mn ? a : mn; mx = b > mx ? b : mx;
        }
        if (lane == 0) { atomicMin(&s_mn, mn); atomicMax(&s_mx, mx); atomicAdd(&s_nv, nv); }
    }
    __syncthreads();
    mn = s_mn; mx = s_mx;
    const uint32_t nvalid = s_nv;
    uint32_t want_max = (uint32_t)(k + (k >> 2) + 8);  // <= BUF
    if (want_max < (uint32_t)WARP_SORT_MAX) want_max = WARP_SORT_MAX;  // as many as the short selection ranks in one go
    unsigned long long T = mx;  // keys up to T are collected
    if (nvalid > want_max) {    // uniform.  k >= 2 here would not be needed: count(<= mn) = 1 <= k always
        unsigned long long lo = mn, hi = mx;  // #(key <= lo) <= k  and  #(key <= hi) >= k; lo itself is always kept
        uint32_t c_hi = nvalid;
        int round = 0;
        if (k > 1) {
            while (hi - lo > 1 && c_hi > want_max) {  // uniform
                const unsigned long long mid = lo + (hi - lo) / 2;
                uint32_t c = 0;
#pragma unroll
                for (int j = 0; j < KPT; ++j) c += mine[j] <= mid ? 1u : 0u;  // mid < mx < the empty-slot pattern
                c = __reduce_add_sync(0xffffffffu, c);
                const int slot = round % 3;
                if (lane == 0 && c) atomicAdd(&s_round[slot], c);
                if (tid == 0) s_round[(slot + 1) % 3] = 0u;  // next round's word; its last readers passed two barriers ago
                __syncthreads();
                c = s_round[slot];
                if (c < (uint32_t)k) lo = mid; else { hi = mid; c_hi = c; }
                ++round;
            }
            T = hi;
        } else {
            T = mn;
        }
    }
#pragma unroll
    for (int j = 0; j < KPT; ++j) warp_push(keys, &cnt, mine[j] <= T && mine[j] != KEY_MAX, mine[j], BUF);
    __syncthreads();
    int kept = block_select_short(keys, &cnt, k, tid, THREADS, sync, BUF);
    // winners: id, and whether too many bits were lost to cancellation (one thread per winner, loads side by side)
    int64_t my_id = -1;
    unsigned long long my_key = KEY_MAX;
    if (tid < kept) {
        my_key = keys[tid];
        const uint32_t pos = (uint32_t)(my_key & 0xFFFFFFFFull);
        my_id = ids[pos];
        if (rs.enabled) {
            int p = 0;
            while (p < nprobe && !(pos >= p_lo[p] && pos < p_hi[p])) ++p;
            if (p < nprobe) {  // always: every candidate comes from a probed list
                const float dist = orderable_f32((uint32_t)(my_key >> 32));
                const float bias = rs.probe_bias[(size_t)q * nprobe + p], vt = rs.vterm[pos];
                const float Tm = fmaxf(fmaxf(bias, fabsf(vt)), fabsf(dist - (bias + vt)));
                if (dist < Tm * (1.f / 32.f)) {
                    const int at = atomicAdd(&nredo, 1);
                    redo[at] = tid;
                    redo_list[at] = p_list[p];
                }
            }
        }
    }
    if (rs.enabled && kept > 0) {  // uniform
        __syncthreads();
        const int nr = nredo;
        if (nr > 0) {  // uniform
            const float* qrow = rs.queries + (size_t)q * rs.d;
            for (int e = warp; e < nr; e += THREADS / 32) {
                const int i = redo[e];
                const uint32_t pos = (uint32_t)(keys[i] & 0xFFFFFFFFull);
                const float dist = direct_l2(rs, qrow, pos, redo_list[e], lane);
                __syncwarp();
                if (lane == 0) keys[i] = make_key(dist, pos);
            }
            __syncthreads();
            if (tid == 0) cnt = kept;
            __syncthreads();
            kept = block_select_short(keys, &cnt, k, tid, THREADS, sync, BUF);  // order by the new values
            if (tid < kept) { my_key = keys[tid]; my_id = ids[(uint32_t)(my_key & 0xFFFFFFFFull)]; }
        }
    }
    for (int i = tid; i < k; i += THREADS) {  // k <= MAX_K = THREADS: one round
        float dist = metric == RAGO_L2 ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
        int64_t id = -1;
        if (i < kept) {
            id = my_id;
            const float sc = orderable_f32((uint32_t)(my_key >> 32));
            dist = metric == RAGO_L2 ? sc : -sc;
        }
        out_ids[(size_t)q * k + i] = id;
        out_dists[(size_t)q * k + i] = dist;
    }
}

cudaError_t launch_merge(const IndexImpl* ix, const int64_t* work_prefix, int nq, int nprobe, int k, int ctas,
                         const int32_t* slot_cnt, const unsigned long long* slot_keys, const unsigned long long* qthresh,
                         const float* queries, const int32_t* probe_list, const float* probe_bias, int64_t* out_ids,
                         float* out_dists, cudaStream_t s) {
    RescoreArgs rs;
    rs.enabled = ix->metric == RAGO_L2 && ix->vterm != nullptr && ix->d % 4 == 0 ? 1 : 0;
    rs.queries = queries; rs.centroids = ix->centroids; rs.coarse_bf16 = ix->coarse_bf16; rs.cbT = ix->cbT;
    rs.codes = ix->codes; rs.list_offsets = ix->list_offsets; rs.probe_list = probe_list;
    rs.probe_bias = probe_bias; rs.vterm = ix->vterm; rs.nlist = ix->nlist; rs.d = ix->d; rs.M = ix->M;
    rs.dsub = ix->dsub;
    const long long worst = (long long)(ctas + 1) * k;  // keys of one query's slots, at most
    if (nq <= 64 && worst <= 4 * 1024)
        launch_overlapped(merge_small_kernel<4>, dim3(nq), dim3(1024), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, rs, out_ids, out_dists);
    else if (nq <= 64 && worst <= 16 * 1024)
        launch_overlapped(merge_small_kernel<16>, dim3(nq), dim3(1024), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, rs, out_ids, out_dists);
    else if (nq <= 64)
        launch_overlapped(merge_kernel<1024>, dim3(nq), dim3(1024), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, rs, out_ids, out_dists);
    else
        launch_overlapped(merge_kernel<256>, dim3(nq), dim3(256), 0, s, work_prefix, ix->ids, nq * nprobe, nprobe, k, ctas,
                          ix->metric, slot_cnt, slot_keys, qthresh, rs, out_ids, out_dists);
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
