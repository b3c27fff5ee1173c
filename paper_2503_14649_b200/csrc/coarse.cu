// Coarse quantiser: query x centroid scores and per-query nprobe selection.
//
// Ranking score, smaller is better:  L2: ||c||^2 - 2<q,c>  (same order as ||q-c||^2),  IP: -<q,c>.
// The nprobe + PROBE_GUARD best lists by that score are re-scored exactly (sum of (q-c)^2, or <q,c>)
// before the final cut, so the probe order follows the plain definition up to fp32 rounding.
// With a bf16 coarse quantiser the query is rounded to bf16 first (coarse step only).
#include <cstring>

#include "plan.cuh"
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

// ---- score matrix for tiny batches (the latency-bound iterative-retrieval shape) -------------------
// For up to CS_MAXQ queries: a warp takes CS_CPW centroid rows at a time and keeps one partial sum per (row, query),
// so the centroid table is read exactly once per batch however few queries there are.  The launch is bound by the
// latency of the table's reads (a few rows per warp, and between two searches the scan pushes much of the table out
// of L2), so a warp asks for CS_CPW x 512 values before it multiplies any of them: 8 KB in flight per warp.  NQ
// (1, 4 or 16) bounds the batch at compile time: the partial sums and their reduction shrink with it; 16 queries are
// multiplied in two groups of 8 against the same registers, because 64 sums beside 64 row values do not fit (with
// half as many values in flight and the next round prefetched the same launch took twice as long).  The grid is
// sized so that most warps have a single step.
constexpr int CS_MAXQ = 16;
constexpr int CS_CPW = 4;    // centroids per warp per step
template <bool BF16, int NQ>
__global__ void __launch_bounds__(256) coarse_small_kernel(const float* __restrict__ Q, const void* __restrict__ C,
                                                           const float* __restrict__ cnorm, int nq, int nlist, int d,
                                                           int metric, float* __restrict__ scores, uint32_t* __restrict__ clear_block) {
    extern __shared__ __align__(16) float qs[];  // [nq][d], rounded to bf16 values for a bf16 index
    grid_dependency_wait();
    grid_dependents_may_launch();
    // first kernel of a search: the workspace's 256-byte error block (error word, ticket) starts at zero; doing it
    // here instead of in a memset of its own keeps two searches on one stream overlapping their launches
    if (clear_block != nullptr && blockIdx.x == 0 && threadIdx.x < 64) clear_block[threadIdx.x] = 0u;
    {   // d is a multiple of 4 and Q 16-byte aligned; eight 16-byte loads in flight per thread
        const int n4 = (nq * d) >> 2;
        const float4* Q4 = reinterpret_cast<const float4*>(Q);
        float4* qs4 = reinterpret_cast<float4*>(qs);
        for (int i0 = threadIdx.x; i0 < n4; i0 += 8 * 256) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = i0 + u * 256 < n4 ? __ldg(Q4 + i0 + u * 256) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (BF16) { v[u].x = round_bf16(v[u].x); v[u].y = round_bf16(v[u].y); v[u].z = round_bf16(v[u].z); v[u].w = round_bf16(v[u].w); }
                if (i0 + u * 256 < n4) qs4[i0 + u * 256] = v[u];
            }
        }
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    constexpr int QG = NQ <= 4 ? NQ : 8;   // queries multiplied against the rows held in registers at a time
    constexpr int NGROUPS = NQ / QG;
    constexpr int CHUNK = 4;               // 16-byte (fp32) / 8-byte (bf16) loads per lane and row in one round: 512 values
    for (int c0 = ((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * CS_CPW; c0 < nlist; c0 += warps * CS_CPW) {
        float cn[CS_CPW];
#pragma unroll
        for (int u = 0; u < CS_CPW; ++u) cn[u] = metric == RAGO_L2 ? __ldg(cnorm + (c0 + u < nlist ? c0 + u : nlist - 1)) : 0.f;
        float4 cv[CS_CPW][CHUNK];
        auto load_rows = [&](int jb) {
#pragma unroll
            for (int u = 0; u < CS_CPW; ++u) {
                const int c = c0 + u < nlist ? c0 + u : nlist - 1;  // rows past the end repeat the last one, unused
#pragma unroll
                for (int h = 0; h < CHUNK; ++h) {
                    const int j0 = jb + h * 128 + lane * 4;
                    if (j0 < d) {
                        if (BF16) {
                            const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(C) + (size_t)c * d + j0);
                            cv[u][h].x = __uint_as_float(raw.x << 16); cv[u][h].y = __uint_as_float(raw.x & 0xFFFF0000u);
                            cv[u][h].z = __uint_as_float(raw.y << 16); cv[u][h].w = __uint_as_float(raw.y & 0xFFFF0000u);
                        } else {
                            cv[u][h] = *reinterpret_cast<const float4*>(static_cast<const float*>(C) + (size_t)c * d + j0);
                        }
                    } else {
                        cv[u][h] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
        };
#pragma unroll
        for (int g = 0; g < NGROUPS; ++g) {
            if (g * QG >= nq) break;  // uniform
            float acc[CS_CPW][QG];
#pragma unroll
            for (int u = 0; u < CS_CPW; ++u)
#pragma unroll
                for (int qi = 0; qi < QG; ++qi) acc[u][qi] = 0.f;
            for (int jb = 0; jb < d; jb += 128 * CHUNK) {
                // the rows of a block of 512 values stay in registers for every group of queries; a longer row is
                // read again for the second group (from the caches)
                if (g == 0 || d > 128 * CHUNK) load_rows(jb);
#pragma unroll
                for (int h = 0; h < CHUNK; ++h) {
                    const int j0 = jb + h * 128 + lane * 4;
                    if (j0 < d) {
#pragma unroll
                        for (int qi = 0; qi < QG; ++qi) {
                            if (g * QG + qi < nq) {  // uniform
                                const float4 qv = *reinterpret_cast<const float4*>(qs + (g * QG + qi) * d + j0);
#pragma unroll
                                for (int u = 0; u < CS_CPW; ++u)
                                    acc[u][qi] = fmaf(qv.x, cv[u][h].x, fmaf(qv.y, cv[u][h].y, fmaf(qv.z, cv[u][h].z, fmaf(qv.w, cv[u][h].w, acc[u][qi]))));
                            }
                        }
                    }
                }
            }
            // Sum over the lanes, all QG queries of a row at once: at each halving a lane keeps the half of its values
            // that its lane-number bit selects and hands over the other half (QG - 1 exchanges instead of 5 QG), then
            // the single value left is summed over the remaining lane bits.  The total of the query whose number is
            // the leading log2(QG) lane bits ends in the lanes whose other bits are clear.
#pragma unroll
            for (int u = 0; u < CS_CPW; ++u) {
                int o = 16;
#pragma unroll
                for (int half = QG / 2; half >= 1; half >>= 1, o >>= 1) {
                    const bool upper = (lane & o) != 0;
#pragma unroll
                    for (int i = 0; i < half; ++i) {
                        const float keep = upper ? acc[u][i + half] : acc[u][i];
                        const float send = upper ? acc[u][i] : acc[u][i + half];
                        acc[u][i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                    }
                }
                float v = acc[u][0];
#pragma unroll
                for (; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                constexpr int REST = 32 / QG;  // lanes that end up with the same query's total
                const int qi = g * QG + (QG == 1 ? 0 : (lane / REST));
                if ((lane & (REST - 1)) == 0 && qi < nq && c0 + u < nlist)
                    scores[(size_t)qi * nlist + c0 + u] = metric == RAGO_L2 ? fmaf(-2.f, v, cn[u]) : -v;
            }
        }
    }
}

template <bool BF16>
static void launch_coarse_small(const IndexImpl* ix, const float* queries, int nq, float* scores, int blocks, size_t qbytes,
                                uint32_t* clear_block, cudaStream_t s) {
    if (nq == 1)
        launch_overlapped(coarse_small_kernel<BF16, 1>, dim3(blocks), dim3(256), qbytes, s, queries, ix->centroids, ix->cnorm,
                          nq, ix->nlist, ix->d, ix->metric, scores, clear_block);
    else if (nq <= 4)
        launch_overlapped(coarse_small_kernel<BF16, 4>, dim3(blocks), dim3(256), qbytes, s, queries, ix->centroids, ix->cnorm,
                          nq, ix->nlist, ix->d, ix->metric, scores, clear_block);
    else
        launch_overlapped(coarse_small_kernel<BF16, CS_MAXQ>, dim3(blocks), dim3(256), qbytes, s, queries, ix->centroids,
                          ix->cnorm, nq, ix->nlist, ix->d, ix->metric, scores, clear_block);
}

bool coarse_small_applies(const IndexImpl* ix, int nq) { return nq <= CS_MAXQ && (size_t)nq * ix->d * 4 <= 48 * 1024; }

// clear_block (may be null): 64 words the tiny-batch kernel zeroes before anything else of the search runs; only
// valid when coarse_small_applies().
cudaError_t launch_coarse_scores(const IndexImpl* ix, const float* queries, int nq, float* scores, uint32_t* clear_block,
                                 cudaStream_t s) {
    const size_t qbytes = (size_t)nq * ix->d * 4;
    if (coarse_small_applies(ix, nq)) {
        const int want = (ix->nlist + 8 * CS_CPW - 1) / (8 * CS_CPW);  // 8 warps per CTA, CS_CPW rows per warp step
        const int cap = ix->num_sms * (nq <= 4 ? 4 : 2);
        const int blocks = want < cap ? want : cap;
        if (ix->coarse_bf16) launch_coarse_small<true>(ix, queries, nq, scores, blocks, qbytes, clear_block, s);
        else launch_coarse_small<false>(ix, queries, nq, scores, blocks, qbytes, clear_block, s);
        count_launch();
        return cudaGetLastError();
    }
    if (clear_block != nullptr) return cudaErrorInvalidValue;
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

// ---- two-level coarse quantiser: candidates of a query through the first level -------------------------------
// The paper's index is a multi-level tree whose levels are scanned top-down (Methodology, "Models and database"
// and the retrieval performance model).  With one level above the coarse centroids: score the n1 level-1
// centroids, keep the best b1 nodes, and only the coarse centroids that are their children become candidates for
// the nprobe selection.  Children of node i are the consecutive lists child_offsets[i] .. child_offsets[i+1]-1.
//
// grid (S, nq): the S CTAs of a query all score the whole first level (n1 rows, L2-resident) and reach the same
// b1 nodes; then CTA s scores its share of the candidate slots (the children of the chosen nodes, in node-rank
// order) and leaves them as raw candidate entries {list, score bits} in cand[q][s][cap] with count cand_cnt[q][s],
// the format select_probes_kernel reads.  Level-1 scores use the direct form (sum (q-c)^2 or <q,c>), so that
// near-ties between nodes are decided as the definition decides them up to fp32 rounding; candidate scores are
// the ranking form of the one-level path (||c||^2 - 2<q,c> or -<q,c>).
constexpr int TREE_THREADS = 512;
constexpr int TREE_RPW = 4;        // rows a warp scores at a time (independent loads in flight)
constexpr int TREE_MAX_B1 = 64;

// Scores of TREE_RPW rows against the query in shared memory, by one warp: DIRECT: sum (q-c)^2 / <q,c> by metric;
// else <q,c> only.  Rows past `nrows` repeat the last valid one.  out[u] valid in every lane.
template <bool BF16, bool DIRECT>
__device__ __forceinline__ void warp_score_rows(const float* qs, const void* C, const int (&row)[TREE_RPW], int d,
                                                int metric, int lane, float (&out)[TREE_RPW]) {
    float acc[TREE_RPW];
#pragma unroll
    for (int u = 0; u < TREE_RPW; ++u) acc[u] = 0.f;
#pragma unroll 4
    for (int j0 = lane * 4; j0 < d; j0 += 128) {  // unrolled: the loads of four steps are in flight together
        float4 cv[TREE_RPW];
#pragma unroll
        for (int u = 0; u < TREE_RPW; ++u) {
            if (BF16) {
                const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(C) + (size_t)row[u] * d + j0);
                cv[u].x = __uint_as_float(raw.x << 16); cv[u].y = __uint_as_float(raw.x & 0xFFFF0000u);
                cv[u].z = __uint_as_float(raw.y << 16); cv[u].w = __uint_as_float(raw.y & 0xFFFF0000u);
            } else {
                cv[u] = *reinterpret_cast<const float4*>(static_cast<const float*>(C) + (size_t)row[u] * d + j0);
            }
        }
        const float4 qv = *reinterpret_cast<const float4*>(qs + j0);
#pragma unroll
        for (int u = 0; u < TREE_RPW; ++u) {
            if (DIRECT && metric == RAGO_L2) {
                const float t0 = qv.x - cv[u].x, t1 = qv.y - cv[u].y, t2 = qv.z - cv[u].z, t3 = qv.w - cv[u].w;
                acc[u] = fmaf(t0, t0, fmaf(t1, t1, fmaf(t2, t2, fmaf(t3, t3, acc[u]))));
            } else {
                acc[u] = fmaf(qv.x, cv[u].x, fmaf(qv.y, cv[u].y, fmaf(qv.z, cv[u].z, fmaf(qv.w, cv[u].w, acc[u]))));
            }
        }
    }
#pragma unroll
    for (int u = 0; u < TREE_RPW; ++u) {
        for (int o = 16; o; o >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], o);
        out[u] = acc[u];
    }
}

template <bool BF16>
__global__ void __launch_bounds__(TREE_THREADS) tree_candidates_kernel(
    const float* __restrict__ Q, const void* __restrict__ C1, const int32_t* __restrict__ child_offsets, int n1, int b1,
    const void* __restrict__ C, const float* __restrict__ cnorm, int d, int metric, int cap,
    unsigned long long* __restrict__ cand, int32_t* __restrict__ cand_cnt, uint32_t* __restrict__ clear_block) {
    extern __shared__ __align__(16) float tree_smem[];  // [d] query, [n1] level-1 keys as two words each
    float* qs = tree_smem;
    unsigned long long* k1 = reinterpret_cast<unsigned long long*>(tree_smem + ((d + 3) & ~3));  // (d * 4) % 16 == 0
    __shared__ int sel_node[TREE_MAX_B1];     // chosen nodes, best first
    __shared__ int sel_first[TREE_MAX_B1];    // first list of each chosen node
    __shared__ int sel_pre[TREE_MAX_B1 + 1];  // candidate slots before each chosen node
    const int q = blockIdx.y, s = blockIdx.x, S = gridDim.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int NW = TREE_THREADS / 32;
    grid_dependency_wait();
    grid_dependents_may_launch();
    // first kernel of a search: the workspace's error block starts at zero (see coarse_small_kernel)
    if (clear_block != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && tid < 64) clear_block[tid] = 0u;
    for (int i = tid; i < d; i += TREE_THREADS) qs[i] = BF16 ? round_bf16(Q[(size_t)q * d + i]) : Q[(size_t)q * d + i];
    __syncthreads();
    // first level: every node, direct form
    for (int r0 = warp * TREE_RPW; r0 < n1; r0 += NW * TREE_RPW) {
        int row[TREE_RPW];
#pragma unroll
        for (int u = 0; u < TREE_RPW; ++u) row[u] = r0 + u < n1 ? r0 + u : n1 - 1;
        float sc[TREE_RPW];
        warp_score_rows<BF16, true>(qs, C1, row, d, metric, lane, sc);
        if (lane == 0) {
#pragma unroll
            for (int u = 0; u < TREE_RPW; ++u)
                if (r0 + u < n1) k1[r0 + u] = make_key(metric == RAGO_L2 ? sc[u] : -sc[u], (uint32_t)(r0 + u));
        }
    }
    __syncthreads();
    // the b1 best nodes, best first (ties: smaller node), by warp 0: b1 rounds of a minimum over the keys
    if (warp == 0) {
        unsigned long long last = 0ull;
        bool first = true;
        for (int r = 0; r < b1; ++r) {
            unsigned long long best = KEY_MAX;
            for (int i = lane; i < n1; i += 32) {
                const unsigned long long k = k1[i];
                if ((first || k > last) && k < best) best = k;  // keys are distinct: the node number is part of them
            }
            for (int o = 16; o; o >>= 1) {
                const unsigned long long other = shfl_xor_u64(best, o);
                best = other < best ? other : best;
            }
            last = best;
            first = false;
            if (lane == 0) sel_node[r] = (int)(best & 0xFFFFFFFFull);
        }
        __syncwarp();
        // the chosen nodes' child ranges: all loads at once, then a running sum (b1 <= 64: two values per lane)
        int cnt0 = 0, cnt1 = 0;
        if (lane < b1) { const int n = sel_node[lane]; const int f = child_offsets[n]; sel_first[lane] = f; cnt0 = child_offsets[n + 1] - f; }
        if (lane + 32 < b1) { const int n = sel_node[lane + 32]; const int f = child_offsets[n]; sel_first[lane + 32] = f; cnt1 = child_offsets[n + 1] - f; }
        int inc0 = cnt0, inc1 = cnt1;
        for (int o = 1; o < 32; o <<= 1) {
            const int y0 = __shfl_up_sync(0xffffffffu, inc0, o), y1 = __shfl_up_sync(0xffffffffu, inc1, o);
            if (lane >= o) { inc0 += y0; inc1 += y1; }
        }
        const int tot0 = __shfl_sync(0xffffffffu, inc0, 31);
        if (lane < b1) sel_pre[lane] = inc0 - cnt0;
        if (lane + 32 < b1) sel_pre[lane + 32] = tot0 + inc1 - cnt1;
        if (lane == 31) sel_pre[b1] = tot0 + inc1;
    }
    __syncthreads();
    // second level: this CTA's share of the candidate slots
    const int total = sel_pre[b1];
    const int c_begin = s * cap < total ? s * cap : total;
    const int c_end = (s + 1) * cap < total ? (s + 1) * cap : total;
    unsigned long long* out = cand + ((size_t)q * S + s) * cap;
    auto list_of = [&](int slot) {
        int r = 0;
        while (r + 1 < b1 && sel_pre[r + 1] <= slot) ++r;
        return sel_first[r] + (slot - sel_pre[r]);
    };
    for (int c0 = c_begin + warp * TREE_RPW; c0 < c_end; c0 += NW * TREE_RPW) {
        int row[TREE_RPW];
#pragma unroll
        for (int u = 0; u < TREE_RPW; ++u) row[u] = list_of(c0 + u < c_end ? c0 + u : c_end - 1);
        float dot[TREE_RPW];
        warp_score_rows<BF16, false>(qs, C, row, d, metric, lane, dot);
        if (lane == 0) {
#pragma unroll
            for (int u = 0; u < TREE_RPW; ++u) {
                if (c0 + u < c_end) {
                    const float sc = metric == RAGO_L2 ? fmaf(-2.f, dot[u], __ldg(cnorm + row[u])) : -dot[u];
                    out[c0 + u - c_begin] = ((unsigned long long)__float_as_uint(sc) << 32) | (uint32_t)row[u];
                }
            }
        }
    }
    if (tid == 0) cand_cnt[(size_t)q * S + s] = c_end - c_begin;
}

cudaError_t launch_tree_candidates(const IndexImpl* ix, const float* queries, int nq, int S, int cap,
                                   unsigned long long* cand, int32_t* cand_cnt, uint32_t* clear_block, cudaStream_t s) {
    const size_t smem = (size_t)((ix->d + 3) & ~3) * 4 + (size_t)ix->tree_n1 * 8;
    if (smem > 48 * 1024) return cudaErrorInvalidValue;
    if (ix->coarse_bf16)
        launch_overlapped(tree_candidates_kernel<true>, dim3(S, nq), dim3(TREE_THREADS), smem, s, queries, ix->tree_level1,
                          ix->tree_child_offsets, ix->tree_n1, ix->tree_b1, ix->centroids, ix->cnorm, ix->d, ix->metric,
                          cap, cand, cand_cnt, clear_block);
    else
        launch_overlapped(tree_candidates_kernel<false>, dim3(S, nq), dim3(TREE_THREADS), smem, s, queries, ix->tree_level1,
                          ix->tree_child_offsets, ix->tree_n1, ix->tree_b1, ix->centroids, ix->cnorm, ix->d, ix->metric,
                          cap, cand, cand_cnt, clear_block);
    count_launch();
    return cudaGetLastError();
}

// ---- per-query selection of the nprobe best lists ----------------------------------------------
constexpr int SEL_MAX_SPLIT = 512;  // candidate lists per query the kernel can index (one per column range of the GEMM)

// Candidates come either from a score row (scores != null: all nlist lists) or from the candidate
// lists the tensor-core kernel left behind (cand[q][split][cap] raw entries, see cand_key, with counts cand_cnt[q][split]).
// First a cut value is found on the ordered score bits (the range is narrowed by counting items per slice in
// shared memory, then bisected if ties or an odd distribution leave it open; items are held in registers when
// they fit, re-read from memory otherwise) such that between nsel and nsel + slack items lie at or below it;
// only those go to shared memory, are sorted, re-scored exactly and sorted again.
// SEL_THREADS threads per query keep up to SEL_REG item scores each in registers: a big CTA for tiny
// batches (latency), a small one when there are enough queries to fill the GPU.
// FROM_SCORES: the items are a row of the score matrix (else the candidate lists the GEMM left).  The two sources
// are separate instantiations because the kernel body runs once per CTA, largely unrolled: its size is what a
// small batch pays for, in instruction fetches.  For the same reason ALL_REGS (the launcher knows that every item
// fits the registers: a score row of at most SEL_REG x SEL_THREADS lists) leaves out the re-reading variants of
// every phase, and the refinement of an oversized tie group always re-reads its items, as one compact loop.
template <bool BF16, int SEL_THREADS, int SEL_REG, bool FROM_SCORES, bool ALL_REGS>
__global__ void __launch_bounds__(SEL_THREADS) select_probes_kernel(
    const float* __restrict__ Q, const void* __restrict__ C, const float* __restrict__ scores,
    const unsigned long long* __restrict__ cand, const int32_t* __restrict__ cand_cnt, uint32_t cand_sign, int nsplit,
    int cap, int nlist, int d, int metric, int nprobe, int32_t* __restrict__ probe_list,
    float* __restrict__ probe_term, float* __restrict__ probe_bias, const FusedPlan fp) {
    extern __shared__ float fp_smem[];  // fused planning only: the table builders' d + M floats
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ unsigned long long keys2[MAX_K + PROBE_GUARD];
    __shared__ int pre[SEL_MAX_SPLIT + 1];  // candidate path: exclusive prefix of the lists' counts
    __shared__ uint32_t hist[256];           // items per slice of the score range
    __shared__ uint32_t s_mn, s_mx, s_nv;    // CTA-wide minimum, maximum, count of the ordered score bits
    __shared__ uint32_t s_cut_cnt;           // items at or below that cut
    __shared__ uint32_t s_wmin[33];          // the warps' minima; [32]: the cut taken from them
    __shared__ uint32_t s_round[3];          // bisection counts, one word per round in rotation
    __shared__ uint32_t s_bin[3];            // slice holding the cut, items of the range up to and including / before it
    __shared__ int cnt;
    const int q = blockIdx.x, tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    auto sync = [] { __syncthreads(); };
    grid_dependency_wait();
    grid_dependents_may_launch();
    if constexpr (SEL_THREADS == PFX_THREADS) {
        if (fp.enabled && q >= fp.nq) {  // uniform: this CTA builds a part of a lookup table (queries only: no ordering needed)
            const int b = q - fp.nq;
            build_table_part(fp.tables, b / fp.table_parts, b % fp.table_parts, fp.table_parts, fp_smem);
            return;
        }
    }
    int nsel = nprobe + PROBE_GUARD;
    if (nsel > nlist) nsel = nlist;
    if (tid == 0) { cnt = 0; s_mn = 0xFFFFFFFFu; s_mx = 0u; s_nv = 0u; s_cut_cnt = 0u; s_round[0] = s_round[1] = s_round[2] = 0u; }
    for (int i = tid; i < 256; i += SEL_THREADS) hist[i] = 0u;
    const float* srow = FROM_SCORES ? scores + (size_t)q * nlist : nullptr;
    if (!FROM_SCORES) {  // the valid entries of the query's lists, numbered consecutively
        // the counts are fetched side by side (one thread reading them in turn paid a global round trip per list)
        for (int sp = tid; sp < nsplit; sp += SEL_THREADS) pre[sp + 1] = cand_cnt[(size_t)q * nsplit + sp];
        __syncthreads();
        if (tid == 0) {
            int acc = 0;
            for (int sp = 0; sp < nsplit; ++sp) { const int c = pre[sp + 1]; pre[sp] = acc; acc += c; }
            pre[nsplit] = acc;
        }
    }
    __syncthreads();
    const int nitems = FROM_SCORES ? nlist : pre[nsplit];
    // key of item l
    auto item = [&](int l) -> unsigned long long {
        if constexpr (FROM_SCORES) return make_key(srow[l], (uint32_t)l);
        int lo_s = 0, hi_s = nsplit;  // pre[lo_s] <= l < pre[hi_s]
        while (hi_s - lo_s > 1) {
            const int mid_s = (lo_s + hi_s) >> 1;
            if (pre[mid_s] <= l) lo_s = mid_s; else hi_s = mid_s;
        }
        return cand_key(cand[((size_t)q * nsplit + lo_s) * cap + (l - pre[lo_s])], cand_sign);
    };
    const bool in_regs = ALL_REGS || nitems <= SEL_REG * SEL_THREADS;
    uint32_t mine[SEL_REG];  // ordered score bits; 0xFFFFFFFF marks an empty slot
    uint32_t mn = 0xFFFFFFFFu, mx = 0u, nvalid = 0;
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < SEL_REG; ++j) {
            const int l = tid + j * SEL_THREADS;
            const unsigned long long k = l < nitems ? item(l) : KEY_MAX;
            mine[j] = k == KEY_MAX ? 0xFFFFFFFFu : (uint32_t)(k >> 32);
            if (k != KEY_MAX) {
                mn = mine[j] < mn ? mine[j] : mn; mx = mine[j] > mx ? mine[j] : mx; ++nvalid;
            }
        }
    } else {
        for (int l = tid; l < nitems; l += SEL_THREADS) {
            const unsigned long long k = item(l);
            if (k != KEY_MAX) {
                const uint32_t o = (uint32_t)(k >> 32);
                mn = o < mn ? o : mn; mx = o > mx ? o : mx; ++nvalid;
            }
        }
    }
    // CTA-wide minimum, maximum and count
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    nvalid = __reduce_add_sync(0xffffffffu, nvalid);
    if (lane == 0) { atomicMin(&s_mn, mn); atomicMax(&s_mx, mx); atomicAdd(&s_nv, nvalid); s_wmin[warp] = mn; }
    __syncthreads();
    // Few lists wanted (nsel <= 32) out of many: the nsel-th smallest of the warps' minima has at least nsel items
    // at or below it, one per warp, and on scores in no particular order only a few dozen in all.  It replaces the
    // slice counts and the bisection below as the cut, for one small sort by one warp.
    uint32_t warp_cut = 0xFFFFFFFFu;
    if (SEL_THREADS == 1024 && in_regs && nsel <= 32) {  // uniform
        if (warp == 0) {
            const uint32_t sorted = warp_sort_u32(s_wmin[lane], lane);
            if (lane == nsel - 1) s_wmin[32] = sorted;
        }
        __syncthreads();
        warp_cut = s_wmin[32];  // 0xFFFFFFFF: fewer than nsel warps hold an item
    }
    mn = s_mn; mx = s_mx; nvalid = s_nv;
    if ((int)nvalid < nsel) nsel = (int)nvalid;  // cannot happen for a well-formed candidate set; stay safe
    int slack = nsel / 4 > 8 ? nsel / 4 : 8;
    if (nsel + slack > TOPK_CAP) slack = TOPK_CAP - nsel;
    // Narrow the range first: 256 equal slices of (lo, hi] (in ordered score bits), one shared-memory count each;
    // the slice that holds the nsel-th smallest item becomes the new range.  Two passes usually leave at most
    // nsel + slack items at or below hi; ties and odd distributions are finished by the bisection below.
    long long lo = (long long)mn - 1, hi = mx;  // invariant: #(score <= lo) < nsel <= #(score <= hi)
    uint32_t c_hi = nvalid, below = 0;          // below = #(score <= lo)
    if (warp_cut != 0xFFFFFFFFu) {  // uniform; in_regs holds
        uint32_t c = 0;
#pragma unroll
        for (int j = 0; j < SEL_REG; ++j) c += mine[j] <= warp_cut ? 1u : 0u;  // warp_cut < the empty-slot pattern
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0 && c) atomicAdd(&s_cut_cnt, c);
        __syncthreads();
        hi = warp_cut;
        c_hi = s_cut_cnt;  // >= nsel
        if (nsel + slack < WARP_SORT_MAX) slack = WARP_SORT_MAX - nsel;  // what one warp sorts is as good as fewer
    }
    for (int pass = 0; pass < 3 && hi - lo > 1 && c_hi > (uint32_t)(nsel + slack); ++pass) {  // uniform
        const uint32_t first = (uint32_t)(lo + 1), range = (uint32_t)(hi - lo - 1);
        const int shift = range < 256u ? 0 : 24 - __clz(range);  // (range >> shift) < 256
        if (in_regs) {
#pragma unroll
            for (int j = 0; j < SEL_REG; ++j)  // hi <= mx < the empty-slot pattern
                if (mine[j] >= first && mine[j] <= (uint32_t)hi) atomicAdd(&hist[(mine[j] - first) >> shift], 1u);
        } else {
            for (int l = tid; l < nitems; l += SEL_THREADS) {
                const unsigned long long k = item(l);
                const uint32_t o = (uint32_t)(k >> 32);
                if (k != KEY_MAX && o >= first && o <= (uint32_t)hi) atomicAdd(&hist[(o - first) >> shift], 1u);
            }
        }
        __syncthreads();
        if (warp == 0) {  // lane i owns slices 8 i .. 8 i + 7
            const uint32_t want = (uint32_t)nsel - below;  // rank of the cut inside the range, >= 1
            uint32_t h[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { h[j] = hist[lane * 8 + j]; tot += h[j]; }
            uint32_t before = tot;  // inclusive scan over the lanes, then made exclusive
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, before, o);
                if (lane >= o) before += v;
            }
            before -= tot;
            if (before < want && before + tot >= want) {  // exactly one lane
                uint32_t c = before, prev = before;
                int bsel = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (c < want) { bsel = j; prev = c; c += h[j]; }
                }
                s_bin[0] = (uint32_t)(lane * 8 + bsel); s_bin[1] = c; s_bin[2] = prev;
            }
        }
        __syncthreads();
        const uint32_t bsel = s_bin[0];
        const long long top = (long long)first + (((long long)bsel + 1) << shift) - 1;
        c_hi = below + s_bin[1];
        below += s_bin[2];
        hi = top < hi ? top : hi;
        lo = (long long)first + ((long long)bsel << shift) - 1;
        for (int i = tid; i < 256; i += SEL_THREADS) hist[i] = 0u;
        __syncthreads();
    }
    // bisection inside the slice: #(score <= lo) < nsel <= #(score <= hi)
    int round = 0;
    while (hi - lo > 1 && c_hi > (uint32_t)(nsel + slack)) {  // uniform
        const uint32_t mid = (uint32_t)(lo + (hi - lo) / 2);
        uint32_t c = 0;
        if (in_regs) {
#pragma unroll
            for (int j = 0; j < SEL_REG; ++j) c += mine[j] <= mid ? 1u : 0u;  // mid <= mx < the empty-slot pattern
        } else {
            for (int l = tid; l < nitems; l += SEL_THREADS) {
                const unsigned long long k = item(l);
                c += (k != KEY_MAX && (uint32_t)(k >> 32) <= mid) ? 1u : 0u;
            }
        }
        c = __reduce_add_sync(0xffffffffu, c);
        const int slot = round % 3;
        if (lane == 0 && c) atomicAdd(&s_round[slot], c);
        if (tid == 0) s_round[(slot + 1) % 3] = 0u;  // next round's word; its last readers passed two barriers ago
        __syncthreads();
        c = s_round[slot];
        if (c < (uint32_t)nsel) lo = mid; else { hi = mid; c_hi = c; }
        ++round;
    }
    const uint32_t T = (uint32_t)hi;
    // A tie group at the cut that would not fit the buffer (thousands of lists with bit-identical scores): which
    // of the tied items are kept must not depend on the order in which warps reach the buffer, and no item
    // below the cut may lose its place to a tied one.  The cut is then refined on the payload (list number) among
    // the items that score exactly T, by the same counting bisection: items below T are all kept, tied ones up to
    // payload P, so that at most nsel + slack are collected and they include the nsel smallest keys.
    uint32_t P = 0xFFFFFFFFu;
    if (c_hi > (uint32_t)TOPK_CAP) {  // uniform
        auto count_cta = [&](uint32_t c) -> uint32_t {  // sum of c over the CTA, same value in every thread
            c = __reduce_add_sync(0xffffffffu, c);
            const int slot = round % 3;
            if (lane == 0 && c) atomicAdd(&s_round[slot], c);
            if (tid == 0) s_round[(slot + 1) % 3] = 0u;
            __syncthreads();
            ++round;
            return s_round[slot];
        };
        uint32_t less = 0;
        for (int l = tid; l < nitems; l += SEL_THREADS) {
            const unsigned long long k = item(l);
            less += (k != KEY_MAX && (uint32_t)(k >> 32) < T) ? 1u : 0u;
        }
        less = count_cta(less);
        const uint32_t need = (uint32_t)nsel - less;  // >= 1: fewer than nsel items lie below T
        long long plo = -1, phi = 0xFFFFFFFFll;       // #(tied, payload <= plo) < need <= #(tied, payload <= phi)
        uint32_t pc_hi = c_hi - less;
        while (phi - plo > 1 && pc_hi > need + (uint32_t)slack) {  // uniform
            const uint32_t mid = (uint32_t)(plo + (phi - plo) / 2);
            uint32_t c = 0;
            for (int l = tid; l < nitems; l += SEL_THREADS) {
                const unsigned long long k = item(l);
                if (k != KEY_MAX && (uint32_t)(k >> 32) == T && (uint32_t)k <= mid) ++c;
            }
            c = count_cta(c);
            if (c < need) plo = mid; else { phi = mid; pc_hi = c; }
        }
        P = (uint32_t)phi;
    }
    // collect the items below the cut, and those at the cut up to payload P
    if (in_regs) {
        bool any = false;  // most warps hold nothing at or below the cut: one vote instead of SEL_REG
#pragma unroll
        for (int j = 0; j < SEL_REG; ++j) any = any || (mine[j] != 0xFFFFFFFFu && mine[j] <= T);
        if (__any_sync(0xffffffffu, any)) {
#pragma unroll
        for (int j = 0; j < SEL_REG; ++j) {
            bool take = mine[j] != 0xFFFFFFFFu && mine[j] <= T;
            unsigned long long key = KEY_MAX;
            if (FROM_SCORES) key = ((unsigned long long)mine[j] << 32) | (uint32_t)(tid + j * SEL_THREADS);
            else if (take) key = item(tid + j * SEL_THREADS);
            if (take && mine[j] == T && (uint32_t)key > P) take = false;
            warp_push(keys, &cnt, take, key);
        }
        }
    } else {
        for (int l0 = 0; l0 < nitems; l0 += SEL_THREADS) {
            const int l = l0 + tid;
            const unsigned long long k = l < nitems ? item(l) : KEY_MAX;
            const uint32_t o = (uint32_t)(k >> 32);
            warp_push(keys, &cnt, k != KEY_MAX && (o < T || (o == T && (uint32_t)k <= P)), k);
        }
    }
    __syncthreads();
    const int kept = block_select_short(keys, &cnt, nsel, tid, SEL_THREADS, sync);
    // exact re-score of the survivors, one warp per candidate
    const float* qrow = Q + (size_t)q * d;
    for (int i = warp; i < kept; i += SEL_THREADS / 32) {
        const uint32_t l = (uint32_t)(keys[i] & 0xFFFFFFFFull);
        float acc = 0.f;
        for (int j = lane * 4; j < d; j += 128) {  // d is a multiple of 4: 16-byte (fp32) / 8-byte (bf16) loads
            float4 qv = *reinterpret_cast<const float4*>(qrow + j);
            float4 cv;
            if (BF16) {
                qv.x = round_bf16(qv.x); qv.y = round_bf16(qv.y); qv.z = round_bf16(qv.z); qv.w = round_bf16(qv.w);
                const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(C) + (size_t)l * d + j);
                cv.x = __uint_as_float(raw.x << 16); cv.y = __uint_as_float(raw.x & 0xFFFF0000u);
                cv.z = __uint_as_float(raw.y << 16); cv.w = __uint_as_float(raw.y & 0xFFFF0000u);
            } else {
                cv = *reinterpret_cast<const float4*>(static_cast<const float*>(C) + (size_t)l * d + j);
            }
            if (metric == RAGO_L2) {
                const float t0 = qv.x - cv.x, t1 = qv.y - cv.y, t2 = qv.z - cv.z, t3 = qv.w - cv.w;
                acc = fmaf(t0, t0, fmaf(t1, t1, fmaf(t2, t2, fmaf(t3, t3, acc))));
            } else {
                acc = fmaf(qv.x, cv.x, fmaf(qv.y, cv.y, fmaf(qv.z, cv.z, fmaf(qv.w, cv.w, acc))));
            }
        }
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) keys2[i] = make_key(metric == RAGO_L2 ? acc : -acc, l);
    }
    __syncthreads();
    for (int i = tid; i < kept; i += SEL_THREADS) keys[i] = keys2[i];
    if (tid == 0) cnt = kept;
    __syncthreads();
    block_select_short(keys, &cnt, kept, tid, SEL_THREADS, sync);  // the usual case: a few survivors, ranked
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
    // Fused planning.  A single query plans from what it still holds in shared memory: no ticket, no fence, no
    // re-read.  With more queries the CTA that finishes its query last (a ticket, nothing waits) plans for the batch.
    if constexpr (SEL_THREADS == PFX_THREADS) {
        if (fp.enabled) {  // uniform
            __shared__ int s_last;
            __shared__ long long plan_sums[32];
            if (fp.nq == 1) {
                long long v = 0;  // tiles of pair tid (nprobe <= MAX_K = SEL_THREADS)
                if (tid < nprobe) {
                    const uint32_t l = (uint32_t)(keys[tid] & 0xFFFFFFFFull);
                    v = (fp.offsets[l + 1] - fp.offsets[l] + fp.tile_vecs - 1) / fp.tile_vecs;
                }
                fp.qthresh[0] = KEY_MAX;  // every thread the same value; the stores leave with the loads above
                for (int i = tid; i < fp.nslots; i += SEL_THREADS) fp.slot_cnt[i] = 0;
                long long incl = v;
                for (int o = 1; o < 32; o <<= 1) {
                    const long long y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += y;
                }
                if (lane == 31) plan_sums[warp] = incl;
                __syncthreads();
                long long before = incl - v;
                for (int w = 0; w < warp; ++w) before += plan_sums[w];  // few warps hold pairs: short for small nprobe
                if (tid < nprobe) fp.prefix[tid] = before;
                if (tid == nprobe - 1) fp.prefix[nprobe] = before + v;
            } else {
                __syncthreads();  // this query's probe lists are written ...
                if (tid == 0) {
                    __threadfence();  // ... and ordered before the ticket (the barrier makes the fence cover them all)
                    s_last = atomicAdd(fp.ticket, 1u) == (uint32_t)(fp.nq - 1) ? 1 : 0;
                    __threadfence();
                }
                __syncthreads();
                if (s_last) {
                    plan_pairs_cta(probe_list, fp.offsets, fp.nq * nprobe, fp.tile_vecs, fp.prefix, fp.qthresh, fp.nq,
                                   fp.slot_cnt, fp.nslots, plan_sums);
                    if (tid == 0) *fp.ticket = 0u;
                }
            }
        }
    }
}

template <bool BF16, int THREADS, int REG>
static void launch_select_source(const IndexImpl* ix, const float* queries, const float* scores,
                                 const unsigned long long* cand, const int32_t* cand_cnt, uint32_t cand_sign, int nsplit, int cap, int nq,
                                 int nprobe, int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan& fp, cudaStream_t s) {
    const dim3 grid(fp.enabled ? nq * (1 + fp.table_parts) : nq);
    const size_t smem = fp.enabled ? (size_t)(ix->d + ix->M) * 4 : 0;
    if (scores && ix->nlist <= THREADS * REG)
        launch_overlapped(select_probes_kernel<BF16, THREADS, REG, true, true>, grid, dim3(THREADS), smem, s,
            queries, ix->centroids, scores, cand, cand_cnt, cand_sign, nsplit, cap, ix->nlist, ix->d, ix->metric, nprobe, probe_list,
            probe_term, probe_bias, fp);
    else if (scores)
        launch_overlapped(select_probes_kernel<BF16, THREADS, REG, true, false>, grid, dim3(THREADS), smem, s,
            queries, ix->centroids, scores, cand, cand_cnt, cand_sign, nsplit, cap, ix->nlist, ix->d, ix->metric, nprobe, probe_list,
            probe_term, probe_bias, fp);
    else
        launch_overlapped(select_probes_kernel<BF16, THREADS, REG, false, false>, grid, dim3(THREADS), smem, s,
            queries, ix->centroids, scores, cand, cand_cnt, cand_sign, nsplit, cap, ix->nlist, ix->d, ix->metric, nprobe, probe_list,
            probe_term, probe_bias, fp);
}
template <int THREADS, int REG>
static void launch_select_shape(const IndexImpl* ix, const float* queries, const float* scores,
                                const unsigned long long* cand, const int32_t* cand_cnt, uint32_t cand_sign, int nsplit, int cap, int nq,
                                int nprobe, int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan& fp,
                                cudaStream_t s) {
    if (ix->coarse_bf16)
        launch_select_source<true, THREADS, REG>(ix, queries, scores, cand, cand_cnt, cand_sign, nsplit, cap, nq, nprobe, probe_list,
                                                 probe_term, probe_bias, fp, s);
    else
        launch_select_source<false, THREADS, REG>(ix, queries, scores, cand, cand_cnt, cand_sign, nsplit, cap, nq, nprobe, probe_list,
                                                  probe_term, probe_bias, fp, s);
}
// fp (may be null): the kernel also plans the scan of the batch and builds its lookup tables (batches of at most 64
// queries, which run the 1024-thread shape).
static cudaError_t launch_select_any(const IndexImpl* ix, const float* queries, const float* scores,
                                     const unsigned long long* cand, const int32_t* cand_cnt, uint32_t cand_sign, int nsplit, int cap, int nq,
                                     int nprobe, int32_t* probe_list, float* probe_term, float* probe_bias,
                                     const FusedPlan* fp, cudaStream_t s) {
    if (nsplit > SEL_MAX_SPLIT) return cudaErrorInvalidValue;
    FusedPlan off;
    std::memset(&off, 0, sizeof(off));
    if (fp && fp->enabled && nq > 64) return cudaErrorInvalidValue;
    if (nq <= 64)
        launch_select_shape<1024, 16>(ix, queries, scores, cand, cand_cnt, cand_sign, nsplit, cap, nq, nprobe, probe_list, probe_term,
                                      probe_bias, fp ? *fp : off, s);
    else
        launch_select_shape<256, 20>(ix, queries, scores, cand, cand_cnt, cand_sign, nsplit, cap, nq, nprobe, probe_list, probe_term,
                                     probe_bias, off, s);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_select_probes(const IndexImpl* ix, const float* queries, const float* scores, int nq, int nprobe,
                                 int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan* fp,
                                 cudaStream_t s) {
    return launch_select_any(ix, queries, scores, nullptr, nullptr, 0u, 0, 0, nq, nprobe, probe_list, probe_term,
                             probe_bias, fp, s);
}

cudaError_t launch_select_probes_cand(const IndexImpl* ix, const float* queries, const unsigned long long* cand,
                                      const int32_t* cand_cnt, uint32_t cand_sign, int nsplit, int cap, int nq, int nprobe,
                                      int32_t* probe_list, float* probe_term, float* probe_bias, const FusedPlan* fp,
                                      cudaStream_t s) {
    return launch_select_any(ix, queries, nullptr, cand, cand_cnt, cand_sign, nsplit, cap, nq, nprobe, probe_list, probe_term,
                             probe_bias, fp, s);
}

}  // namespace rago
