// Exact flat search: score = <q, y_i> over bf16 inputs, fp32 accumulation, k largest per query.
//
// Main path (k <= 960): the tensor-core kernel of gemm_select.cu with rows = queries and columns =
// database rows; every CTA streams its own range of the database once (both 128-query row tiles are
// multiplied against a database tile while it is hot) and keeps each query's k best of that range;
// flat_merge_kernel merges the ranges.  No score is ever written to memory.
// Fallback (larger k): the database is processed in panels of PANEL rows on the fp32 pipes: scores of
// a panel go to scratch, each (query, 64K-row chunk) keeps its k best, and the same merge finishes.
#include "topk.cuh"

namespace rago {

constexpr int FBM = 64, FBN = 64, FBK = 16;
constexpr int FLAT_CHUNK = 1 << 16;   // rows per selection chunk
constexpr int FLAT_PANEL = 1 << 20;   // rows scored per pass

__global__ void __launch_bounds__(256) flat_scores_kernel(const __nv_bfloat16* __restrict__ Q,
                                                          const __nv_bfloat16* __restrict__ Y, int nq,
                                                          long long row_begin, int nrows, int d,
                                                          float* __restrict__ scores) {
    __shared__ __align__(16) float As[FBK][FBM + 4];
    __shared__ __align__(16) float Bs[FBK][FBN + 4];
    const int tid = threadIdx.x;
    const int row0 = blockIdx.y * FBM, col0 = blockIdx.x * FBN;
    const int lr = tid >> 2, lk = (tid & 3) * 4;
    const int ty = tid >> 4, tx = tid & 15;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < d; k0 += FBK) {
        float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
        if (row0 + lr < nq) {
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = __bfloat162float(Q[(size_t)(row0 + lr) * d + k0 + lk + i]);
        }
        if (col0 + lr < nrows) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                b[i] = __bfloat162float(Y[(size_t)(row_begin + col0 + lr) * d + k0 + lk + i]);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk + i][lr] = a[i];
            Bs[lk + i][lr] = b[i];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < FBK; ++kk) {
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
            if (c < nrows) scores[(size_t)r * FLAT_PANEL + c] = -acc[i][j];  // smaller = better
        }
    }
}

constexpr int FSEL_THREADS = 256;

// grid (chunks in panel, nq): k best of one chunk of one query -> slot (q, global chunk).
__global__ void __launch_bounds__(FSEL_THREADS) flat_select_kernel(const float* __restrict__ scores,
                                                                   long long row_begin, int nrows, int k,
                                                                   int chunk_begin, int nchunks_total,
                                                                   int32_t* __restrict__ slot_cnt,
                                                                   unsigned long long* __restrict__ slot_keys) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    const int tid = threadIdx.x, q = blockIdx.y, ch = blockIdx.x;
    auto sync = [] { __syncthreads(); };
    if (tid == 0) cnt = 0;
    __syncthreads();
    const int c0 = ch * FLAT_CHUNK;
    int c1 = c0 + FLAT_CHUNK;
    if (c1 > nrows) c1 = nrows;
    const float* srow = scores + (size_t)q * FLAT_PANEL;
    unsigned long long tau = KEY_MAX;
    int ub = 0;
    for (int i0 = c0; i0 < c1; i0 += FSEL_THREADS) {
        const int i = i0 + tid;
        unsigned long long key = KEY_MAX;
        if (i < c1) key = make_key(srow[i], (uint32_t)(row_begin + i));
        warp_push(keys, &cnt, i < c1 && key < tau, key);
        ub += FSEL_THREADS;
        if (ub + FSEL_THREADS > TOPK_CAP) {
            __syncthreads();
            const int kept = block_select(keys, &cnt, k, tid, FSEL_THREADS, sync);
            if (kept == k) tau = keys[k - 1];
            ub = kept;
            __syncthreads();
        }
    }
    __syncthreads();
    const int kept = block_select(keys, &cnt, k, tid, FSEL_THREADS, sync);
    const size_t slot = (size_t)q * nchunks_total + chunk_begin + ch;
    for (int i = tid; i < kept; i += FSEL_THREADS) slot_keys[slot * k + i] = keys[i];
    if (tid == 0) slot_cnt[slot] = kept;
}

// slot (q, ch) holds slot_cnt keys at slot_keys[(q * nchunks + ch) * stride ...]; with `raw` they are the raw
// candidate entries of the tensor-core kernel (cand_key turns them into keys).
__global__ void __launch_bounds__(FSEL_THREADS) flat_merge_kernel(int nchunks, int k, int stride, int raw, uint32_t raw_sign,
                                                                  const int32_t* __restrict__ slot_cnt,
                                                                  const unsigned long long* __restrict__ slot_keys,
                                                                  int64_t* __restrict__ out_ids,
                                                                  float* __restrict__ out_scores) {
    __shared__ unsigned long long keys[TOPK_CAP];
    __shared__ int cnt;
    const int tid = threadIdx.x, q = blockIdx.x;
    auto sync = [] { __syncthreads(); };
    if (tid == 0) cnt = 0;
    __syncthreads();
    unsigned long long tau = KEY_MAX;
    for (int ch = 0; ch < nchunks; ++ch) {
        const size_t slot = (size_t)q * nchunks + ch;
        const int c = slot_cnt[slot];
        if (cnt + c > TOPK_CAP) {
            const int kept = block_select(keys, &cnt, k, tid, FSEL_THREADS, sync);
            if (kept == k) tau = keys[k - 1];
            __syncthreads();
        }
        for (int i0 = 0; i0 < c; i0 += FSEL_THREADS) {
            const int i = i0 + tid;
            unsigned long long key = KEY_MAX;
            if (i < c) key = raw ? cand_key(slot_keys[slot * stride + i], raw_sign) : slot_keys[slot * stride + i];
            warp_push(keys, &cnt, i < c && key < tau, key);
        }
        __syncthreads();
    }
    const int kept = block_select(keys, &cnt, k, tid, FSEL_THREADS, sync);
    for (int i = tid; i < k; i += FSEL_THREADS) {
        int64_t id = -1;
        float sc = __int_as_float(0xff800000);
        if (i < kept) {
            id = (int64_t)(uint32_t)(keys[i] & 0xFFFFFFFFull);
            sc = -orderable_f32((uint32_t)(keys[i] >> 32));
        }
        out_ids[(size_t)q * k + i] = id;
        out_scores[(size_t)q * k + i] = sc;
    }
}

static int sm_count() {
    static int sms = 0;
    if (!sms) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            sms = n;
        else {
            cudaGetLastError();
            return 148;  // no device yet (size queries on a host without one): the B200 count
        }
    }
    return sms;
}

static bool flat_on_tensor_cores(int d, int k) { return gemm_cand_cap(k) != 0 && d % 8 == 0; }

// Pilot pass of the flat search: worth it for large databases; the sample must hold 4 k rows.
static int flat_pilot_cols(int64_t N, int k) {
    if (N < (1 << 18)) return 0;
    const int64_t np = N / gemm_pilot_stride(N);
    return np >= 4LL * k ? (int)np : 0;
}

// Workspace, tensor-core path: [err 256 B][cand nq*nlists*cap u64][cand_cnt nq*nlists i32][pilot scores nq*np f32][row_tau nq f32]
//            (nlists = column ranges of the grid x GEMM_COL_HALVES candidate lists per query)
//            fallback:         [err 256 B][scores nq*PANEL f32][slot_cnt nq*nchunks i32][slot_keys nq*nchunks*k u64]
size_t flat_workspace_bytes(int64_t N, int d, int nq, int k) {
    if (flat_on_tensor_cores(d, k)) {
        int mg, nsplit, mgroups;
        gemm_grid(nq > 0 ? nq : 1, N > 0 ? N : 1, d, sm_count(), &mg, &nsplit, &mgroups);
        const size_t nlists = (size_t)nsplit * GEMM_COL_HALVES;
        return 256 + align_up((size_t)nq * nlists * gemm_cand_cap(k) * 8, 256) + align_up((size_t)nq * nlists * 4, 256) +
               align_up((size_t)nq * flat_pilot_cols(N, k) * 4, 256) + align_up((size_t)nq * 4, 256);
    }
    const size_t nchunks = (size_t)((N + FLAT_CHUNK - 1) / FLAT_CHUNK);
    size_t b = 256;
    b += align_up((size_t)nq * FLAT_PANEL * 4, 256);
    b += align_up((size_t)nq * (nchunks ? nchunks : 1) * 4, 256);
    b += align_up((size_t)nq * (nchunks ? nchunks : 1) * k * 8, 256);
    return b;
}

cudaError_t launch_flat_search(const void* db, int64_t N, int d, const void* queries, int nq, int k, int64_t* out_ids,
                               float* out_scores, void* workspace, cudaStream_t s) {
    if (flat_on_tensor_cores(d, k) && N > 0) {
        cudaError_t e = gemm_select_init();
        if (e != cudaSuccess) return e;
        int mg, nsplit, mgroups;
        gemm_grid(nq, N, d, sm_count(), &mg, &nsplit, &mgroups);
        const int cap = gemm_cand_cap(k);
        const int nlists = nsplit * GEMM_COL_HALVES;
        uint8_t* w = static_cast<uint8_t*>(workspace) + 256;
        unsigned long long* cand = reinterpret_cast<unsigned long long*>(w);
        w += align_up((size_t)nq * nlists * cap * 8, 256);
        int32_t* cand_cnt = reinterpret_cast<int32_t*>(w);
        w += align_up((size_t)nq * nlists * 4, 256);
        const int np = flat_pilot_cols(N, k);
        float* pilot_scores = reinterpret_cast<float*>(w);
        w += align_up((size_t)nq * np * 4, 256);
        float* row_tau = reinterpret_cast<float*>(w);
        alignas(64) unsigned char tmap_a[128], tmap_b[128], tmap_bh[128];
        e = make_tmap_bf16(tmap_a, queries, (uint64_t)nq, (uint64_t)d, 128);
        if (e == cudaSuccess) e = make_tmap_bf16(tmap_b, db, (uint64_t)N, (uint64_t)d, 256);
        if (e == cudaSuccess) e = make_tmap_bf16(tmap_bh, db, (uint64_t)N, (uint64_t)d, 128);
        if (e != cudaSuccess) return e;
        GemmLaunch G;
        G.tmap_a = tmap_a; G.tmap_b = tmap_b; G.tmap_b_half = tmap_bh;
        G.nrows = nq; G.ncols = N; G.d = d;
        G.a_part_rows = nq; G.b_part_rows = N;
        G.nterms = 1;
        for (int t = 0; t < 6; ++t) G.term_a[t] = G.term_b[t] = 0;
        G.mg = mg; G.nsplit = nsplit;
        G.alpha = -1.f;  // smaller = better
        G.colterm = nullptr; G.colterm_stride = 1;
        G.row_tau = nullptr;
        G.mode = 0; G.nsel = k < N ? k : (int)N; G.cap = cap;
        G.cand = cand; G.cand_cnt = cand_cnt; G.scores = nullptr;
        G.err = static_cast<uint32_t*>(workspace);
        if (np) {
            // pilot pass over every stride-th row: each query starts from the k-th best score of that sample
            alignas(64) unsigned char tmap_p[128], tmap_ph[128];
            const int ps = gemm_pilot_stride(N);
            e = make_tmap_bf16(tmap_p, db, (uint64_t)np, (uint64_t)d, 256, (uint64_t)ps * d);
            if (e == cudaSuccess) e = make_tmap_bf16(tmap_ph, db, (uint64_t)np, (uint64_t)d, 128, (uint64_t)ps * d);
            if (e != cudaSuccess) return e;
            GemmLaunch P = G;
            int pg = 1;
            P.tmap_b = tmap_p; P.tmap_b_half = tmap_ph;
            P.ncols = np; P.b_part_rows = np;
            gemm_grid(nq, np, d, sm_count(), &P.mg, &P.nsplit, &pg);
            P.mode = 1; P.scores = pilot_scores;
            e = launch_gemm_select(P, s);
            if (e == cudaSuccess) e = launch_row_tau(pilot_scores, nq, np, G.nsel, row_tau, s);
            if (e != cudaSuccess) return e;
            G.row_tau = row_tau;
        }
        e = launch_gemm_select(G, s);
        if (e != cudaSuccess) return e;
        flat_merge_kernel<<<nq, FSEL_THREADS, 0, s>>>(nlists, k, cap, 1, gemm_cand_sign(G.alpha, G.colterm), cand_cnt, cand,
                                                      out_ids, out_scores);
        count_launch();
        return cudaGetLastError();
    }
    const int nchunks = (int)((N + FLAT_CHUNK - 1) / FLAT_CHUNK);
    uint8_t* w = static_cast<uint8_t*>(workspace) + 256;
    float* scores = reinterpret_cast<float*>(w);
    w += align_up((size_t)nq * FLAT_PANEL * 4, 256);
    int32_t* slot_cnt = reinterpret_cast<int32_t*>(w);
    w += align_up((size_t)nq * (nchunks ? nchunks : 1) * 4, 256);
    unsigned long long* slot_keys = reinterpret_cast<unsigned long long*>(w);
    for (int64_t r0 = 0; r0 < N; r0 += FLAT_PANEL) {
        const int nrows = (int)((N - r0) < FLAT_PANEL ? (N - r0) : FLAT_PANEL);
        dim3 g((nrows + FBN - 1) / FBN, (nq + FBM - 1) / FBM);
        flat_scores_kernel<<<g, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(queries),
                                             static_cast<const __nv_bfloat16*>(db), nq, r0, nrows, d, scores);
        dim3 gs((nrows + FLAT_CHUNK - 1) / FLAT_CHUNK, nq);
        flat_select_kernel<<<gs, FSEL_THREADS, 0, s>>>(scores, r0, nrows, k, (int)(r0 / FLAT_CHUNK), nchunks,
                                                       slot_cnt, slot_keys);
        count_launch(2);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    flat_merge_kernel<<<nq, FSEL_THREADS, 0, s>>>(nchunks, k, k, 0, 0u, slot_cnt, slot_keys, out_ids, out_scores);
    count_launch();
    return cudaGetLastError();
}

}  // namespace rago
