// C ABI of the retrieval library: argument checks, workspace layout, stage launches.
#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "plan.cuh"

namespace rago {

static std::atomic<long long> g_launches{0};
static thread_local char g_err[512] = "";

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

static rago_status fail(rago_status st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}

static rago_status cuda_fail(cudaError_t e, const char* what) {
    return fail(RAGO_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Workspace carving.  Every region starts on a 256-byte boundary; the first 256 bytes hold the
// device error word.
struct Layout {
    size_t err, probe_list, probe_term, probe_bias, scores, pair_tiles, work_prefix, qthresh, slot_cnt, slot_keys, total;
    size_t qparts, cand, cand_cnt;  // tensor-core coarse step: query parts, candidate lists and their counts
    size_t pilot_scores, row_tau;   // pilot pass: scores of the sampled lists, per-query starting thresholds
    size_t lut_img, lut_inv, lut_scale;        // small batches: lookup tables built ahead of the scan, and their scales
    int prebuilt;
    int pilot_cols;                 // 0: no pilot pass
    size_t nslots;
    int tc, tc_mode, tc_cap, tc_mg, tc_nsplit;  // coarse plan for this (nq, nprobe)
    int tree_S, tree_cap;           // two-level coarse quantiser: CTAs per query and candidate slots per CTA (0: not used)
};

// Which coarse kernel a batch takes.  The tensor-core kernel pays off once a batch fills a good part of
// a 128-row tile; tiny batches (the latency-bound iterative-retrieval shape) stay on the fp32 pipes.
constexpr int TC_MIN_NQ = 17;
static bool use_tensor_cores(const IndexImpl* ix, int nq) {
    if (!ix->tc_ok || ix->coarse_mode == 1) return false;
    return ix->coarse_mode == 2 || nq >= TC_MIN_NQ;
}

static Layout make_layout(const IndexImpl* ix, int nq, int nprobe, int k) {
    Layout L;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        const size_t at = o;
        o += align_up(bytes ? bytes : 1, 256);
        return at;
    };
    const size_t npairs = (size_t)nq * nprobe;
    L.nslots = (size_t)nq + (size_t)ix->plan.ctas;  // one slot per (CTA, query) incidence
    L.err = take(256);
    L.probe_list = take(npairs * 4);
    L.probe_term = take(npairs * 4);
    L.probe_bias = take(npairs * 4);
    L.tree_S = L.tree_cap = 0;
    if (ix->tree_n1) {  // a few CTAs per query when the batch alone cannot fill the GPU
        int S = (ix->num_sms + nq - 1) / (nq > 0 ? nq : 1);  // every CTA of a query repeats the first level: not too many
        S = S < 1 ? 1 : (S > 32 ? 32 : S);
        L.tree_S = S;
        L.tree_cap = (ix->tree_max_cand + S - 1) / S;
    }
    L.tc = !ix->tree_n1 && use_tensor_cores(ix, nq) ? 1 : 0;
    L.tc_mode = 1; L.tc_cap = 0; L.tc_mg = 1; L.tc_nsplit = 1;
    L.qparts = L.cand = L.cand_cnt = L.pilot_scores = L.row_tau = 0;
    L.pilot_cols = 0;
    if (L.tc) {
        int nsel = nprobe + PROBE_GUARD;
        if (nsel > ix->nlist) nsel = ix->nlist;
        int mgroups = 1;
        gemm_grid(nq, ix->nlist, ix->d * ix->cparts_n, ix->num_sms, &L.tc_mg, &L.tc_nsplit, &mgroups);
        L.tc_cap = gemm_cand_cap(nsel);
        L.tc_mode = L.tc_cap ? 0 : 1;
        L.qparts = take((size_t)ix->cparts_n * nq * ix->d * 2);
        if (L.tc_mode == 0) {
            L.cand = take((size_t)nq * L.tc_nsplit * GEMM_COL_HALVES * L.tc_cap * 8);
            L.cand_cnt = take((size_t)nq * L.tc_nsplit * GEMM_COL_HALVES * 4);
            // a pilot pass pays off when a CTA sees many column tiles per row and the sample can hold nsel values
            const int np = ix->pilot_stride ? ix->nlist / ix->pilot_stride : 0;
            if (np >= 4 * nsel && ix->nlist >= 8192) {
                L.pilot_cols = np;
                L.pilot_scores = take((size_t)nq * np * 4);
                L.row_tau = take((size_t)nq * 4);
            }
        }
    }
    if (L.tree_S) {
        L.cand = take((size_t)nq * L.tree_S * L.tree_cap * 8);
        L.cand_cnt = take((size_t)nq * L.tree_S * 4);
    }
    L.scores = take(!L.tree_S && (!L.tc || L.tc_mode == 1) ? (size_t)nq * ix->nlist * 4 : 0);
    L.pair_tiles = take(npairs * 4);
    L.work_prefix = take((npairs + 1) * 8);
    L.qthresh = take((size_t)nq * 8);
    L.slot_cnt = take(L.nslots * 4);
    L.slot_keys = take(L.nslots * (size_t)k * 8);
    L.prebuilt = nq <= PREBUILT_MAX_NQ ? 1 : 0;
    // reserved for larger batches too, so that a workspace sized for nq queries also serves fewer
    const size_t nlut = nq < PREBUILT_MAX_NQ ? nq : PREBUILT_MAX_NQ;
    L.lut_img = take(nlut * ix->plan.lut_bytes);
    L.lut_inv = take(nlut * 4);
    L.lut_scale = take(nlut * 4);
    L.total = o;
    return L;
}

// Every pointer an index holds, and everything derived at load, belongs to one device.
static rago_status check_device(const IndexImpl* ix) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev != ix->device)
        return fail(RAGO_EINVAL, "the current device (%d) is not the index's device (%d)", dev, ix->device);
    return RAGO_OK;
}

static rago_status check_search_args(const IndexImpl* ix, int nq, int nprobe, int k) {
    if (!ix) return fail(RAGO_EINVAL, "index is null");
    if (nq < 0) return fail(RAGO_EINVAL, "nq = %d is negative", nq);
    if (nprobe < 1 || nprobe > ix->nlist) return fail(RAGO_EINVAL, "nprobe = %d outside [1, nlist = %d]", nprobe, ix->nlist);
    if (nprobe > MAX_K) return fail(RAGO_EUNSUPPORTED, "nprobe = %d exceeds %d", nprobe, MAX_K);
    if (k < 1) return fail(RAGO_EINVAL, "k = %d must be at least 1", k);
    if (k > MAX_K) return fail(RAGO_EUNSUPPORTED, "k = %d exceeds %d", k, MAX_K);
    if ((long long)nq * nprobe > 0x7fffffffLL - 4096) return fail(RAGO_EUNSUPPORTED, "nq * nprobe too large");
    if (ix->tree_n1 && nprobe > ix->tree_min_cand)
        return fail(RAGO_EINVAL, "nprobe = %d, but %d level-1 nodes can have as few as %d lists between them", nprobe,
                    ix->tree_b1, ix->tree_min_cand);
    return RAGO_OK;
}

static void record(IndexImpl* ix, int i, cudaStream_t s) {
    if (ix->profile) cudaEventRecord(ix->ev[i], s);
}

// fp (may be null): the selection kernel also plans the scan and builds the lookup tables (small batches).
static rago_status run_coarse(const IndexImpl* ix, const float* queries, int nq, int nprobe, uint8_t* ws,
                              const Layout& L, const FusedPlan* fp, bool kernel_clears, cudaStream_t s) {
    IndexImpl* mix = const_cast<IndexImpl*>(ix);
    cudaError_t e;
    int32_t* probe_list = reinterpret_cast<int32_t*>(ws + L.probe_list);
    float* probe_term = reinterpret_cast<float*>(ws + L.probe_term);
    float* probe_bias = reinterpret_cast<float*>(ws + L.probe_bias);
    float* scores = reinterpret_cast<float*>(ws + L.scores);
    record(mix, 0, s);
    if (L.tree_S) {
        unsigned long long* cand = reinterpret_cast<unsigned long long*>(ws + L.cand);
        int32_t* cand_cnt = reinterpret_cast<int32_t*>(ws + L.cand_cnt);
        e = launch_tree_candidates(ix, queries, nq, L.tree_S, L.tree_cap, cand, cand_cnt,
                                   kernel_clears ? reinterpret_cast<uint32_t*>(ws + L.err) : nullptr, s);
        if (e != cudaSuccess) return cuda_fail(e, "two-level coarse kernel");
        record(mix, 1, s);
        e = launch_select_probes_cand(ix, queries, cand, cand_cnt, 0u, L.tree_S, L.tree_cap, nq, nprobe, probe_list,
                                      probe_term, probe_bias, fp, s);
    } else if (L.tc) {
        // queries -> stacked bf16 parts, then the tensor-core kernel with the selection fused in
        const int parts = ix->cparts_n;
        e = launch_split_bf16(queries, (size_t)nq * ix->d, parts, ws + L.qparts, s);
        if (e != cudaSuccess) return cuda_fail(e, "query split kernel");
        alignas(64) unsigned char tmap_a[128];
        e = make_tmap_bf16(tmap_a, ws + L.qparts, (uint64_t)parts * nq, (uint64_t)ix->d, 128);
        if (e != cudaSuccess) return cuda_fail(e, "encoding the query tensor map");
        GemmLaunch G;
        G.tmap_a = tmap_a; G.tmap_b = ix->tmap_b; G.tmap_b_half = ix->tmap_b_half;
        G.nrows = nq; G.ncols = ix->nlist; G.d = ix->d;
        G.a_part_rows = nq; G.b_part_rows = ix->nlist;
        if (parts == 1) {
            G.nterms = 1; G.term_a[0] = 0; G.term_b[0] = 0;
            for (int t = 1; t < 6; ++t) G.term_a[t] = G.term_b[t] = 0;
        } else {  // smallest products first: (2,0) (1,1) (0,2) (1,0) (0,1) (0,0)
            const int ta[6] = {2, 1, 0, 1, 0, 0}, tb[6] = {0, 1, 2, 0, 1, 0};
            G.nterms = 6;
            for (int t = 0; t < 6; ++t) { G.term_a[t] = ta[t]; G.term_b[t] = tb[t]; }
        }
        G.mg = L.tc_mg; G.nsplit = L.tc_nsplit;
        G.alpha = ix->metric == RAGO_L2 ? -2.f : -1.f;
        G.colterm = ix->metric == RAGO_L2 ? ix->cnorm : nullptr;
        G.colterm_stride = 1;
        G.row_tau = nullptr;
        G.mode = L.tc_mode; G.cap = L.tc_cap;
        G.nsel = nprobe + PROBE_GUARD < ix->nlist ? nprobe + PROBE_GUARD : ix->nlist;
        G.cand = reinterpret_cast<unsigned long long*>(ws + L.cand);
        G.cand_cnt = reinterpret_cast<int32_t*>(ws + L.cand_cnt);
        G.scores = scores;
        G.err = reinterpret_cast<uint32_t*>(ws + L.err);
        if (L.pilot_cols) {
            // pilot pass: score every pilot_stride-th list, take each query's nsel-th smallest as its starting threshold
            GemmLaunch P = G;
            int mgroups = 1;
            P.tmap_b = ix->tmap_b_pilot; P.tmap_b_half = ix->tmap_b_pilot_half;
            P.ncols = L.pilot_cols; P.b_part_rows = L.pilot_cols;
            gemm_grid(nq, L.pilot_cols, ix->d * ix->cparts_n, ix->num_sms, &P.mg, &P.nsplit, &mgroups);
            P.colterm_stride = ix->pilot_stride;
            P.mode = 1;
            P.scores = reinterpret_cast<float*>(ws + L.pilot_scores);
            e = launch_gemm_select(P, s);
            if (e == cudaSuccess)
                e = launch_row_tau(P.scores, nq, L.pilot_cols, G.nsel, reinterpret_cast<float*>(ws + L.row_tau), s);
            if (e != cudaSuccess) return cuda_fail(e, "pilot pass of the coarse step");
            G.row_tau = reinterpret_cast<float*>(ws + L.row_tau);
        }
        e = launch_gemm_select(G, s);
        if (e != cudaSuccess) return cuda_fail(e, "tensor-core coarse kernel");
        record(mix, 1, s);
        if (L.tc_mode == 0)
            e = launch_select_probes_cand(ix, queries, G.cand, G.cand_cnt, gemm_cand_sign(G.alpha, G.colterm),
                                          L.tc_nsplit * GEMM_COL_HALVES, L.tc_cap, nq, nprobe, probe_list,
                                          probe_term, probe_bias, fp, s);
        else
            e = launch_select_probes(ix, queries, scores, nq, nprobe, probe_list, probe_term, probe_bias, fp, s);
    } else {
        e = launch_coarse_scores(ix, queries, nq, scores, kernel_clears ? reinterpret_cast<uint32_t*>(ws + L.err) : nullptr, s);
        if (e != cudaSuccess) return cuda_fail(e, "coarse score kernel");
        record(mix, 1, s);
        e = launch_select_probes(ix, queries, scores, nq, nprobe, probe_list, probe_term, probe_bias, fp, s);
    }
    if (e != cudaSuccess) return cuda_fail(e, "probe selection kernel");
    record(mix, 2, s);
    return RAGO_OK;
}

}  // namespace rago

using namespace rago;

extern "C" {

const char* rago_last_error(void) { return g_err; }
int64_t rago_kernel_launches(void) { return g_launches.load(); }

rago_status rago_index_load(rago_index** out, const void* coarse_centroids, rago_dtype coarse_dtype,
                            const float* pq_codebooks, const uint8_t* codes, const int64_t* list_offsets,
                            const int64_t* ids, int64_t N, int32_t d, int32_t nlist, int32_t M, rago_metric metric,
                            void* cuda_stream) {
    if (!out) return fail(RAGO_EINVAL, "out is null");
    *out = nullptr;
    if (!coarse_centroids || !pq_codebooks || !list_offsets) return fail(RAGO_EINVAL, "null index array");
    if (N < 0 || d <= 0 || nlist <= 0 || M <= 0) return fail(RAGO_EINVAL, "sizes must be positive");
    if (N > 0 && (!codes || !ids)) return fail(RAGO_EINVAL, "codes / ids are null but N > 0");
    if (metric != RAGO_L2 && metric != RAGO_IP) return fail(RAGO_EINVAL, "unknown metric %d", (int)metric);
    if (coarse_dtype != RAGO_F32 && coarse_dtype != RAGO_BF16) return fail(RAGO_EINVAL, "unknown coarse dtype");
    if (d % M != 0) return fail(RAGO_EINVAL, "d = %d is not a multiple of M = %d", d, M);
    if (!scan_supported(M)) return fail(RAGO_EUNSUPPORTED, "M = %d: supported sub-space counts are 16,32,48,64,80,96,128", M);
    if (d > 4096) return fail(RAGO_EUNSUPPORTED, "d = %d exceeds 4096", d);
    if (N >= (1LL << 32)) return fail(RAGO_EUNSUPPORTED, "N = %lld needs more than 32-bit positions", (long long)N);
    if (!aligned(coarse_centroids, 16) || !aligned(pq_codebooks, 16) || !aligned(codes, 16) ||
        !aligned(list_offsets, 8) || !aligned(ids, 8))
        return fail(RAGO_EALIGN, "index arrays must be 16-byte aligned (offsets and ids 8-byte)");
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    std::vector<int64_t> off((size_t)nlist + 1);
    cudaError_t e = cudaMemcpyAsync(off.data(), list_offsets, off.size() * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "reading list_offsets");
    if (off[0] != 0 || off[nlist] != N) return fail(RAGO_EINVAL, "list_offsets must start at 0 and end at N");
    for (int l = 0; l < nlist; ++l)
        if (off[l + 1] < off[l]) return fail(RAGO_EINVAL, "list_offsets decrease at list %d", l);

    IndexImpl* ix = new (std::nothrow) IndexImpl();
    if (!ix) return fail(RAGO_ENOMEM, "host allocation failed");
    std::memset(ix, 0, sizeof(*ix));
    ix->centroids = coarse_centroids;
    ix->coarse_bf16 = coarse_dtype == RAGO_BF16;
    ix->codebooks = pq_codebooks;
    ix->codes = codes;
    ix->list_offsets = list_offsets;
    ix->ids = ids;
    ix->N = N; ix->d = d; ix->nlist = nlist; ix->M = M; ix->dsub = d / M; ix->metric = metric;
    e = cudaGetDevice(&ix->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ix->num_sms, cudaDevAttrMultiProcessorCount, ix->device);
    if (e == cudaSuccess) e = cudaMalloc(&ix->cnorm, (size_t)nlist * 4);
    if (e == cudaSuccess) e = cudaMalloc(&ix->cbT, (size_t)KSUB * d * 4);
    if (e == cudaSuccess) e = cudaMalloc(&ix->cwmax, (size_t)M * 4);
    if (e == cudaSuccess && metric == RAGO_L2 && N > 0) e = cudaMalloc(&ix->vterm, ((size_t)N + 4) * 4);  // + slack: tiles copy whole 16-byte groups
    if (e != cudaSuccess) {
        rago_status st = e == cudaErrorMemoryAllocation ? fail(RAGO_ENOMEM, "device allocation failed")
                                                         : cuda_fail(e, "index setup");
        rago_index_free(reinterpret_cast<rago_index*>(ix));
        return st;
    }
    for (int i = 0; i <= RAGO_NUM_STAGES && e == cudaSuccess; ++i) e = cudaEventCreate(&ix->ev[i]);
    if (e == cudaSuccess) { ix->ev_valid = 1; e = scan_plan(ix, &ix->plan); }
    if (e == cudaSuccess) e = launch_centroid_norms(coarse_centroids, ix->coarse_bf16, nlist, d, ix->cnorm, s);
    if (e == cudaSuccess) e = launch_transpose_codebook(pq_codebooks, M, ix->dsub, ix->cbT, s);
    if (e == cudaSuccess) e = launch_codeword_norms(pq_codebooks, M, ix->dsub, ix->cwmax, s);
    if (e == cudaSuccess && ix->vterm) e = launch_vector_terms(ix, ix->vterm, s);
    // tensor-core coarse operand: the centroids as stacked bf16 parts, and their tensor map
    if (e == cudaSuccess && d % 8 == 0) {
        const void* bsrc = coarse_centroids;
        ix->cparts_n = 1;
        if (!ix->coarse_bf16) {
            ix->cparts_n = 3;
            e = cudaMalloc(&ix->cparts, (size_t)3 * nlist * d * 2);
            if (e == cudaSuccess) e = launch_split_bf16(static_cast<const float*>(coarse_centroids), (size_t)nlist * d, 3, ix->cparts, s);
            bsrc = ix->cparts;
        }
        if (e == cudaSuccess && gemm_select_init() == cudaSuccess &&
            make_tmap_bf16(ix->tmap_b, bsrc, (uint64_t)ix->cparts_n * nlist, (uint64_t)d, 256) == cudaSuccess &&
            make_tmap_bf16(ix->tmap_b_half, bsrc, (uint64_t)ix->cparts_n * nlist, (uint64_t)d, 128) == cudaSuccess)
            ix->tc_ok = 1;
        const int ps = gemm_pilot_stride(nlist);
        if (ix->tc_ok && nlist % ps == 0 &&
            make_tmap_bf16(ix->tmap_b_pilot, bsrc, (uint64_t)ix->cparts_n * (nlist / ps), (uint64_t)d, 256,
                           (uint64_t)ps * d) == cudaSuccess &&
            make_tmap_bf16(ix->tmap_b_pilot_half, bsrc, (uint64_t)ix->cparts_n * (nlist / ps), (uint64_t)d, 128,
                           (uint64_t)ps * d) == cudaSuccess)
            ix->pilot_stride = ps;
        cudaGetLastError();  // a missing tensor-core path is not an error: the fp32 kernel serves every batch
    }
    if (e == cudaSuccess) e = noalloc_prepare();  // the built-in scratch of rago_search_probes_noalloc becomes resident now
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        rago_status st = cuda_fail(e, "index setup kernels");
        rago_index_free(reinterpret_cast<rago_index*>(ix));
        return st;
    }
    *out = reinterpret_cast<rago_index*>(ix);
    return RAGO_OK;
}

rago_status rago_index_free(rago_index* index) {
    if (!index) return RAGO_OK;
    IndexImpl* ix = reinterpret_cast<IndexImpl*>(index);
    cudaDeviceSynchronize();
    if (ix->cnorm) cudaFree(ix->cnorm);
    if (ix->cbT) cudaFree(ix->cbT);
    if (ix->cwmax) cudaFree(ix->cwmax);
    if (ix->vterm) cudaFree(ix->vterm);
    if (ix->cparts) cudaFree(ix->cparts);
    if (ix->ev_valid)
        for (int i = 0; i <= RAGO_NUM_STAGES; ++i) cudaEventDestroy(ix->ev[i]);
    delete ix;
    return RAGO_OK;
}

rago_status rago_search_workspace_bytes(const rago_index* index, int32_t nq, int32_t nprobe, int32_t k,
                                        size_t* out_bytes) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    if (!out_bytes) return fail(RAGO_EINVAL, "out_bytes is null");
    rago_status st = check_search_args(ix, nq, nprobe, k);
    if (st != RAGO_OK) return st;
    *out_bytes = make_layout(ix, nq, nprobe, k).total;
    return RAGO_OK;
}

rago_status rago_host_staging_bytes(const rago_index* index, int32_t nq, int32_t k, size_t* out_bytes) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    if (!ix || !out_bytes || nq < 0 || k < 1) return fail(RAGO_EINVAL, "bad arguments");
    *out_bytes = align_up((size_t)nq * ix->d * 4, 256) + align_up((size_t)nq * k * 8, 256) +
                 align_up((size_t)nq * k * 4, 256);
    return RAGO_OK;
}

rago_status rago_search_probes(const rago_index* index, const float* queries, int32_t nq, int32_t nprobe,
                               int32_t* out_lists, float* out_coarse, void* workspace, size_t workspace_bytes,
                               void* cuda_stream) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    rago_status st = check_search_args(ix, nq, nprobe, 1);
    if (st != RAGO_OK) return st;
    if (nq == 0) return RAGO_OK;
    if (!queries || !out_lists || !out_coarse || !workspace) return fail(RAGO_EINVAL, "null pointer");
    if (!aligned(queries, 16) || !aligned(workspace, 256)) return fail(RAGO_EALIGN, "queries need 16-byte, workspace 256-byte alignment");
    st = check_device(ix);
    if (st != RAGO_OK) return st;
    const Layout L = make_layout(ix, nq, nprobe, 1);
    if (workspace_bytes < L.total) return fail(RAGO_ENOMEM, "workspace holds %zu bytes, %zu needed", workspace_bytes, L.total);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaError_t e = cudaMemsetAsync(ws + L.err, 0, 256, s);
    if (e != cudaSuccess) return cuda_fail(e, "clearing the error word");
    st = run_coarse(ix, queries, nq, nprobe, ws, L, nullptr, false, s);
    if (st != RAGO_OK) return st;
    const size_t bytes = (size_t)nq * nprobe * 4;
    e = cudaMemcpyAsync(out_lists, ws + L.probe_list, bytes, cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_coarse, ws + L.probe_term, bytes, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e, "copying probe table");
    return RAGO_OK;
}

rago_status rago_search(const rago_index* index, const float* queries, int32_t nq, int32_t nprobe, int32_t k,
                        int64_t* out_ids, float* out_dists, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    rago_status st = check_search_args(ix, nq, nprobe, k);
    if (st != RAGO_OK) return st;
    if (nq == 0) return RAGO_OK;
    if (!queries || !out_ids || !out_dists || !workspace) return fail(RAGO_EINVAL, "null pointer");
    if (!aligned(queries, 16) || !aligned(workspace, 256) || !aligned(out_ids, 8) || !aligned(out_dists, 4))
        return fail(RAGO_EALIGN, "queries need 16-byte, workspace 256-byte alignment");
    st = check_device(ix);
    if (st != RAGO_OK) return st;
    const Layout L = make_layout(ix, nq, nprobe, k);
    if (workspace_bytes < L.total) return fail(RAGO_ENOMEM, "workspace holds %zu bytes, %zu needed", workspace_bytes, L.total);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    IndexImpl* mix = const_cast<IndexImpl*>(ix);
    const int npairs = nq * nprobe;

    // The error block is cleared first: by the tiny-batch coarse kernel or the two-level kernel itself when that is the first kernel
    // of the search (a memset between two searches would keep their launches from overlapping), else by a memset.
    const bool kernel_clears = L.tree_S ? true : (!L.tc && coarse_small_applies(ix, nq));
    cudaError_t e = kernel_clears ? cudaSuccess : cudaMemsetAsync(ws + L.err, 0, 256, s);
    if (e != cudaSuccess) return cuda_fail(e, "clearing the error word");
    int32_t* probe_list = reinterpret_cast<int32_t*>(ws + L.probe_list);
    float* probe_term = reinterpret_cast<float*>(ws + L.probe_bias);  // what the scan adds per (query, list)
    int64_t* work_prefix = reinterpret_cast<int64_t*>(ws + L.work_prefix);
    unsigned long long* qthresh = reinterpret_cast<unsigned long long*>(ws + L.qthresh);
    int32_t* slot_cnt = reinterpret_cast<int32_t*>(ws + L.slot_cnt);
    unsigned long long* slot_keys = reinterpret_cast<unsigned long long*>(ws + L.slot_keys);
    // small batches: the lookup tables are built ahead of the scan
    uint8_t* lut_img = L.prebuilt ? ws + L.lut_img : nullptr;
    float* lut_inv = L.prebuilt ? reinterpret_cast<float*>(ws + L.lut_inv) : nullptr;

    // Batches of at most 64 queries: the selection launch also builds the tables and plans the scan (its last CTA
    // to finish), one launch less on the latency-bound path.  The ticket word lies in the block cleared above.
    FusedPlan fp;
    const bool fused = fused_plan_args(ix, nq, npairs, queries, lut_img, lut_inv, work_prefix, qthresh, slot_cnt,
                                       (int)L.nslots, reinterpret_cast<uint32_t*>(ws + L.err) + ERR_TICKET_WORD, &fp);
    st = run_coarse(ix, queries, nq, nprobe, ws, L, fused ? &fp : nullptr, kernel_clears, s);
    if (st != RAGO_OK) return st;
    if (!fused) {
        e = launch_plan_work(ix, probe_list, npairs, ix->plan.tile_vecs, reinterpret_cast<int32_t*>(ws + L.pair_tiles),
                             work_prefix, qthresh, nq, slot_cnt, (int)L.nslots, queries, lut_img, lut_inv,
                             L.prebuilt ? reinterpret_cast<float*>(ws + L.lut_scale) : nullptr, s);
        if (e != cudaSuccess) return cuda_fail(e, "work planning");
    }
    record(mix, 3, s);
    e = launch_scan(ix, ix->plan, queries, probe_list, probe_term, work_prefix, nq, nprobe, k, qthresh, slot_cnt,
                    slot_keys, reinterpret_cast<uint32_t*>(ws + L.err), lut_img, lut_inv, s);
    if (e != cudaSuccess) return cuda_fail(e, "scan kernel");
    record(mix, 4, s);
    e = launch_merge(ix, work_prefix, nq, nprobe, k, ix->plan.ctas, slot_cnt, slot_keys, qthresh, queries, probe_list, probe_term,
                     out_ids, out_dists, s);
    if (e != cudaSuccess) return cuda_fail(e, "merge kernel");
    record(mix, 5, s);
    return RAGO_OK;
}

rago_status rago_search_host(const rago_index* index, const float* host_queries, int32_t nq, int32_t nprobe,
                             int32_t k, int64_t* host_out_ids, float* host_out_dists, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    rago_status st = check_search_args(ix, nq, nprobe, k);
    if (st != RAGO_OK) return st;
    if (nq == 0) return RAGO_OK;
    if (!host_queries || !host_out_ids || !host_out_dists || !workspace) return fail(RAGO_EINVAL, "null pointer");
    if (!aligned(workspace, 256)) return fail(RAGO_EALIGN, "workspace needs 256-byte alignment");
    st = check_device(ix);
    if (st != RAGO_OK) return st;
    const Layout L = make_layout(ix, nq, nprobe, k);
    size_t staging = 0;
    rago_host_staging_bytes(index, nq, k, &staging);
    if (workspace_bytes < L.total + staging)
        return fail(RAGO_ENOMEM, "workspace holds %zu bytes, %zu needed", workspace_bytes, L.total + staging);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* st0 = ws + L.total;
    float* dq = reinterpret_cast<float*>(st0);
    int64_t* dids = reinterpret_cast<int64_t*>(st0 + align_up((size_t)nq * ix->d * 4, 256));
    float* ddist = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(dids) + align_up((size_t)nq * k * 8, 256));
    cudaError_t e = cudaMemcpyAsync(dq, host_queries, (size_t)nq * ix->d * 4, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e, "copying queries to the device");
    st = rago_search(index, dq, nq, nprobe, k, dids, ddist, workspace, L.total, cuda_stream);
    if (st != RAGO_OK) return st;
    e = cudaMemcpyAsync(host_out_ids, dids, (size_t)nq * k * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_out_dists, ddist, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "copying results to the host");
    return RAGO_OK;
}

rago_status rago_flat_workspace_bytes(int64_t N, int32_t d, int32_t nq, int32_t k, size_t* out_bytes) {
    if (!out_bytes) return fail(RAGO_EINVAL, "out_bytes is null");
    if (N < 0 || d <= 0 || nq < 0 || k < 1) return fail(RAGO_EINVAL, "bad sizes");
    if (k > MAX_K) return fail(RAGO_EUNSUPPORTED, "k = %d exceeds %d", k, MAX_K);
    *out_bytes = flat_workspace_bytes(N, d, nq, k);
    return RAGO_OK;
}

rago_status rago_flat_search(const void* db, int64_t N, int32_t d, const void* queries, int32_t nq, int32_t k,
                             int64_t* out_ids, float* out_scores, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
    if (N < 0 || d <= 0 || nq < 0) return fail(RAGO_EINVAL, "bad sizes");
    if (k < 1) return fail(RAGO_EINVAL, "k = %d must be at least 1", k);
    if (k > MAX_K) return fail(RAGO_EUNSUPPORTED, "k = %d exceeds %d", k, MAX_K);
    if (d % 64 != 0 || d > 4096) return fail(RAGO_EUNSUPPORTED, "d = %d must be a multiple of 64, at most 4096", d);
    if (N >= (1LL << 31)) return fail(RAGO_EUNSUPPORTED, "N needs more than 31-bit row numbers");
    if (nq == 0) return RAGO_OK;
    if ((N > 0 && !db) || !queries || !out_ids || !out_scores || !workspace) return fail(RAGO_EINVAL, "null pointer");
    if (!aligned(db, 16) || !aligned(queries, 16) || !aligned(workspace, 256))
        return fail(RAGO_EALIGN, "db and queries need 16-byte, workspace 256-byte alignment");
    const size_t need = flat_workspace_bytes(N, d, nq, k);
    if (workspace_bytes < need) return fail(RAGO_ENOMEM, "workspace holds %zu bytes, %zu needed", workspace_bytes, need);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, 256, s);
    if (e == cudaSuccess) e = launch_flat_search(db, N, d, queries, nq, k, out_ids, out_scores, workspace, s);
    if (e != cudaSuccess) return cuda_fail(e, "flat search");
    return RAGO_OK;
}

rago_status rago_check(void* workspace, void* cuda_stream) {
    if (!workspace) return fail(RAGO_EINVAL, "workspace is null");
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint32_t w = 0;
    cudaError_t e = cudaMemcpyAsync(&w, workspace, 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "reading the error word");
    if (w == ERR_WAIT_TIMEOUT) return fail(RAGO_ETIMEOUT, "a bounded device-side wait expired");
    if (w == ERR_SMEM_LAYOUT) return fail(RAGO_ECUDA, "the scan kernel's shared-memory plan does not fit this device");
    if (w != ERR_NONE) return fail(RAGO_ECUDA, "device error word = %u", w);
    return RAGO_OK;
}

rago_status rago_index_set_coarse_tree(rago_index* index, const void* level1_centroids, const int32_t* child_offsets,
                                       int32_t n1, int32_t b1, void* cuda_stream) {
    if (!index) return fail(RAGO_EINVAL, "index is null");
    IndexImpl* ix = reinterpret_cast<IndexImpl*>(index);
    rago_status st = check_device(ix);
    if (st != RAGO_OK) return st;
    if (n1 == 0) {  // back to the one-level quantiser
        ix->tree_n1 = ix->tree_b1 = 0;
        ix->tree_level1 = nullptr; ix->tree_child_offsets = nullptr;
        return RAGO_OK;
    }
    if (!level1_centroids || !child_offsets) return fail(RAGO_EINVAL, "null pointer");
    if (n1 < 1 || n1 > ix->nlist) return fail(RAGO_EINVAL, "n1 = %d outside [1, nlist = %d]", n1, ix->nlist);
    if (b1 < 1 || b1 > n1) return fail(RAGO_EINVAL, "b1 = %d outside [1, n1 = %d]", b1, n1);
    if (n1 > TREE_LIMIT_N1 || b1 > TREE_LIMIT_B1)
        return fail(RAGO_EUNSUPPORTED, "n1 = %d / b1 = %d exceed %d / %d", n1, b1, TREE_LIMIT_N1, TREE_LIMIT_B1);
    if (ix->d % 4 != 0) return fail(RAGO_EUNSUPPORTED, "d = %d must be a multiple of 4 for the two-level quantiser", ix->d);
    if (!aligned(level1_centroids, 16) || !aligned(child_offsets, 4)) return fail(RAGO_EALIGN, "level-1 centroids need 16-byte alignment");
    if ((size_t)ix->d * 4 + (size_t)n1 * 8 > 48 * 1024)
        return fail(RAGO_EUNSUPPORTED, "d = %d with n1 = %d does not fit the kernel's shared memory", ix->d, n1);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    std::vector<int32_t> off((size_t)n1 + 1);
    cudaError_t e = cudaMemcpyAsync(off.data(), child_offsets, off.size() * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "reading child_offsets");
    if (off[0] != 0 || off[n1] != ix->nlist) return fail(RAGO_EINVAL, "child_offsets must start at 0 and end at nlist");
    std::vector<int> cnt(n1);
    for (int i = 0; i < n1; ++i) {
        if (off[i + 1] < off[i]) return fail(RAGO_EINVAL, "child_offsets decrease at node %d", i);
        cnt[i] = off[i + 1] - off[i];
    }
    std::sort(cnt.begin(), cnt.end());
    long long mn = 0, mx = 0;
    for (int i = 0; i < b1; ++i) { mn += cnt[i]; mx += cnt[n1 - 1 - i]; }
    ix->tree_level1 = level1_centroids;
    ix->tree_child_offsets = child_offsets;
    ix->tree_n1 = n1; ix->tree_b1 = b1;
    ix->tree_min_cand = (int)mn; ix->tree_max_cand = (int)mx;
    return RAGO_OK;
}

rago_status rago_debug_set_gemm_pairing(int32_t mode) {
    if (mode < 0 || mode > 3) return fail(RAGO_EINVAL, "mode = %d: 0 by operand size, 1 single, 2 pair in a CTA, 3 CTA pair", mode);
    gemm_set_pairing(mode);
    return RAGO_OK;
}

rago_status rago_selftest_wait_timeout(void* workspace, uint32_t max_polls, int32_t with_tmem, void* cuda_stream) {
    if (!workspace) return fail(RAGO_EINVAL, "workspace is null");
    if (!aligned(workspace, 256)) return fail(RAGO_EALIGN, "workspace needs 256-byte alignment");
    if (max_polls < 1 || max_polls > 4096) return fail(RAGO_EINVAL, "max_polls = %u outside [1, 4096]", max_polls);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint32_t* w = static_cast<uint32_t*>(workspace);
    cudaError_t e = cudaMemsetAsync(workspace, 0, 256, s);
    if (e == cudaSuccess) e = launch_selftest_wait(w, max_polls, with_tmem ? 1 : 0, w + 8, s);
    if (e != cudaSuccess) return cuda_fail(e, "wait self-test");
    return RAGO_OK;
}

rago_status rago_set_coarse_mode(rago_index* index, int32_t mode) {
    if (!index) return fail(RAGO_EINVAL, "index is null");
    if (mode < 0 || mode > 2) return fail(RAGO_EINVAL, "mode = %d: 0 auto, 1 fp32 pipes, 2 tensor cores", mode);
    IndexImpl* ix = reinterpret_cast<IndexImpl*>(index);
    if (mode == 2 && !ix->tc_ok) return fail(RAGO_EUNSUPPORTED, "the tensor-core coarse path is not available for this index");
    ix->coarse_mode = mode;
    return RAGO_OK;
}

rago_status rago_profile_enable(rago_index* index, int32_t enable) {
    if (!index) return fail(RAGO_EINVAL, "index is null");
    reinterpret_cast<IndexImpl*>(index)->profile = enable ? 1 : 0;
    return RAGO_OK;
}

rago_status rago_profile_read(rago_index* index, float* out_ms) {
    IndexImpl* ix = reinterpret_cast<IndexImpl*>(index);
    if (!ix || !out_ms) return fail(RAGO_EINVAL, "null pointer");
    if (!ix->profile) return fail(RAGO_EINVAL, "profiling is not enabled");
    cudaError_t e = cudaEventSynchronize(ix->ev[RAGO_NUM_STAGES]);
    for (int i = 0; i < RAGO_NUM_STAGES && e == cudaSuccess; ++i)
        e = cudaEventElapsedTime(&out_ms[i], ix->ev[i], ix->ev[i + 1]);
    if (e != cudaSuccess) return cuda_fail(e, "reading stage timings");
    return RAGO_OK;
}

}  // extern "C"
