/*
 * rago.h -- C ABI of the B200 (sm_100a) retrieval library.
 *
 * The library implements the retrieval stage that retrieval-augmented generation adds to LLM
 * serving, as the RAGO paper states it (Background, "Vector search for retrieval"): return the K
 * database vectors most similar to a D-dimensional query under L2 distance or cosine / inner
 * product, either approximately with IVF-PQ (an inverted file over product-quantised vectors,
 * one byte per sub-space) or exactly by brute force for small databases (case study II).  The
 * paper's cost model for the stage is the number of bytes of quantised vectors scanned per query
 * (RAGSchema section, "Retrieval component").
 *
 * Conventions for every call
 *   - "dev" pointers are CUDA device pointers in the current device's address space; "host"
 *     pointers are ordinary host memory.  Nothing here takes or returns a framework type.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns without synchronising, unless stated otherwise.
 *   - The caller owns every buffer it passes.  An index BORROWS its arrays: they must stay valid
 *     and unchanged until rago_index_free.  Scratch memory is caller-provided ("workspace"), with
 *     one exception (rago_search_probes_noalloc, which uses an array built into the library); the
 *     search calls allocate nothing.
 *   - An index belongs to the device that was current when it was loaded; every call that takes an
 *     index must be made with that device current, otherwise it returns RAGO_EINVAL.
 *   - Errors are return codes.  Argument errors are found on the host before anything is
 *     launched.  rago_last_error() returns a thread-local description of the last failure.
 *   - L2 means SQUARED Euclidean distance, smaller is better, results ascending.  IP means inner
 *     product, larger is better, results descending.  Missing results (fewer than k candidates)
 *     are id -1 with +INFINITY (L2) or -INFINITY (IP).
 *   - Product-quantisation codes are 8 bits (256 codewords per sub-space, rago_index_load) or 4 bits
 *     (16 codewords, two codes per byte, rago_index_load_pq4).
 */
#ifndef RAGO_H
#define RAGO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rago_index rago_index; /* opaque */

typedef enum {
    RAGO_OK = 0,
    RAGO_EINVAL = 1,       /* null pointer, non-positive size, k or nprobe out of range, bad offsets */
    RAGO_EALIGN = 2,       /* a pointer is not aligned as documented */
    RAGO_EUNSUPPORTED = 3, /* shape outside the supported envelope (see rago_index_load) */
    RAGO_ENOMEM = 4,       /* workspace too small, or an allocation at index load failed */
    RAGO_ECUDA = 5,        /* a CUDA runtime call failed */
    RAGO_ETIMEOUT = 6      /* a bounded device-side wait expired (reported by rago_check) */
} rago_status;

typedef enum { RAGO_L2 = 0, RAGO_IP = 1 } rago_metric;
typedef enum { RAGO_F32 = 0, RAGO_BF16 = 1 } rago_dtype;

/* Number of per-stage timings rago_profile_read returns:
 * 0 coarse distances, 1 probe selection, 2 work planning, 3 table build + scan, 4 merge. */
#define RAGO_NUM_STAGES 5

/*
 * Build a search handle over an IVF-PQ index that already lives in device memory
 * (IVF-PQ: Background, "Vector search for retrieval"; storage is the usual inverted file:
 * vectors of one list stored contiguously, lists addressed by offsets).
 *
 *   coarse_centroids  dev [nlist][d], row-major, RAGO_F32 or RAGO_BF16 (16-byte aligned)
 *   pq_codebooks      dev [M][256][d/M] fp32: codeword j of sub-space m
 *   codes             dev [N][M] uint8, 16-byte aligned; vectors of list l occupy rows
 *                     list_offsets[l] .. list_offsets[l+1]-1.  A code quantises the RESIDUAL
 *                     (vector - its list's centroid); one codebook set serves all lists.
 *   list_offsets      dev [nlist+1] int64, offsets[0]=0, non-decreasing, offsets[nlist]=N
 *   ids               dev [N] int64, caller-chosen ids reported in results
 *   N, d, nlist, M    sizes; d % M == 0
 *   metric            RAGO_L2 or RAGO_IP.  For IP the score of a vector is
 *                     <q, centroid> + sum over sub-spaces of <q_m, codeword>.
 *
 * Supported envelope: M a multiple of 16 with M <= 192 and M not in {112, 144, 176};
 * d <= 4096; N < 2^32; nlist < 2^31.  Anything else returns RAGO_EUNSUPPORTED.
 *
 * This call synchronises: it copies list_offsets to the host to validate them, allocates the
 * small derived arrays the library owns (centroid norms, a transposed codebook) and fills them.
 * On success *out receives the handle.
 */
rago_status rago_index_load(rago_index** out, const void* coarse_centroids, rago_dtype coarse_dtype,
                            const float* pq_codebooks, const uint8_t* codes, const int64_t* list_offsets,
                            const int64_t* ids, int64_t N, int32_t d, int32_t nlist, int32_t M,
                            rago_metric metric, void* cuda_stream);

/*
 * Load an index whose product quantiser uses 4-bit codes: the paper's low-precision PQ variant (Sec. 2,
 * vector search background: 4-bit codes make the scan memory-bound, 8-bit codes compute-bound on CPUs).
 * M4 sub-spaces of 16 codewords each; two codes share a byte, sub-space 2j in the low nibble of byte j and
 * sub-space 2j + 1 in the high nibble, so a vector occupies M4 / 2 bytes.
 *
 *   pq4_codebooks  device, fp32 [M4][16][d / M4], 16-byte aligned; read during the call only
 *   packed_codes   device, uint8 [N][M4 / 2], list-contiguous like rago_index_load's codes; borrowed
 *   everything else as in rago_index_load
 *
 * The result is an ordinary rago_index with M = M4 / 2 code bytes per vector: every search call takes it, and
 * scores follow the same definitions with the decoded vector centroid + concatenated 4-bit codewords.
 * M4 / 2 must be one of the supported code sizes (16, 32, 48, 64, 80, 96, 128).  Allocates and frees a
 * temporary of 1024 * d bytes and synchronises cuda_stream.  Errors as rago_index_load, plus RAGO_EINVAL for an
 * odd M4.
 */
rago_status rago_index_load_pq4(rago_index** out, const void* coarse_centroids, rago_dtype coarse_dtype,
                                const float* pq4_codebooks, const uint8_t* packed_codes, const int64_t* list_offsets,
                                const int64_t* ids, int64_t N, int32_t d, int32_t nlist, int32_t M4,
                                rago_metric metric, void* cuda_stream);

/*
 * Put a second quantiser level above the coarse centroids, or remove it (n1 = 0).  The paper's index is a
 * multi-level tree whose levels are scanned top-down, each level's best nodes deciding which nodes of the next
 * are scored (Methodology: "Models and database", and the retrieval performance model: one scan operator per
 * level).  With the level set, the coarse step of every search on this index scores the n1 level-1 centroids,
 * keeps the best b1 nodes (same score as the coarse step: squared L2 distance or inner product, with the query
 * rounded to bf16 for a RAGO_BF16 quantiser; ties to the smaller node number), and chooses the nprobe probe lists
 * among the children of those nodes only.  Everything after the coarse step is unchanged.  The result is what
 * the two-level definition gives, which differs from the one-level search whenever a good list hangs under a
 * node that was not kept; b1 = n1 reproduces the one-level search.
 *
 *   level1_centroids  dev [n1][d], row-major, the index's coarse dtype, 16-byte aligned; borrowed until the
 *                     level is removed or the index freed
 *   child_offsets     dev [n1 + 1] int32, offsets[0] = 0, non-decreasing, offsets[n1] = nlist: node i owns the
 *                     consecutive lists offsets[i] .. offsets[i + 1] - 1; borrowed likewise
 *   n1, b1            1 <= b1 <= n1 <= nlist; b1 <= 64, n1 <= 4096, d a multiple of 4, d * 4 + n1 * 8 <= 48 KB,
 *                     else RAGO_EUNSUPPORTED
 *
 * A search whose nprobe exceeds the number of lists the b1 smallest nodes own is refused with RAGO_EINVAL
 * (the b1 kept nodes might not have nprobe children).  Workspace sizes change with the level: ask for them
 * after this call.  Synchronises cuda_stream (it reads child_offsets to validate them).
 * rago_search_probes_noalloc is not available while a level is set.
 */
rago_status rago_index_set_coarse_tree(rago_index* index, const void* level1_centroids, const int32_t* child_offsets,
                                       int32_t n1, int32_t b1, void* cuda_stream);

/* Release the handle and the arrays the library allocated for it (never the borrowed ones).
 * Synchronises the device first.  NULL is accepted. */
rago_status rago_index_free(rago_index* index);

/* Bytes of device scratch rago_search / rago_search_probes / rago_search_host need for a batch
 * of nq queries with these nprobe and k (1 <= nprobe <= nlist, 1 <= k <= 1024).  Its largest parts are
 * the per-query lookup tables (64 to 160 KB each, for at most 4096 queries of a batch: 128 KB per
 * query at M = 96) and, for batches the tensor-core coarse step does not take, nq * nlist scores. */
rago_status rago_search_workspace_bytes(const rago_index* index, int32_t nq, int32_t nprobe, int32_t k,
                                        size_t* out_bytes);

/*
 * Batched IVF-PQ search (the whole hot path): coarse query-to-centroid distances with nprobe
 * selection, per-(query, list) lookup tables, table-sum scan of the probed lists, k best.
 *
 *   queries    dev [nq][d] fp32, 16-byte aligned
 *   out_ids    dev [nq][k] int64, best first
 *   out_dists  dev [nq][k] fp32: squared L2 distance, or inner-product score
 *   workspace  dev, 256-byte aligned, at least rago_search_workspace_bytes(...) bytes; contents
 *              are scratch.  Two searches that overlap on the GPU need distinct workspaces.
 *
 * With a RAGO_BF16 coarse quantiser the query is rounded to bf16 (nearest-even) for the coarse
 * step only; tables are built from the fp32 query.  Ties are broken by storage position.
 * nq == 0 is a no-op.
 *
 * Accuracy of out_dists (fp32).  Candidates are RANKED by an expanded form of the score,
 * ||q-c||^2 + (||r||^2 + 2<c,r>) - 2<q,r> for L2 and <q,c> + <q,r> for IP (c the list's centroid, r the
 * decoded residual), whose table sum is exact in fixed point (per-query step at most max|entry| * M / 2^30);
 * its absolute error is a few fp32 ulps of the LARGEST of its terms.  Reported L2 distances are accurate to
 * about 1e-5 RELATIVE: a result whose value is below 1/32 of its largest term (a query that nearly coincides
 * with a stored vector) is re-computed in the direct form sum_j ((q_j - c_j) - cw_j)^2 before it is written,
 * and the k results are re-ordered by the corrected values.  Two candidates whose true distances differ by
 * less than the ranking error may still swap places at the k-th position.  IP scores are sums of mixed
 * sign: their error is absolute, a few ulps of max(|<q,c>|, |<q,r>|), not relative to the (possibly
 * cancelling) result.
 */
rago_status rago_search(const rago_index* index, const float* queries, int32_t nq, int32_t nprobe, int32_t k,
                        int64_t* out_ids, float* out_dists, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/*
 * The coarse step alone (test hook for the first stage of rago_search).
 *   out_lists   dev [nq][nprobe] int32 list numbers, best first
 *   out_coarse  dev [nq][nprobe] fp32: squared L2 distance to the centroid, or <q, centroid>
 */
rago_status rago_search_probes(const rago_index* index, const float* queries, int32_t nq, int32_t nprobe,
                               int32_t* out_lists, float* out_coarse, void* workspace, size_t workspace_bytes,
                               void* cuda_stream);

/*
 * The coarse step for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this call; it exists for deployment reasons only.)
 *
 * Who needs it: a retrieval worker that shares its GPU with an LLM server whose memory pool has
 * already claimed the free HBM, so that a cudaMalloc for a workspace would fail or stall the
 * other tenant; code that runs where an allocation is not allowed because it synchronises the
 * device (inside a latency-critical serving loop, or between the steps of another stream's
 * pipeline); and embedders that hand the library nothing but input and output buffers.
 *
 * Same inputs, outputs and results as rago_search_probes, but there is no workspace argument:
 * the query-by-list score matrix is kept in an array of RAGO_NOALLOC_SCRATCH_BYTES that is part
 * of the library image.  A GPU gives up that much memory from the first rago_index_load on it
 * (which looks the array up, so the CUDA runtime loads it then; a failure shows there as
 * RAGO_ECUDA) until the process ends.  The call itself allocates and frees nothing.
 *
 *   limit     align256(nq * nlist * 4) + align256(nq * nprobe * 4) <= RAGO_NOALLOC_SCRATCH_BYTES;
 *             a larger batch is refused with RAGO_ENOMEM and a message that names the limit
 *             (split the batch, or use rago_search_probes).
 *   set-up    rago_index_load looks up the array's device address (cudaGetSymbolAddress) with the
 *             index's device current, once per device, and this call reuses it.  Should that
 *             look-up have failed, the first call here repeats it; such a first call must come
 *             before any stream capture.
 *   device    the array's address differs per device: the call returns RAGO_EINVAL unless the
 *             current device is the index's.
 *   sharing   all calls on a device use the same array and find the previous call's contents in
 *             it.  Nothing needs clearing (every word read is written first by the same call),
 *             but two calls that overlap on the GPU - different streams, or different host
 *             threads - race on it and return garbage.  Serialise them on one stream.
 */
#define RAGO_NOALLOC_SCRATCH_BYTES (4 * 1024 * 1024)
rago_status rago_search_probes_noalloc(const rago_index* index, const float* queries, int32_t nq, int32_t nprobe,
                                       int32_t* out_lists, float* out_coarse, void* cuda_stream);

/*
 * rago_search for callers whose queries and results live in HOST memory: copies the queries to
 * the device, searches, copies ids and distances back, all on `cuda_stream`, then synchronises
 * that stream.  `workspace` must be 256-byte aligned and hold
 * rago_search_workspace_bytes(...) + rago_host_staging_bytes(...) bytes.  Pinned host buffers
 * make the copies asynchronous; pageable ones work too.
 */
rago_status rago_search_host(const rago_index* index, const float* host_queries, int32_t nq, int32_t nprobe,
                             int32_t k, int64_t* host_out_ids, float* host_out_dists, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);
rago_status rago_host_staging_bytes(const rago_index* index, int32_t nq, int32_t k, size_t* out_bytes);

/*
 * Exact (brute-force) search for small databases: score = <q, y_i> over bf16 inputs with fp32
 * accumulation, k largest, best first.  For cosine similarity pass unit-norm rows and queries.
 *
 *   db          dev [N][d] bf16 row-major, 16-byte aligned; d a multiple of 64, d <= 4096
 *   queries     dev [nq][d] bf16, 16-byte aligned
 *   out_ids     dev [nq][k] int64 row numbers; out_scores dev [nq][k] fp32
 *   workspace   dev, 256-byte aligned, rago_flat_workspace_bytes(...) bytes
 *   1 <= k <= 1024, N < 2^31.
 */
rago_status rago_flat_search(const void* db, int64_t N, int32_t d, const void* queries, int32_t nq, int32_t k,
                             int64_t* out_ids, float* out_scores, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);
rago_status rago_flat_workspace_bytes(int64_t N, int32_t d, int32_t nq, int32_t k, size_t* out_bytes);

/*
 * Synchronise `cuda_stream` and report whether any kernel launched through `workspace` since
 * the last check recorded a device-side error (RAGO_ETIMEOUT: a bounded wait on a copy or on the
 * tensor pipe gave up; the results of that call are then undefined).  Device waits never spin
 * without a limit.
 */
rago_status rago_check(void* workspace, void* cuda_stream);

/*
 * Test hook (no counterpart in the paper).  The tensor-core kernel has three main loops: one row tile of 128
 * queries per CTA; two row tiles per CTA that share every tile of the other operand; or a cluster of two CTAs
 * (one SM pair, tcgen05 cta_group::2) that shares it.  By default batches of more than 128 queries take the
 * CTA pair and smaller ones the single row tile; this call forces the choice process-wide so that tests and
 * measurements reach every loop: 0 = default, 1 = never share, 2 = share inside a CTA, 3 = share across a CTA
 * pair (2 and 3 apply to batches of more than 128 queries).  Workspace sizes depend on it: set it before asking for them.  Not thread-safe against
 * running searches.
 */
rago_status rago_debug_set_gemm_pairing(int32_t mode);

/*
 * Test hook for the failure path of rago_check (no counterpart in the paper: the library's kernels wait on
 * copies and on the tensor pipe, every such wait is bounded, and this call lets a test see a bound expire
 * without anything being wrong).  Launches one small kernel in which a wait on a barrier that nothing signals
 * gives up after `max_polls` polls (1 .. 4096, each at most 4 microseconds) exactly as a wait inside a search
 * kernel would: it records RAGO_ETIMEOUT in the first word of `workspace`, a second waiting warp is released by
 * the abort flag, and with `with_tmem` != 0 the kernel holds and then releases the SM's tensor memory the way
 * the tensor-core kernel does.  The kernel ends normally; the device stays usable.
 *
 *   workspace   dev, 256-byte aligned, at least 256 bytes.  After the call (asynchronous on cuda_stream)
 *               rago_check(workspace, stream) returns RAGO_ETIMEOUT; words 8 and 9 of the workspace are 1 if
 *               the first wait expired and if the second was released by the abort flag.  Any later search
 *               call that is given this workspace clears the error word first.
 */
rago_status rago_selftest_wait_timeout(void* workspace, uint32_t max_polls, int32_t with_tmem, void* cuda_stream);

/*
 * Which kernel computes the coarse scores: 0 = automatic (tensor cores for batches of more than 16
 * queries, the fp32 kernel for smaller ones), 1 = always the fp32 kernel, 2 = always tensor cores.
 * The tensor-core kernel multiplies bf16 operands; fp32 queries and centroids are split into three
 * bf16 parts each and the six leading part products are accumulated in fp32, so both kernels rank
 * the lists alike up to fp32 rounding, and either way the best nprobe + 8 lists are re-scored
 * exactly before the final cut.  Workspace sizes depend on the mode: set it before asking for
 * them.  Mode 2 on an index whose d is not a multiple of 8 returns RAGO_EUNSUPPORTED.
 */
rago_status rago_set_coarse_mode(rago_index* index, int32_t mode);

/*
 * Aggregation step of a database that is split into shards with independent indexes (paper, Sec. 4,
 * retrieval performance model: queries go to every shard, results are aggregated).  Every shard has
 * answered the same nq queries with k_in results each (rago_search's output layout, padding id -1
 * allowed anywhere); for each query the k_out best entries of the union are written best first.
 *
 *   part_ids    device, int64: shard p's row of query q starts at part_ids[p * part_stride + q * k_in];
 *               the gathered buffers of nparts ranks laid end to end have part_stride = nq * k_in
 *   part_dists  device, fp32, same layout: L2 distances or inner products as rago_search returns them
 *   out_ids     device, int64 [nq][k_out]; out_dists device, fp32 [nq][k_out]; short unions are padded with
 *               id -1 and +inf (L2) / -inf (IP); entries with equal scores keep the order (shard, rank)
 *   metric      RAGO_L2 or RAGO_IP, the metric of the shards' indexes
 *
 * ids are copied through unchanged: they should be unique across shards, which is the caller's
 * business.  1 <= k_out <= 1024, nparts * k_in < 2^31.  Needs no workspace, borrows every pointer, is
 * asynchronous on cuda_stream.  RAGO_EINVAL / RAGO_EUNSUPPORTED on bad sizes, nothing is launched then.
 */
rago_status rago_merge_results(const int64_t* part_ids, const float* part_dists, int32_t nparts,
                               int64_t part_stride, int32_t nq, int32_t k_in, int32_t k_out, int32_t metric,
                               int64_t* out_ids, float* out_dists, void* cuda_stream);

/* Per-stage device timings of rago_search.  When enabled, rago_search records CUDA events on the
 * caller's stream around each stage; rago_profile_read synchronises and returns the last call's
 * stage times in milliseconds (out_ms[RAGO_NUM_STAGES]). */
rago_status rago_profile_enable(rago_index* index, int32_t enable);
rago_status rago_profile_read(rago_index* index, float* out_ms);

/* Number of kernels the library has launched in this process since it was loaded. */
int64_t rago_kernel_launches(void);

/* Description of the calling thread's last error ("" if none).  Static storage. */
const char* rago_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RAGO_H */
