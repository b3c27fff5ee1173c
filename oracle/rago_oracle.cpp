// CPU oracle for the retrieval hot path: IVF-PQ search and exact flat search.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// search computes; only the tests, the smoke check and the benchmark's
// cpu_baseline / reference arm may build or call it.  It shares no code with
// the CUDA library and must never be reached from the product path.
//
// What it follows (RAGO paper, "Vector search for retrieval" in the Background
// section, and the retrieval-component paragraph of the RAGSchema section):
//   * vector search returns the K database vectors most similar to a
//     D-dimensional query under L2 distance or cosine / inner-product
//     similarity;
//   * IVF-PQ = an inverted file (a coarse clustering whose nearest `nprobe`
//     lists are visited) over product-quantised vectors (one byte per
//     sub-space, as in the PQ paper the RAGO paper cites);
//   * the retrieval work is the bytes of quantised vectors scanned;
//   * small databases are searched by brute force.
// IVF-PQ is an approximation, so the oracle is the algorithm step by step:
// coarse ranking, per-probe lookup tables, table-sum scan, top-k.  Flat search
// is the plain definition.  One thread works on one query; all sums are
// accumulated in double and rounded to float once.
//
// Readings taken where the paper is silent: squared L2; residual PQ (codes
// quantise vector - centroid) with one codebook set for all lists;
// inner-product score = <q, centroid> + sum of table entries; a bf16 coarse
// quantiser rounds the query to bf16 (nearest-even) for the coarse step only
// and the inner-product bias reuses that coarse value; ties go to the smaller
// list number / smaller id; missing results are id -1 with +inf (L2) or -inf
// (inner product).
//
// Two-level coarse quantiser (functions with "tree" in their name).  The paper
// indexes its database with a multi-level tree (Methodology, "Models and
// database": three levels, balanced fan-out) and models a search as scanning
// the levels top-down (Methodology, retrieval performance modelling: a sequence
// of scan operations, one per level).  With two levels above the vectors that
// is: score every level-1 centroid, keep the best b1 nodes, score the coarse
// centroids that are their children, keep the best nprobe of those as the
// probe lists; everything after that is unchanged.  Children of node i are the
// consecutive lists child_offsets[i] .. child_offsets[i+1]-1.  Pins: with
// b1 = all nodes the result equals the one-level search; a hand-worked
// example; a numpy restatement.
//
// Parity pins (tests/test_oracle_pins.py): hand-worked 2-D and 4-D examples,
// numpy brute force, decode-then-exact, lossless-PQ exhaustive search ==
// exact kNN, bf16 rounding against a library conversion.  Nothing here is
// "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <utility>
#include <vector>

namespace {

constexpr int KSUB = 256;
enum Metric { L2 = 0, IP = 1 };

// bfloat16 <-> float, round to nearest, ties to even (finite inputs).
inline uint16_t f32_to_bf16_bits(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return uint16_t((u >> 16) | 0x40);  // NaN stays NaN
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return uint16_t(u >> 16);
}
inline float bf16_bits_to_f32(uint16_t h) {
    uint32_t u = uint32_t(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

struct Index {
    const void* centroids;  // [nlist][d] float, or bf16 bits when coarse_bf16
    int coarse_bf16;
    const float* codebooks;  // [M][256][dsub]
    const uint8_t* codes;    // [N][M]
    const int64_t* offsets;  // [nlist+1]
    const int64_t* ids;      // [N]
    int64_t N;
    int d, nlist, M, metric;
    int dsub() const { return d / M; }
    double centroid(int l, int j) const {
        if (coarse_bf16) return double(bf16_bits_to_f32(static_cast<const uint16_t*>(centroids)[size_t(l) * d + j]));
        return double(static_cast<const float*>(centroids)[size_t(l) * d + j]);
    }
};

// "a is a better result than b" for (score, tie key); smaller tie key wins ties.
inline bool better(int metric, double sa, int64_t ta, double sb, int64_t tb) {
    if (sa != sb) return metric == L2 ? sa < sb : sa > sb;
    return ta < tb;
}

// Step 1: coarse score of every list for one query.
//   L2: sum_j (q_j - c_lj)^2       IP: sum_j q_j * c_lj
// With a bf16 coarse quantiser the query is first rounded to bf16.
void coarse_scores(const Index& ix, const float* q, std::vector<double>& s) {
    s.assign(ix.nlist, 0.0);
    std::vector<double> qq(ix.d);
    for (int j = 0; j < ix.d; ++j)
        qq[j] = ix.coarse_bf16 ? double(bf16_bits_to_f32(f32_to_bf16_bits(q[j]))) : double(q[j]);
    for (int l = 0; l < ix.nlist; ++l) {
        double acc = 0.0;
        for (int j = 0; j < ix.d; ++j) {
            double c = ix.centroid(l, j);
            if (ix.metric == L2) {
                double t = qq[j] - c;
                acc += t * t;
            } else {
                acc += qq[j] * c;
            }
        }
        s[l] = acc;
    }
}

void select_probes(const Index& ix, const std::vector<double>& s, int nprobe, std::vector<int>& probes) {
    std::vector<int> order(ix.nlist);
    for (int l = 0; l < ix.nlist; ++l) order[l] = l;
    std::sort(order.begin(), order.end(),
              [&](int a, int b) { return better(ix.metric, s[a], a, s[b], b); });
    probes.assign(order.begin(), order.begin() + nprobe);
}

// Step 2: lookup table of one (query, probed list).
//   L2: r = q - c_p;  T[m][j] = sum_t (r[m*dsub+t] - cb[m][j][t])^2
//   IP:               T[m][j] = sum_t  q[m*dsub+t] * cb[m][j][t]   (same for every list)
void build_table(const Index& ix, const float* q, int list, std::vector<double>& T) {
    const int ds = ix.dsub();
    T.assign(size_t(ix.M) * KSUB, 0.0);
    for (int m = 0; m < ix.M; ++m) {
        for (int j = 0; j < KSUB; ++j) {
            const float* cw = ix.codebooks + (size_t(m) * KSUB + j) * ds;
            double acc = 0.0;
            for (int t = 0; t < ds; ++t) {
                if (ix.metric == L2) {
                    // residual formed in float like the stored data would be, then widened
                    float r = q[m * ds + t] - float(ix.centroid(list, m * ds + t));
                    double e = double(r) - double(cw[t]);
                    acc += e * e;
                } else {
                    acc += double(q[m * ds + t]) * double(cw[t]);
                }
            }
            T[size_t(m) * KSUB + j] = acc;
        }
    }
}

struct Cand {
    double score;
    int64_t id;
};

// Steps 1-4 for one query.
struct Tree {
    const void* level1;         // [n1][d], same storage type as the coarse centroids
    const int32_t* child_offsets;  // [n1 + 1]
    int n1, b1;
};

// Probe lists through a two-level coarse quantiser: the best b1 level-1 nodes by the coarse score
// formula applied to the level-1 centroids, then the best nprobe of their children by the lists'
// own coarse scores cs (ties: smaller node / smaller list number).  Fewer than nprobe children
// among the chosen nodes leaves the tail of `probes` at -1.
void tree_probes(const Index& ix, const Tree& tr, const float* q, const std::vector<double>& cs, int nprobe,
                 std::vector<int>& probes) {
    Index top = ix;
    top.centroids = tr.level1;
    top.nlist = tr.n1;
    std::vector<double> s1;
    coarse_scores(top, q, s1);
    std::vector<int> nodes;
    select_probes(top, s1, tr.b1, nodes);
    std::vector<int> cand;
    for (int node : nodes)
        for (int l = tr.child_offsets[node]; l < tr.child_offsets[node + 1]; ++l) cand.push_back(l);
    std::sort(cand.begin(), cand.end(), [&](int a, int b) { return better(ix.metric, cs[a], a, cs[b], b); });
    probes.assign(nprobe, -1);
    for (int p = 0; p < nprobe && p < int(cand.size()); ++p) probes[p] = cand[p];
}

void search_one(const Index& ix, const float* q, int nprobe, int k, int64_t* out_ids, float* out_dists,
                int32_t* out_probes, const Tree* tree = nullptr) {
    std::vector<double> cs;
    coarse_scores(ix, q, cs);
    std::vector<int> probes;
    if (tree)
        tree_probes(ix, *tree, q, cs, nprobe, probes);
    else
        select_probes(ix, cs, nprobe, probes);
    std::vector<Cand> cands;
    std::vector<double> T;
    for (int p = 0; p < nprobe; ++p) {
        const int list = probes[p];
        if (out_probes) out_probes[p] = list;
        if (list < 0) continue;  // two-level quantiser with fewer than nprobe children among the chosen nodes
        if (ix.offsets[list + 1] == ix.offsets[list]) continue;
        build_table(ix, q, list, T);
        const double bias = ix.metric == IP ? cs[list] : 0.0;
        // Step 3: table-sum (asymmetric distance) of every vector of the list.
        for (int64_t i = ix.offsets[list]; i < ix.offsets[list + 1]; ++i) {
            double acc = 0.0;
            for (int m = 0; m < ix.M; ++m) acc += T[size_t(m) * KSUB + ix.codes[size_t(i) * ix.M + m]];
            cands.push_back({acc + bias, ix.ids[i]});
        }
    }
    // Step 4: k best of everything scanned.
    const size_t kk = std::min<size_t>(k, cands.size());
    std::partial_sort(cands.begin(), cands.begin() + kk, cands.end(), [&](const Cand& a, const Cand& b) {
        return better(ix.metric, a.score, a.id, b.score, b.id);
    });
    const float pad = ix.metric == L2 ? std::numeric_limits<float>::infinity()
                                      : -std::numeric_limits<float>::infinity();
    for (int t = 0; t < k; ++t) {
        out_ids[t] = size_t(t) < kk ? cands[t].id : -1;
        out_dists[t] = size_t(t) < kk ? float(cands[t].score) : pad;
    }
}

template <class F>
void parallel_for(int n, int nthreads, F f) {
    if (nthreads <= 1 || n <= 1) {
        for (int i = 0; i < n; ++i) f(i);
        return;
    }
    std::vector<std::thread> th;
    for (int t = 0; t < nthreads; ++t)
        th.emplace_back([=] {
            for (int i = t; i < n; i += nthreads) f(i);
        });
    for (auto& x : th) x.join();
}

Index make_index(const void* centroids, int coarse_bf16, const float* codebooks, const uint8_t* codes,
                 const int64_t* offsets, const int64_t* ids, int64_t N, int d, int nlist, int M, int metric) {
    return Index{centroids, coarse_bf16, codebooks, codes, offsets, ids, N, d, nlist, M, metric};
}

bool bad(int64_t N, int d, int nlist, int M, int metric) {
    return N < 0 || d <= 0 || nlist <= 0 || M <= 0 || d % M != 0 || (metric != L2 && metric != IP);
}

}  // namespace

extern "C" {

// Coarse step alone: best-first probe lists and their coarse scores (double).
int oracle_coarse(const void* centroids, int coarse_bf16, int d, int nlist, int metric, const float* queries, int nq,
                  int nprobe, int32_t* out_lists, double* out_scores, int nthreads) {
    if (d <= 0 || nlist <= 0 || nprobe <= 0 || nprobe > nlist) return 1;
    Index ix = make_index(centroids, coarse_bf16, nullptr, nullptr, nullptr, nullptr, 0, d, nlist, 1, metric);
    parallel_for(nq, nthreads, [&](int qi) {
        std::vector<double> cs;
        coarse_scores(ix, queries + size_t(qi) * d, cs);
        std::vector<int> probes;
        select_probes(ix, cs, nprobe, probes);
        for (int p = 0; p < nprobe; ++p) {
            out_lists[size_t(qi) * nprobe + p] = probes[p];
            out_scores[size_t(qi) * nprobe + p] = cs[probes[p]];
        }
    });
    return 0;
}

// Full IVF-PQ search.  out_probes may be null.
int oracle_ivfpq_search(const void* centroids, int coarse_bf16, const float* codebooks, const uint8_t* codes,
                        const int64_t* offsets, const int64_t* ids, int64_t N, int d, int nlist, int M, int metric,
                        const float* queries, int nq, int nprobe, int k, int64_t* out_ids, float* out_dists,
                        int32_t* out_probes, int nthreads) {
    if (bad(N, d, nlist, M, metric) || nprobe <= 0 || nprobe > nlist || k <= 0) return 1;
    Index ix = make_index(centroids, coarse_bf16, codebooks, codes, offsets, ids, N, d, nlist, M, metric);
    parallel_for(nq, nthreads, [&](int qi) {
        search_one(ix, queries + size_t(qi) * d, nprobe, k, out_ids + size_t(qi) * k, out_dists + size_t(qi) * k,
                   out_probes ? out_probes + size_t(qi) * nprobe : nullptr);
    });
    return 0;
}

// Coarse step through a two-level quantiser: best-first probe lists (-1 where the chosen nodes have too few
// children) and their coarse scores.
int oracle_coarse_tree(const void* centroids, int coarse_bf16, int d, int nlist, int metric, const void* level1,
                       const int32_t* child_offsets, int n1, int b1, const float* queries, int nq, int nprobe,
                       int32_t* out_lists, double* out_scores, int nthreads) {
    if (d <= 0 || nlist <= 0 || nprobe <= 0 || nprobe > nlist || n1 <= 0 || b1 <= 0 || b1 > n1) return 1;
    Index ix = make_index(centroids, coarse_bf16, nullptr, nullptr, nullptr, nullptr, 0, d, nlist, 1, metric);
    Tree tr{level1, child_offsets, n1, b1};
    parallel_for(nq, nthreads, [&](int qi) {
        std::vector<double> cs;
        coarse_scores(ix, queries + size_t(qi) * d, cs);
        std::vector<int> probes;
        tree_probes(ix, tr, queries + size_t(qi) * d, cs, nprobe, probes);
        for (int p = 0; p < nprobe; ++p) {
            out_lists[size_t(qi) * nprobe + p] = probes[p];
            out_scores[size_t(qi) * nprobe + p] = probes[p] >= 0 ? cs[probes[p]] : 0.0;
        }
    });
    return 0;
}

// Full IVF-PQ search whose probe lists come from the two-level quantiser.
int oracle_ivfpq_search_tree(const void* centroids, int coarse_bf16, const float* codebooks, const uint8_t* codes,
                             const int64_t* offsets, const int64_t* ids, int64_t N, int d, int nlist, int M, int metric,
                             const void* level1, const int32_t* child_offsets, int n1, int b1, const float* queries,
                             int nq, int nprobe, int k, int64_t* out_ids, float* out_dists, int32_t* out_probes,
                             int nthreads) {
    if (bad(N, d, nlist, M, metric) || nprobe <= 0 || nprobe > nlist || k <= 0 || n1 <= 0 || b1 <= 0 || b1 > n1) return 1;
    Index ix = make_index(centroids, coarse_bf16, codebooks, codes, offsets, ids, N, d, nlist, M, metric);
    Tree tr{level1, child_offsets, n1, b1};
    parallel_for(nq, nthreads, [&](int qi) {
        search_one(ix, queries + size_t(qi) * d, nprobe, k, out_ids + size_t(qi) * k, out_dists + size_t(qi) * k,
                   out_probes ? out_probes + size_t(qi) * nprobe : nullptr, &tr);
    });
    return 0;
}

// Table-sum score of the vector at storage position `pos` (inside list `list`) for one query.
int oracle_adc_score(const void* centroids, int coarse_bf16, const float* codebooks, const uint8_t* codes, int d,
                     int nlist, int M, int metric, const float* query, int list, int64_t pos, double* out) {
    if (bad(0, d, nlist, M, metric) || list < 0 || list >= nlist) return 1;
    Index ix = make_index(centroids, coarse_bf16, codebooks, codes, nullptr, nullptr, 0, d, nlist, M, metric);
    std::vector<double> T, cs;
    build_table(ix, query, list, T);
    double acc = 0.0;
    for (int m = 0; m < M; ++m) acc += T[size_t(m) * KSUB + codes[size_t(pos) * M + m]];
    if (metric == IP) {
        coarse_scores(ix, query, cs);
        acc += cs[list];
    }
    *out = acc;
    return 0;
}

// Second formulation: reconstruct y^ = c_list + concat_m cb[m][code_m], then score it directly
// (||q - y^||^2, or <q, y^> with the centroid part taken at coarse precision).
int oracle_decode_score(const void* centroids, int coarse_bf16, const float* codebooks, const uint8_t* codes, int d,
                        int nlist, int M, int metric, const float* query, int list, int64_t pos, double* out,
                        double* out_decoded /* [d] or null */) {
    if (bad(0, d, nlist, M, metric) || list < 0 || list >= nlist) return 1;
    Index ix = make_index(centroids, coarse_bf16, codebooks, codes, nullptr, nullptr, 0, d, nlist, M, metric);
    const int ds = ix.dsub();
    double acc = 0.0;
    for (int j = 0; j < d; ++j) {
        const int m = j / ds, t = j % ds;
        const double cw = double(codebooks[(size_t(m) * KSUB + codes[size_t(pos) * M + m]) * ds + t]);
        const double c = ix.centroid(list, j);
        if (out_decoded) out_decoded[j] = c + cw;
        if (metric == L2) {
            double e = double(query[j]) - (c + cw);  // no float residual here: plain ||q - y^||^2
            acc += e * e;
        } else {
            double qc = coarse_bf16 ? double(bf16_bits_to_f32(f32_to_bf16_bits(query[j]))) : double(query[j]);
            acc += qc * c + double(query[j]) * cw;
        }
    }
    *out = acc;
    return 0;
}

// Exact flat search: score = sum_j q_j * y_ij over bf16 inputs widened exactly; k largest.
int oracle_flat_search(const uint16_t* db, int64_t N, int d, const uint16_t* queries, int nq, int k, int64_t* out_ids,
                       float* out_scores, int nthreads) {
    if (N < 0 || d <= 0 || k <= 0) return 1;
    parallel_for(nq, nthreads, [&](int qi) {
        std::vector<double> q(d);
        for (int j = 0; j < d; ++j) q[j] = double(bf16_bits_to_f32(queries[size_t(qi) * d + j]));
        std::vector<Cand> c(static_cast<size_t>(N));
        for (int64_t i = 0; i < N; ++i) {
            double acc = 0.0;
            for (int j = 0; j < d; ++j) acc += q[j] * double(bf16_bits_to_f32(db[size_t(i) * d + j]));
            c[size_t(i)] = {acc, i};
        }
        const size_t kk = std::min<size_t>(k, c.size());
        std::partial_sort(c.begin(), c.begin() + kk, c.end(),
                          [](const Cand& a, const Cand& b) { return better(IP, a.score, a.id, b.score, b.id); });
        for (int t = 0; t < k; ++t) {
            out_ids[size_t(qi) * k + t] = size_t(t) < kk ? c[t].id : -1;
            out_scores[size_t(qi) * k + t] =
                size_t(t) < kk ? float(c[t].score) : -std::numeric_limits<float>::infinity();
        }
    });
    return 0;
}

// Score of chosen rows only (for sampled checks at full size).
int oracle_flat_scores(const uint16_t* db, int d, const uint16_t* query, const int64_t* rows, int nrows, double* out) {
    for (int r = 0; r < nrows; ++r) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j)
            acc += double(bf16_bits_to_f32(query[j])) * double(bf16_bits_to_f32(db[size_t(rows[r]) * d + j]));
        out[r] = acc;
    }
    return 0;
}

void oracle_f32_to_bf16(const float* in, uint16_t* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_bits(in[i]);
}

}  // extern "C"
