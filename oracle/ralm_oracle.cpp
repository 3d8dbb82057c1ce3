// CPU oracle for exact dense retrieval, speculation-cache lookup and verification.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, plain reference the CUDA library is
// checked against. It shares no code, header, table or helper with the CUDA path and
// must never be called from it. Only the tests, the smoke check and the benchmark's
// CPU-baseline leg may load it.
//
// What it computes (RaLMSpec, Algorithm 1 and Section 3):
//   * C.retrieve(q_1..q_s)  -- the batched verification retrieval with an exact dense
//     retriever: every query is scored against every corpus row and the k best rows are
//     returned (Algorithm 1, "batched verification" step; Section 3 "Batched
//     verification"; Section 5.1 "Retrievers": exact dense retriever).
//   * Q.retrieve(q_i)       -- the speculative retrieval from a request's local cache,
//     ranked with the same metric as the knowledge-base retriever (Algorithm 1,
//     "speculative retrieval" step; Section 3 "Speculative retrieval"; Fig. 3 caption).
//   * m = argmin_i d^_i != d_i -- the first mis-speculated position (Algorithm 1,
//     verification step; Section 3 toy example: A,B,A against A,B,C).
//
// The method returns exactly what sequential retrieval returns, so the oracle is the
// plain definition: widen fp16 to fp64 exactly, accumulate left to right in fp64, order
// all rows by a total order, truncate to k. No blocking, no fusion. Threads only split
// independent rows (each row's score is computed by one thread, start to finish).
//
// Total order (the paper is silent on ties): inner product -> (score descending, id
// ascending); L2 -> (squared distance ascending, id ascending).
//
// Parity pins for every function here live in tests/test_oracle_pins.py.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <numeric>
#include <thread>
#include <vector>

namespace {

constexpr int kMetricIP = 0;
constexpr int kMetricL2 = 1;

// IEEE 754 binary16 -> binary64, exact. 1 sign bit, 5 exponent bits (bias 15), 10
// mantissa bits. Exponent field 0: subnormal, value = m * 2^-24. Field 31: inf / NaN.
double half_to_double(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int e = (h >> 10) & 0x1f;
    const int m = h & 0x3ff;
    double v;
    if (e == 0) {
        v = std::ldexp(static_cast<double>(m), -24);
    } else if (e == 31) {
        v = (m == 0) ? std::numeric_limits<double>::infinity()
                     : std::numeric_limits<double>::quiet_NaN();
    } else {
        v = std::ldexp(static_cast<double>(1024 + m), e - 25);
    }
    return sign ? -v : v;
}

// Score of one (query, row) pair. IP: sum_t q[t]*x[t]. L2: sum_t (q[t]-x[t])^2.
// Left-to-right fp64 accumulation; every product / difference of two fp16 values is
// exact in fp64.
double pair_score(const uint16_t *x, const uint16_t *q, int d, int metric) {
    double acc = 0.0;
    if (metric == kMetricIP) {
        for (int t = 0; t < d; ++t) acc += half_to_double(q[t]) * half_to_double(x[t]);
    } else {
        for (int t = 0; t < d; ++t) {
            const double diff = half_to_double(q[t]) - half_to_double(x[t]);
            acc += diff * diff;
        }
    }
    return acc;
}

// true if (sa, ia) ranks strictly before (sb, ib).
bool ranks_before(double sa, int64_t ia, double sb, int64_t ib, int metric) {
    if (sa != sb) return (metric == kMetricIP) ? (sa > sb) : (sa < sb);
    return ia < ib;
}

double pad_score(int metric) {
    const double inf = std::numeric_limits<double>::infinity();
    return (metric == kMetricIP) ? -inf : inf;
}

int resolve_threads(int threads) {
    if (threads > 0) return threads;
    const unsigned hc = std::thread::hardware_concurrency();
    return hc ? static_cast<int>(hc) : 1;
}

}  // namespace

extern "C" {

double ralm_oracle_half_to_double(uint16_t h) { return half_to_double(h); }

double ralm_oracle_pair_score(const uint16_t *x, const uint16_t *q, int32_t d,
                              int32_t metric) {
    return pair_score(x, q, d, metric);
}

// out[j] = score(query, row j) for j in [0, n_rows). `threads` <= 0 means all cores.
// Returns the number of threads used.
int32_t ralm_oracle_scores(const uint16_t *rows, int64_t n_rows, int32_t d,
                           const uint16_t *query, int32_t metric, double *out,
                           int32_t threads) {
    const int T = static_cast<int>(
        std::max<int64_t>(1, std::min<int64_t>(resolve_threads(threads), n_rows)));
    auto work = [&](int64_t lo, int64_t hi) {
        for (int64_t j = lo; j < hi; ++j)
            out[j] = pair_score(rows + j * static_cast<int64_t>(d), query, d, metric);
    };
    if (T == 1) {
        work(0, n_rows);
        return 1;
    }
    std::vector<std::thread> pool;
    for (int i = 0; i < T; ++i) {
        const int64_t lo = n_rows * i / T, hi = n_rows * (i + 1) / T;
        pool.emplace_back(work, lo, hi);
    }
    for (auto &th : pool) th.join();
    return T;
}

// Rank all N rows by the total order on `scores`, write the first k (ids, scores), pad
// with (-1, -inf | +inf) when k > N.
void ralm_oracle_rank(const double *scores, int64_t N, int32_t metric, int32_t k,
                      int64_t *ids_out, double *scores_out) {
    std::vector<int64_t> order(static_cast<size_t>(N));
    std::iota(order.begin(), order.end(), int64_t{0});
    const int64_t keep = std::min<int64_t>(k, N);
    std::partial_sort(order.begin(), order.begin() + keep, order.end(),
                      [&](int64_t a, int64_t b) {
                          return ranks_before(scores[a], a, scores[b], b, metric);
                      });
    for (int64_t p = 0; p < k; ++p) {
        if (p < keep) {
            ids_out[p] = order[p];
            scores_out[p] = scores[order[p]];
        } else {
            ids_out[p] = -1;
            scores_out[p] = pad_score(metric);
        }
    }
}

// C.retrieve(q_1..q_s): ids [s][k], scores [s][k]. Returns threads used.
int32_t ralm_oracle_search(const uint16_t *corpus, int64_t N, int32_t d,
                           const uint16_t *queries, int32_t s, int32_t metric, int32_t k,
                           int64_t *ids, double *scores, int32_t threads) {
    std::vector<double> all(static_cast<size_t>(N));
    int32_t used = 1;
    for (int32_t i = 0; i < s; ++i) {
        if (N > 0)
            used = ralm_oracle_scores(corpus, N, d, queries + static_cast<int64_t>(i) * d,
                                      metric, all.data(), threads);
        ralm_oracle_rank(all.data(), N, metric, k, ids + static_cast<int64_t>(i) * k,
                         scores + static_cast<int64_t>(i) * k);
    }
    return used;
}

// Q.retrieve: for request r and its query u, the corpus ranking restricted to the set
// { cache_ids[r][c] : 0 <= cache_ids[r][c] < N }. -1 marks an empty slot; any other
// out-of-range value is ignored as well. The cache is a set: a repeated id counts once.
// cache_ids [R][C]; queries [R][q][d]; ids, scores [R][q][k].
void ralm_oracle_cache_search(const uint16_t *corpus, int64_t N, int32_t d, int32_t metric,
                              const int64_t *cache_ids, int32_t R, int32_t C,
                              const uint16_t *queries, int32_t q, int32_t k, int64_t *ids,
                              double *scores) {
    for (int32_t r = 0; r < R; ++r) {
        std::vector<int64_t> members;
        for (int32_t c = 0; c < C; ++c) {
            const int64_t j = cache_ids[static_cast<int64_t>(r) * C + c];
            if (j >= 0 && j < N) members.push_back(j);
        }
        std::sort(members.begin(), members.end());
        members.erase(std::unique(members.begin(), members.end()), members.end());
        for (int32_t u = 0; u < q; ++u) {
            const uint16_t *qv = queries + (static_cast<int64_t>(r) * q + u) * d;
            std::vector<std::pair<double, int64_t>> scored;
            for (int64_t j : members)
                scored.emplace_back(pair_score(corpus + j * d, qv, d, metric), j);
            std::sort(scored.begin(), scored.end(),
                      [&](const std::pair<double, int64_t> &a,
                          const std::pair<double, int64_t> &b) {
                          return ranks_before(a.first, a.second, b.first, b.second, metric);
                      });
            int64_t *io = ids + (static_cast<int64_t>(r) * q + u) * k;
            double *so = scores + (static_cast<int64_t>(r) * q + u) * k;
            for (int32_t p = 0; p < k; ++p) {
                if (p < static_cast<int32_t>(scored.size())) {
                    io[p] = scored[p].second;
                    so[p] = scored[p].first;
                } else {
                    io[p] = -1;
                    so[p] = pad_score(metric);
                }
            }
        }
    }
}

// first_mismatch[r] = smallest i in [0, stride) such that some c < cmp_k has
// speculated[r][i*cmp_k + c] != retrieved[r][i*ld + c]; `stride` when all steps match.
// 0-based: the algorithm's "m <= s" test (1-based m) becomes first_mismatch < stride.
void ralm_oracle_verify(const int64_t *speculated, const int64_t *retrieved, int32_t R,
                        int32_t stride, int32_t ld, int32_t cmp_k, int32_t *first_mismatch) {
    for (int32_t r = 0; r < R; ++r) {
        int32_t m = stride;
        for (int32_t i = 0; i < stride && m == stride; ++i) {
            for (int32_t c = 0; c < cmp_k; ++c) {
                const int64_t a = speculated[(static_cast<int64_t>(r) * stride + i) * cmp_k + c];
                const int64_t b = retrieved[(static_cast<int64_t>(r) * stride + i) * ld + c];
                if (a != b) {
                    m = i;
                    break;
                }
            }
        }
        first_mismatch[r] = m;
    }
}

}  // extern "C"
