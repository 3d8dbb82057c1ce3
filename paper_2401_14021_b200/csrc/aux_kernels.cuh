// Small kernels beside the scan: cross-CTA merge of partial top-k lists, the per-request
// speculation-cache lookup (score + rank) and the first-mismatch verification.
#pragma once

#include "common.cuh"

namespace ralm {

constexpr int kMergeThreads = 1024;
constexpr int kMergeSortMax = 4096;  // keys sorted in one go when all lists fit
constexpr int kMergeSelectMaxK = 32;  // up to this k, and from kMergeSelectMin keys on, the merge
constexpr int kMergeSelectMin = 256;  // selects the k largest keys one by one instead of sorting

// Largest 64-bit key of the warp, in every lane (two 32-bit warp reductions).
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
    const uint32_t hi = static_cast<uint32_t>(v >> 32);
    const uint32_t top = __reduce_max_sync(0xffffffffu, hi);
    const uint32_t lo = __reduce_max_sync(0xffffffffu, hi == top ? static_cast<uint32_t>(v) : 0u);
    return (static_cast<uint64_t>(top) << 32) | lo;
}

__device__ __forceinline__ void write_result(uint64_t key, bool l2, int64_t *id_out,
                                             float *score_out) {
    if (key == 0ull) {
        *id_out = -1;
        *score_out = l2 ? INFINITY : -INFINITY;
    } else {
        *id_out = static_cast<int64_t>(key_row(key));
        const float v = key_value(key);
        *score_out = l2 ? (0.0f - v) : v;
    }
}

// ------------------------------------------------------------------------------------
// Threshold from the maxima of a sample launch: one CTA per query. vals holds G values for the
// query (vals[g * stride + query], -inf = the group saw no row), each the best rank value of a
// different, disjoint group of rows, so the k-th largest of them is reached by k different rows.
// Writes it to thr_out[query], or -inf when fewer than k groups saw a row. G <= kMaximaSortMax.
// ------------------------------------------------------------------------------------
constexpr int kMaximaSortMax = 8192;
__global__ void __launch_bounds__(kMergeThreads, 1)
kth_of_maxima_kernel(const float *__restrict__ vals, int G, int stride, int k, float *__restrict__ thr_out) {
    __shared__ uint32_t buf[kMaximaSortMax];   // order-preserving bits; 0 = no row
    const int q = blockIdx.x;
    const int tid = threadIdx.x;
    const int P = next_pow2(G > 1 ? G : 2);
    for (int i = tid; i < P; i += kMergeThreads) {
        uint32_t bits = 0;
        if (i < G) {
            const float v = vals[static_cast<size_t>(i) * stride + q];
            if (v != -INFINITY) bits = ordered_bits(v + 0.0f);
        }
        buf[i] = bits;
    }
    __syncthreads();
    bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
    if (tid == 0) thr_out[q] = (k <= G && buf[k - 1] != 0u) ? from_ordered_bits(buf[k - 1]) : -INFINITY;
}

// ------------------------------------------------------------------------------------
// Merge: one CTA per query (and, with gridDim.y > 1, per group of lists). `partial` holds B lists
// of k keys, each sorted descending and padded with 0, laid out [B][s][k]. Writes ids [s][k]
// (int64) and scores [s][k] (fp32).
// ------------------------------------------------------------------------------------
// extra_slot >= 0: one more list takes part, stored at that block index of `partial`.
// With keys_out the merged list is written as keys instead, at keys_out[(blockIdx.y * s + q) * k]
// (and, with thr_out, the k-th value, or -inf when there are fewer than k rows, to thr_out[q]):
// the result of scanning a sample of the corpus, which seeds the thresholds of the main scan and
// rejoins the final merge as one more partial list; or the first level of a two-level merge,
// where CTA (q, y) merges the y-th of gridDim.y equal groups of the lists (few queries and long
// lists leave a single level with a handful of CTAs that each walk through every list).
__global__ void __launch_bounds__(kMergeThreads, 1)
merge_kernel(const uint64_t *__restrict__ partial, int B, int s, int k, int l2,
             int64_t *__restrict__ ids, float *__restrict__ scores, uint64_t *__restrict__ keys_out = nullptr,
             float *__restrict__ thr_out = nullptr, int extra_slot = -1) {
    __shared__ uint64_t buf[kMergeSortMax];
    __shared__ uint64_t warp_best[2][32];
    __shared__ int kept;
    const int q = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int all_lists = B + (extra_slot >= 0 ? 1 : 0);
    const int per_group = (all_lists + gridDim.y - 1) / gridDim.y;
    const int first = blockIdx.y * per_group;
    const int lists = max(min(all_lists - first, per_group), 0);
    auto list_at = [&](int b) -> const uint64_t * {   // the b-th list of this CTA's group, query q
        b += first;
        return partial + (static_cast<size_t>(b < B ? b : extra_slot) * s + q) * k;
    };
    const long long total = static_cast<long long>(lists) * k;
    if (total <= kMergeSortMax && total > kMergeSelectMin && k <= kMergeSelectMaxK) {
        // Many short lists (148 lists of 20 keys): k rounds of "take the largest key left" over
        // keys held in registers cost a fraction of sorting all of them (a 4096-key bitonic
        // sort is 78 passes with a barrier each). Keys are distinct: a row is in one list only.
        uint64_t mine[kMergeSortMax / kMergeThreads];
#pragma unroll
        for (int j = 0; j < kMergeSortMax / kMergeThreads; ++j) {
            const int i = tid + j * kMergeThreads;
            mine[j] = 0;
            if (i < total) {
                const int b = i / k;
                mine[j] = list_at(b)[i - b * k];
            }
        }
        for (int r = 0; r < k; ++r) {
            uint64_t m = mine[0];
#pragma unroll
            for (int j = 1; j < kMergeSortMax / kMergeThreads; ++j) m = mine[j] > m ? mine[j] : m;
            m = warp_max_u64(m);
            if (lane == 0) warp_best[r & 1][warp] = m;
            __syncthreads();   // (two buffers: a warp is at most one round ahead of another)
            const uint64_t winner = warp_max_u64(warp_best[r & 1][lane]);
#pragma unroll
            for (int j = 0; j < kMergeSortMax / kMergeThreads; ++j)
                if (mine[j] == winner) mine[j] = 0;
            if (tid == 0) buf[r] = winner;
        }
        __syncthreads();
    } else if (total <= kMergeSortMax) {
        const int P = next_pow2(total > 1 ? static_cast<int>(total) : 2);
        for (int i = tid; i < P; i += kMergeThreads) {
            uint64_t key = 0;
            if (i < total) {
                const int b = i / k, j = i - b * k;
                key = list_at(b)[j];
            }
            buf[i] = key;
        }
        __syncthreads();
        bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
    } else {
        // Long lists. If m lists each hold r keys from some value up, m * r >= k keys reach that
        // value and nothing below it can be among the best k of all. So: take every list's r-th
        // key, r = ceil(2k / lists); the m-th largest of them, m = ceil(k / r), is such a value
        // (the cut). Rows are dealt to the CTAs in turn, so about 2k keys lie above it: those are
        // kept and sorted at once. Where fewer than m lists hold r keys the cut is 0 and every key
        // is kept (a scan that started from good thresholds leaves each CTA with a few keys).
        const int r = min(k, max(1, (2 * k + lists - 1) / lists));
        const int m = (k + r - 1) / r;
        uint64_t cut = 0ull;
        if (lists <= kMergeSortMax) {
            const int P = next_pow2(lists > 1 ? lists : 2);
            for (int b = tid; b < P; b += kMergeThreads) buf[b] = (b < lists) ? list_at(b)[r - 1] : 0ull;
            __syncthreads();
            bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
            cut = (m <= lists) ? buf[m - 1] : 0ull;
        }
        if (tid == 0) kept = 0;
        __syncthreads();
        bool sorted = false;
        {
            for (int b = warp; b < lists; b += kMergeThreads / 32) {
                const uint64_t *list = list_at(b);
                for (int j0 = 0; j0 < k; j0 += 32) {   // descending: the first key below the cut ends the list
                    const uint64_t key = (j0 + lane < k) ? list[j0 + lane] : 0ull;
                    if (key >= cut && key != 0ull) {
                        const int at = atomicAdd(&kept, 1);
                        if (at < kMergeSortMax) buf[at] = key;
                    }
                    if (__any_sync(0xffffffffu, key < cut || key == 0ull)) break;
                }
            }
            __syncthreads();
            const int n = kept;
            if (n <= kMergeSortMax) {
                const int P = next_pow2(n > k ? n : (k > 1 ? k : 2));   // (the first k slots are read below)
                for (int i = n + tid; i < P; i += kMergeThreads) buf[i] = 0ull;
                __syncthreads();
                bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
                sorted = true;
            }
            __syncthreads();
        }
        if (!sorted) {
            // running best list merged with one sorted list at a time: the element-wise maximum
            // of a descending list and a reversed descending list holds the best P keys of both
            // and is bitonic
            const int P = next_pow2(k);
            const uint64_t *list0 = list_at(0);
            for (int i = tid; i < P; i += kMergeThreads) buf[i] = (i < k) ? list0[i] : 0ull;
            __syncthreads();
            for (int b = 1; b < lists; ++b) {
                const uint64_t *list = list_at(b);
                for (int i = tid; i < P; i += kMergeThreads) {
                    const int j = P - 1 - i;
                    const uint64_t other = (j < k) ? list[j] : 0ull;
                    const uint64_t mine = buf[i];
                    buf[i] = mine > other ? mine : other;
                }
                __syncthreads();
                bitonic_merge_desc(buf, P, tid, kMergeThreads, -1);
            }
        }
    }
    for (int i = tid; i < k; i += kMergeThreads) {
        const uint64_t key = (i < total) ? buf[i] : 0ull;
        if (keys_out) {
            keys_out[(static_cast<size_t>(blockIdx.y) * s + q) * k + i] = key;
            if (thr_out && i == k - 1) thr_out[q] = key ? key_value(key) : -INFINITY;
        } else {
            write_result(key, l2 != 0, ids + static_cast<size_t>(q) * k + i,
                         scores + static_cast<size_t>(q) * k + i);
        }
    }
}

// ------------------------------------------------------------------------------------
// Merge of G result lists of a row-sharded search: shard g searched its own rows and reports,
// per query, k (id, score) pairs sorted by the ranking order, ids local to the shard (-1 =
// padding); row_offset[g] is the global id of the shard's first row. One CTA per query turns
// the pairs back into ranking keys with global ids and merges them exactly like merge_kernel.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMergeThreads, 1)
merge_lists_kernel(const int64_t *__restrict__ ids, const float *__restrict__ scores,
                   const int64_t *__restrict__ row_offset, int G, int s, int k, int l2,
                   int64_t *__restrict__ out_ids, float *__restrict__ out_scores) {
    __shared__ uint64_t buf[kMergeSortMax];
    const int q = blockIdx.x;
    const int tid = threadIdx.x;
    auto load = [&](int g, int j) -> uint64_t {
        const size_t at = (static_cast<size_t>(g) * s + q) * k + j;
        const int64_t id = ids[at];
        if (id < 0) return 0ull;
        const float v = l2 ? (0.0f - scores[at]) : scores[at];
        return make_key(v, static_cast<uint32_t>(id + row_offset[g]));
    };
    const long long total = static_cast<long long>(G) * k;
    if (total <= kMergeSortMax) {
        const int P = next_pow2(total > 1 ? static_cast<int>(total) : 2);
        for (int i = tid; i < P; i += kMergeThreads) buf[i] = (i < total) ? load(i / k, i % k) : 0ull;
        __syncthreads();
        bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
    } else {
        const int P = next_pow2(k);
        for (int i = tid; i < P; i += kMergeThreads) buf[i] = (i < k) ? load(0, i) : 0ull;
        __syncthreads();
        for (int g = 1; g < G; ++g) {
            for (int i = tid; i < P; i += kMergeThreads) {
                const int j = P - 1 - i;
                const uint64_t other = (j < k) ? load(g, j) : 0ull;
                const uint64_t mine = buf[i];
                buf[i] = mine > other ? mine : other;
            }
            __syncthreads();
            bitonic_merge_desc(buf, P, tid, kMergeThreads, -1);
        }
    }
    for (int i = tid; i < k; i += kMergeThreads)
        write_result((i < total) ? buf[i] : 0ull, l2 != 0, out_ids + static_cast<size_t>(q) * k + i,
                     out_scores + static_cast<size_t>(q) * k + i);
}

// ------------------------------------------------------------------------------------
// Cache lookup, step 1: score. One warp per (request, cache slot); the warp scores its
// cached corpus row against up to 8 of the request's queries at a time and stores one key
// per query in keys[r][u][c] (Cp = C rounded up to a power of two; slots >= C hold 0).
// grid = (R, ceil(Cp / slots_per_cta)), block = 256 (the request index in x: y stops at 65535).
// ------------------------------------------------------------------------------------
constexpr int kCacheThreads = 256;
constexpr int kCacheSlotsPerCta = 32;

__global__ void __launch_bounds__(kCacheThreads)
cache_score_kernel(const __half *__restrict__ corpus, long long N, int d, int l2,
                   const int64_t *__restrict__ cache_ids, int C, int Cp,
                   const __half *__restrict__ queries, int q, uint64_t *__restrict__ keys,
                   int *status) {
    const int r = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pieces = d >> 3;
    for (int c = blockIdx.y * kCacheSlotsPerCta + warp; c < (blockIdx.y + 1) * kCacheSlotsPerCta && c < Cp;
         c += kCacheThreads / 32) {
        long long id = -1;
        if (c < C) id = cache_ids[static_cast<size_t>(r) * C + c];
        const bool valid = id >= 0 && id < N;
        if (c < C && !valid && id != -1 && lane == 0) atomicMax(status, kStatusBadCacheId);
        const __half *row = corpus + (valid ? id : 0) * d;
        for (int u0 = 0; u0 < q; u0 += 8) {
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
            if (valid) {
                for (int pc = lane; pc < pieces; pc += 32) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(row + pc * 8);
                    const uint32_t xw[4] = {raw.x, raw.y, raw.z, raw.w};
                    float2 x[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        x[e] = __half22float2(*reinterpret_cast<const __half2 *>(&xw[e]));
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (u0 + j < q) {
                            const uint4 qr = *reinterpret_cast<const uint4 *>(
                                queries + (static_cast<size_t>(r) * q + u0 + j) * d + pc * 8);
                            const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 qv =
                                    __half22float2(*reinterpret_cast<const __half2 *>(&qw[e]));
                                if (l2) {
                                    const float dx = x[e].x - qv.x, dy = x[e].y - qv.y;
                                    acc[j] = fmaf(dx, dx, acc[j]);
                                    acc[j] = fmaf(dy, dy, acc[j]);
                                } else {
                                    acc[j] = fmaf(x[e].x, qv.x, acc[j]);
                                    acc[j] = fmaf(x[e].y, qv.y, acc[j]);
                                }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
            }
            if (lane < 8 && u0 + lane < q) {
                float v = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (j == lane) v = acc[j];
                if (l2) v = 0.0f - v;
                keys[(static_cast<size_t>(r) * q + u0 + lane) * Cp + c] =
                    valid ? make_key(v, static_cast<uint32_t>(id)) : 0ull;
            }
        }
    }
}

// Cache lookup, step 2: rank. One CTA per (request, query): sort the Cp keys, drop repeated
// ids (equal keys are adjacent after the sort), write the best k.
__global__ void __launch_bounds__(kMergeThreads, 1)
cache_rank_kernel(const uint64_t *__restrict__ keys, int Cp, int k, int l2,
                  int64_t *__restrict__ ids, float *__restrict__ scores) {
    __shared__ uint64_t buf[kMergeSortMax];
    __shared__ int warp_total[kMergeSortMax / 32];
    const int tid = threadIdx.x;
    const size_t ru = blockIdx.x;
    const int P = Cp < 2 ? 2 : Cp;
    for (int i = tid; i < P; i += kMergeThreads) buf[i] = (i < Cp) ? keys[ru * Cp + i] : 0ull;
    __syncthreads();
    bitonic_sort_desc(buf, P, tid, kMergeThreads, -1);
    // keep[i]: a real key that differs from its predecessor
    const int lane = tid & 31;
    const int chunks = (P + 31) / 32;  // 32-element chunks, one per warp iteration
    for (int ch = tid >> 5; ch < chunks; ch += kMergeThreads / 32) {
        const int i = ch * 32 + lane;
        const bool keep = i < P && buf[i] != 0ull && (i == 0 || buf[i] != buf[i - 1]);
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_total[ch] = __popc(m);
    }
    __syncthreads();
    for (int i = tid; i < k; i += kMergeThreads) {
        ids[ru * k + i] = -1;
        scores[ru * k + i] = l2 ? INFINITY : -INFINITY;
    }
    __syncthreads();
    for (int ch = tid >> 5; ch < chunks; ch += kMergeThreads / 32) {
        const int i = ch * 32 + lane;
        const bool keep = i < P && buf[i] != 0ull && (i == 0 || buf[i] != buf[i - 1]);
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        int base = 0;
        for (int c2 = 0; c2 < ch; ++c2) base += warp_total[c2];
        const int rank = base + __popc(m & ((1u << lane) - 1u));
        if (keep && rank < k) write_result(buf[i], l2 != 0, ids + ru * k + rank, scores + ru * k + rank);
    }
}

// ------------------------------------------------------------------------------------
// Cache update after a verification step: one CTA per request. The request's slots sit in
// shared memory; candidates are taken strictly in order (step, rank, offset), each tested
// against all slots by the whole CTA and, if absent, written at the request's ring cursor.
// The order is part of the result (what a full ring evicts depends on it), so the loop over
// candidates is sequential and only the membership test is parallel.
// ------------------------------------------------------------------------------------
constexpr int kCacheUpdateThreads = 256;

__global__ void __launch_bounds__(kCacheUpdateThreads)
cache_update_kernel(int64_t *__restrict__ cache_ids, int *__restrict__ cursor, int C,
                    const int64_t *__restrict__ retrieved, int stride, int ld, int top,
                    const int *__restrict__ steps, int next_n, long long N) {
    extern __shared__ __align__(16) unsigned char cu_smem[];
    int64_t *slots = reinterpret_cast<int64_t *>(cu_smem);
    const int r = blockIdx.x;
    const int tid = threadIdx.x;
    int64_t *mine = cache_ids + static_cast<size_t>(r) * C;
    for (int i = tid; i < C; i += kCacheUpdateThreads) slots[i] = mine[i];
    int cur = cursor[r] % C;
    if (cur < 0) cur += C;
    int n_steps = steps ? steps[r] : stride;
    n_steps = n_steps < 0 ? 0 : (n_steps > stride ? stride : n_steps);
    __syncthreads();
    const int first = next_n > 0 ? 1 : 0, last = next_n > 0 ? next_n : 0;
    for (int i = 0; i < n_steps; ++i) {
        for (int j = 0; j < top; ++j) {
            const long long doc = retrieved[(static_cast<size_t>(r) * stride + i) * ld + j];
            if (doc < 0) continue;
            for (int o = first; o <= last; ++o) {
                const long long c = doc + o;
                if (c >= N) break;
                int found = 0;
                for (int sidx = tid; sidx < C; sidx += kCacheUpdateThreads) found |= (slots[sidx] == c);
                if (!__syncthreads_or(found)) {
                    if (tid == 0) slots[cur] = c;
                    cur = (cur + 1 == C) ? 0 : cur + 1;
                    __syncthreads();
                }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < C; i += kCacheUpdateThreads) mine[i] = slots[i];
    if (tid == 0) cursor[r] = cur;
}

// ------------------------------------------------------------------------------------
// Self-test of the bounded waits: a wait on a barrier that nothing ever completes must give up
// after `limit_cycles`, record the time-out in the status word and return normally.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(long long limit_cycles, int *status) {
    __shared__ uint64_t never;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (threadIdx.x == 0 && !mbar_wait_bounded_for(smem_u32(&never), 0, limit_cycles))
        atomicMax(status, kStatusTimeout);
}

// ------------------------------------------------------------------------------------
// Squared norms of the corpus rows (L2 indexes, once at creation): one warp per row, fp32.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
row_norm_kernel(const __half *__restrict__ corpus, long long N, int d, float *__restrict__ norms) {
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long row = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); row < N;
         row += warps) {
        const uint4 *src = reinterpret_cast<const uint4 *>(corpus + row * d);
        float2 sum = make_float2(0.f, 0.f);
        for (int piece = lane; piece * 8 < d; piece += 32) {
            const uint4 raw = __ldg(src + piece);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&w[e]));
                sum.x = fmaf(x.x, x.x, sum.x);
                sum.y = fmaf(x.y, x.y, sum.y);
            }
        }
        float v = sum.x + sum.y;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) norms[row] = v;
    }
}

// ------------------------------------------------------------------------------------
// Verification: one warp per request; lanes take speculation steps 32 at a time.
// ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
verify_kernel(const int64_t *__restrict__ spec, const int64_t *__restrict__ retr, int R, int stride,
              int ld, int cmp_k, int *__restrict__ first_mismatch) {
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= R) return;
    int m = stride;
    for (int base = 0; base < stride && m == stride; base += 32) {
        const int i = base + lane;
        bool differ = false;
        if (i < stride) {
            const int64_t *a = spec + (static_cast<size_t>(r) * stride + i) * cmp_k;
            const int64_t *b = retr + (static_cast<size_t>(r) * stride + i) * ld;
            for (int c = 0; c < cmp_k; ++c) differ |= (a[c] != b[c]);
        }
        const unsigned mask = __ballot_sync(0xffffffffu, differ);
        if (mask) m = base + __ffs(mask) - 1;
    }
    if (lane == 0) first_mismatch[r] = m;
}

}  // namespace ralm
