// Corpus scan for large query batches (up to 512 queries per pass; inner product, and L2 through
// the same inner-product tiles, see TcParams::mode) on the
// fifth-generation tensor cores: scores = corpus tile [128 rows] x queries^T [up to 256] with
// tcgen05.mma, fp16 operands, fp32 accumulators in tensor memory (TMEM), fused with the
// per-CTA top-k selection so that the N x s score matrix never exists in memory.
//
// One persistent CTA per SM, 6 warps:
//   warp 0      producer: one thread issues the TMA tile loads. A stage holds one K chunk
//               (64 fp16 = 128 bytes per row, the 128-byte swizzle span) of 128 corpus rows
//               and of up to 256 queries; stages form a ring guarded by full/empty mbarriers.
//   warp 1      MMA: one thread issues tcgen05.mma (M = 128, N = 16..256, K = 16 per
//               instruction, 4 per chunk). A work unit is (row tile, half of the queries);
//               the two halves of TMEM (256 columns each) alternate between units, so one
//               accumulator is drained while the next is being filled.
//   warps 2..5  selection: each warp owns one quarter of the TMEM lanes (32 corpus rows),
//               reads the scores with tcgen05.ld, compares each with its query's threshold
//               (the CTA's current k-th best, or a better bound handed in by the caller) and
//               appends what passes to that query's candidate list in global memory. Lists are
//               compacted (sorted in registers, cut to k, threshold raised) by the same warps
//               between units, before they can overflow.
//
// A launch covers the row tiles [tile0, tile0 + ntiles) and may start from given thresholds:
// the host scans a small sample of the corpus first, merges it, and starts the main launch
// from the sample's k-th scores, which makes appends rare (the selection would otherwise, at
// hundreds of queries, cost more than the MMAs).
//
// The kernel is bound by the bytes it stages per MMA, so by default it runs as clusters of two
// CTAs (cta_group::2): a row tile is then 256 rows, each CTA stages its own 128 rows but only
// half of the queries of a chunk, the pair's leader issues one M = 256 MMA for both, and each
// CTA selects from the 128 rows that land in its own TMEM. No load is multicast.
//
// Every wait is bounded; when one runs out the CTA records kStatusTimeout, lets copies and
// MMAs in flight finish, frees its TMEM and returns (a pair leaves through a cluster barrier).
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace ralm {

constexpr int kTcThreads = 192;
constexpr int kTcTileM = 128;    // corpus rows per tile = TMEM lanes
constexpr int kTcMaxN = 256;     // queries per accumulator = TMEM columns per half
constexpr int kTcChunkK = 64;    // fp16 per K chunk (128 bytes: one swizzle span)
constexpr int kTcMaxQueries = 2 * kTcMaxN;
constexpr int kTcABytes = kTcTileM * kTcChunkK * 2;
constexpr int kTcMaxStages = 12;
constexpr int kTcCap = 256;      // candidate slots per (CTA, query)
constexpr int kTcSoft = 120;     // a list holding this many is compacted before the next unit (at most
                                 // 128 more arrive in a unit; just under 128 so that the usual sort is
                                 // one of 128 keys)
constexpr int kTcMaxK = 64;      // k <= about kTcSoft / 2 keeps compactions rare
constexpr int kTcTmemCols = 512;

struct TcParams {
    uint64_t *partial;  // [gridDim.x][s_total][k] sorted keys, 0 = empty
    uint64_t *cand;     // [gridDim.x][cand_q][kTcCap] candidate lists
    int *status;
    long long N;        // rows of this launch end here (the whole corpus, or the end of a sample)
    long long tile0;    // first row tile (of 128 rows, 256 for pairs) of this launch
    const float *thr_init;  // [s_total] starting thresholds (scores that k rows are known to reach), or null
    long long ntiles;   // row tiles of this launch
    int nchunks;        // ceil(d / 64)
    int s;              // queries in this pass (<= 512)
    int s_total;
    int q_base;
    int k;
    int nb;             // queries per accumulator (16..256; a multiple of 16, of 32 for CTA pairs);
                        // a CTA stages nb query rows per chunk, nb / 2 in a pair
    int nhalves;        // ceil(s / nb): 1 or 2
    int stages;
    int stage_bytes;    // kTcABytes + (staged query rows) * 128, a multiple of 1024
    int off_stage;      // shared-memory offset of the stage ring (1024-byte aligned)
    int cand_q;         // queries the candidate workspace was sized for (>= s)
    // L2 (squared distance) on the same inner-product tiles. mode 0: inner product. The tensor-
    // core value v = 2 x.q - |x|^2 - |q|^2 = -distance^2 cancels, so it is never ranked:
    // mode 1 (sample launch): keys are the LOWER BOUNDS v - slack (|x|^2 + |q|^2); their merged
    //         k-th value is a rank value that k rows are known to reach;
    // mode 2 (main launch, over all rows): a pair passes the filter when v + slack (|x|^2 + |q|^2)
    //         reaches the threshold, and is then scored again in the direct sum-of-squared-
    //         differences form from global memory; only that value is ranked and returned.
    int mode;
    int d;
    float slack;
    const float *norms;      // |x|^2 of every corpus row (fp32)
    const __half *corpus;    // the rows and queries themselves, for the direct form
    const __half *queries;   // [s][d] of this pass
};

struct TcHeader {
    uint64_t full[kTcMaxStages];
    uint64_t empty[kTcMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort;
    int dirty[3];  // [u % 3]: some candidate list reached kTcSoft during unit u
};
constexpr int kTcHeaderBytes = 512;
static_assert(sizeof(TcHeader) <= kTcHeaderBytes, "header too large");
// shared-memory layout after the header
constexpr int kTcOffThr = kTcHeaderBytes;                      // float [512]
constexpr int kTcOffCnt = kTcOffThr + kTcMaxQueries * 4;       // int [512]
constexpr int kTcOffSorted = kTcOffCnt + kTcMaxQueries * 4;    // int [512]
constexpr int kTcOffQn = kTcOffSorted + kTcMaxQueries * 4;      // float [512]: |q|^2 (L2)
constexpr int kTcOffEnd = kTcOffQn + kTcMaxQueries * 4;

// ---- tcgen05 / TMA wrappers -------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, fp16 x fp16 -> fp32
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                           uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Shared-memory operand descriptor: K-major tile, 128-byte swizzle, rows 128 bytes apart,
// groups of 8 rows 1024 bytes apart; `addr` may be advanced by 32 bytes per K step of 16.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
    uint64_t desc = (addr & 0x3FFFFu) >> 4;         // start address, 16-byte units
    desc |= static_cast<uint64_t>(1) << 16;         // leading byte offset (unused with swizzle)
    desc |= static_cast<uint64_t>(1024 >> 4) << 32; // stride byte offset: next group of 8 rows
    desc |= static_cast<uint64_t>(1) << 46;         // descriptor version of this architecture
    desc |= static_cast<uint64_t>(2) << 61;         // 128-byte swizzle
    return desc;
}
// Instruction descriptor: fp16 A and B (both K-major), fp32 accumulator, M = m, N = n.
__device__ __forceinline__ uint32_t tc_idesc(int n, int m) {
    return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}
// 32 consecutive columns of this thread's TMEM lane, then wait for the load.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
          "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// Bitonic sort (descending) of 32 * E keys held by one warp in registers: key i lives in
// x[i / 32] of lane i % 32. Exchanges at distance >= 32 stay inside a lane, the others are
// shuffles; nothing touches memory.
template <int E>
__device__ __forceinline__ void warp_sort_desc(uint64_t (&x)[E], int lane) {
#pragma unroll
    for (int size = 2; size <= 32 * E; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride >= 32) {
                const int es = stride >> 5;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if ((e & es) == 0) {
                        const bool desc = ((e << 5) & size) == 0;
                        const uint64_t a = x[e], b = x[e | es];
                        const bool swap = desc ? (a < b) : (a > b);
                        x[e] = swap ? b : a;
                        x[e | es] = swap ? a : b;
                    }
                }
            } else {
                const bool lower = (lane & stride) == 0;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const bool desc = (((e << 5) | lane) & size) == 0;
                    const uint64_t other = __shfl_xor_sync(0xffffffffu, x[e], stride);
                    const bool keep_max = lower == desc;
                    const bool mine_larger = x[e] > other;
                    x[e] = (keep_max == mine_larger) ? x[e] : other;
                }
            }
        }
    }
}

// One selection warp sorts query q's candidate list (n <= 32 * E keys in global memory), keeps
// the best k there, raises the threshold.
template <int E>
__device__ __forceinline__ void tc_compact_sorted(uint64_t *list, float *thr, int *cnt, int *sorted, int q,
                                                  int n, int k, int lane) {
    uint64_t x[E];
#pragma unroll
    for (int e = 0; e < E; ++e) x[e] = (e * 32 + lane < n) ? list[e * 32 + lane] : 0ull;
    warp_sort_desc<E>(x, lane);
    const int keep = n < k ? n : k;
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (e * 32 + lane < keep) list[e * 32 + lane] = x[e];
    // the k-th best key sits in x[(k - 1) / 32] of lane (k - 1) % 32
    uint64_t kth = 0;
#pragma unroll
    for (int e = 0; e < E; ++e)
        if (e == ((k - 1) >> 5)) kth = x[e];
    kth = __shfl_sync(0xffffffffu, kth, (k - 1) & 31);
    if (lane == 0) {
        cnt[q] = keep;
        sorted[q] = keep;
        thr[q] = (n >= k) ? key_value(kth) : -INFINITY;
    }
    __syncwarp();
}

__device__ __forceinline__ void tc_compact_query(uint64_t *list, float *thr, int *cnt, int *sorted, int q,
                                                 int k, int lane) {
    const int n = cnt[q];
    if (n <= 32) tc_compact_sorted<1>(list, thr, cnt, sorted, q, n, k, lane);
    else if (n <= 64) tc_compact_sorted<2>(list, thr, cnt, sorted, q, n, k, lane);
    else if (n <= 128) tc_compact_sorted<4>(list, thr, cnt, sorted, q, n, k, lane);
    else tc_compact_sorted<8>(list, thr, cnt, sorted, q, n, k, lane);
}

// The rare part of the selection: some score of this warp's 32 rows x 32 columns passes its
// threshold. Out of line, and re-reading the scores from TMEM, so that the common path (no score
// passes) stays a short loop with few live registers. The warp appends as a whole: lane L
// learns which rows pass column L (one ballot per column that has any), reserves that many
// slots of query L's list with ONE atomic instruction (32 different lists), and every passing
// row then stores its key at its rank within the reservation.
__device__ __noinline__ void tc_append_chunk(uint32_t taddr, const float *thr_chunk, int *cnt_chunk,
                                             uint64_t *cand_chunk, uint32_t row, bool row_ok,
                                             volatile int *dirty, int lane) {
    uint32_t v[32];
    tmem_ld32(taddr, v);
    const float4 *t4 = reinterpret_cast<const float4 *>(thr_chunk);
    uint32_t hit = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 th = t4[i];
        hit |= (__uint_as_float(v[4 * i + 0]) >= th.x ? 1u : 0u) << (4 * i + 0);
        hit |= (__uint_as_float(v[4 * i + 1]) >= th.y ? 1u : 0u) << (4 * i + 1);
        hit |= (__uint_as_float(v[4 * i + 2]) >= th.z ? 1u : 0u) << (4 * i + 2);
        hit |= (__uint_as_float(v[4 * i + 3]) >= th.w ? 1u : 0u) << (4 * i + 3);
    }
    if (!row_ok) hit = 0;
    const uint32_t any_col = __reduce_or_sync(0xffffffffu, hit);
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        if (any_col & (1u << b)) {
            const uint32_t m = __ballot_sync(0xffffffffu, (hit >> b) & 1u);
            if (lane == b) mine = m;
        }
    }
    int base = 0;
    if (mine) {
        base = atomicAdd(&cnt_chunk[lane], __popc(mine));
        if (base + __popc(mine) >= kTcSoft) *dirty = 1;
    }
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        if (any_col & (1u << b)) {
            const int base_b = __shfl_sync(0xffffffffu, base, b);
            const uint32_t rows_b = __shfl_sync(0xffffffffu, mine, b);
            if ((hit >> b) & 1u)
                cand_chunk[static_cast<size_t>(b) * kTcCap + base_b + __popc(rows_b & below)] =
                    make_key(__uint_as_float(v[b]), row);
        }
    }
}

// Squared distance between one corpus row and one query, both read from global memory (the row
// has just passed through L2, the queries live there), by the whole warp in the direct
// sum-of-squared-differences form. Every lane returns the full sum.
__device__ __forceinline__ float tc_direct_l2(const __half *row, const __half *query, int d, int lane) {
    float2 sum = make_float2(0.f, 0.f);
    for (int piece = lane; piece * 8 < d; piece += 32) {
        const uint4 xr = __ldg(reinterpret_cast<const uint4 *>(row) + piece);
        const uint4 qr = __ldg(reinterpret_cast<const uint4 *>(query) + piece);
        const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
        const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&xw[e]));
            const float2 q = __half22float2(*reinterpret_cast<const __half2 *>(&qw[e]));
            const float dx = x.x - q.x, dy = x.y - q.y;
            sum.x = fmaf(dx, dx, sum.x);
            sum.y = fmaf(dy, dy, sum.y);
        }
    }
    float v = sum.x + sum.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// The rare part of the selection for L2 (see tc_append_chunk for the appending itself).
// bound_sign = -1: sample launch, the value kept is the lower bound; +1: main launch, pairs that
// pass the filter are scored again in the direct form and kept only if that value passes.
__device__ __noinline__ void tc_append_chunk_l2(uint32_t taddr, const float *thr_chunk, const float *qn_chunk,
                                                int *cnt_chunk, uint64_t *cand_chunk, uint32_t row, bool row_ok,
                                                float nx, float slack, float bound_sign, const __half *corpus,
                                                const __half *queries_chunk, int d, volatile int *dirty,
                                                int lane) {
    uint32_t v[32];
    tmem_ld32(taddr, v);
    uint32_t hit = 0;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        const float s2 = nx + qn_chunk[b];
        const float val = fmaf(2.0f, __uint_as_float(v[b]), 0.0f - s2);
        const float bound = fmaf(bound_sign * slack, s2, val);
        hit |= (bound >= thr_chunk[b] ? 1u : 0u) << b;
        v[b] = __float_as_uint(bound);      // what the sample launch ranks
    }
    if (!row_ok) hit = 0;
    uint32_t any_col = __reduce_or_sync(0xffffffffu, hit);
    if (bound_sign > 0.0f) {
#pragma unroll
        for (int b = 0; b < 32; ++b) {
            if (any_col & (1u << b)) {
                unsigned m = __ballot_sync(0xffffffffu, (hit >> b) & 1u);
                while (m) {
                    const int src = __ffs(m) - 1;
                    m &= m - 1;
                    const uint32_t row_src = __shfl_sync(0xffffffffu, row, src);
                    const float dist = tc_direct_l2(corpus + static_cast<size_t>(row_src) * d,
                                                    queries_chunk + static_cast<size_t>(b) * d, d, lane);
                    if (lane == src) {
                        const float exact = 0.0f - dist;
                        v[b] = __float_as_uint(exact);
                        if (!(exact >= thr_chunk[b])) hit &= ~(1u << b);
                    }
                }
            }
        }
        any_col = __reduce_or_sync(0xffffffffu, hit);
    }
    uint32_t mine = 0;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        if (any_col & (1u << b)) {
            const uint32_t m = __ballot_sync(0xffffffffu, (hit >> b) & 1u);
            if (lane == b) mine = m;
        }
    }
    int base = 0;
    if (mine) {
        base = atomicAdd(&cnt_chunk[lane], __popc(mine));
        if (base + __popc(mine) >= kTcSoft) *dirty = 1;
    }
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        if (any_col & (1u << b)) {
            const int base_b = __shfl_sync(0xffffffffu, base, b);
            const uint32_t rows_b = __shfl_sync(0xffffffffu, mine, b);
            if ((hit >> b) & 1u)
                cand_chunk[static_cast<size_t>(b) * kTcCap + base_b + __popc(rows_b & below)] =
                    make_key(__uint_as_float(v[b]), row);
        }
    }
}

// ---- CTA-pair helpers (PAIR = true: two CTAs of a cluster work as one MMA unit) -----------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tile load whose completion is signalled on an mbarrier that may live in the other CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y,
                                                 uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(cluster_bar)
        : "memory");
}
// Arrive on the barrier at this offset in both CTAs of the pair once the MMAs issued so far are done.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"(static_cast<uint16_t>(3))
        : "memory");
}
__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// PAIR = false: every CTA is on its own (M = 128 rows per MMA).
// PAIR = true: clusters of two CTAs. A row tile is 256 rows; CTA r of the pair stages rows
// 128 r .. 128 r + 127 and half of the query rows of each K chunk, the leader (rank 0) issues
// one M = 256 MMA for both, and each CTA finds the scores of its own 128 rows in its own
// TMEM. Per CTA and chunk this stages 16 KB + nb/2 query rows instead of 16 KB + nb.
template <bool PAIR>
__global__ void __launch_bounds__(kTcThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_q,
               const TcParams p) {
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    TcHeader *hdr = reinterpret_cast<TcHeader *>(tc_smem);
    float *thr = reinterpret_cast<float *>(tc_smem + kTcOffThr);
    int *cnt = reinterpret_cast<int *>(tc_smem + kTcOffCnt);
    int *sorted = reinterpret_cast<int *>(tc_smem + kTcOffSorted);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int S = p.stages;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // 0 = leader of the pair
    const bool leader = rank == 0;
    const int group = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int ngroups = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    constexpr int kGroupRows = PAIR ? 2 * kTcTileM : kTcTileM;
    const int nb_cta = PAIR ? p.nb / 2 : p.nb;             // query rows this CTA stages per chunk

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(smem_u32(&hdr->full[i]), 1);
            mbar_init(smem_u32(&hdr->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&hdr->tmem_full[i]), 1);
            // one arrival per selection warp (of both CTAs for a pair)
            mbar_init(smem_u32(&hdr->tmem_empty[i]), PAIR ? 8 : 4);
        }
        mbar_init(smem_u32(&hdr->drain), 1);
        mbar_fence_init();
        hdr->abort = 0;
        hdr->dirty[0] = hdr->dirty[1] = hdr->dirty[2] = 0;
    }
    for (int q = threadIdx.x; q < kTcMaxQueries; q += kTcThreads) {
        // absent queries never pass; the others start at a score that k rows are already known
        // to reach, when the caller has one
        thr[q] = (q < p.s) ? (p.thr_init ? p.thr_init[p.q_base + q] : -INFINITY) : INFINITY;
        cnt[q] = 0;
        sorted[q] = 0;
    }
    float *qn = reinterpret_cast<float *>(tc_smem + kTcOffQn);
    if (p.mode != 0) {
        for (int q = threadIdx.x; q < kTcMaxQueries; q += kTcThreads) {
            float acc = 0.f;
            if (q < p.s) {
                const __half *qv = p.queries + static_cast<size_t>(q) * p.d;
                for (int i = 0; i < p.d; ++i) {
                    const float a = __half2float(qv[i]);
                    acc = fmaf(a, a, acc);
                }
            }
            qn[q] = acc;
        }
    }
    if (warp == 1) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&hdr->tmem_base)),
                         "r"(kTcTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32(&hdr->tmem_base)),
                         "r"(kTcTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_barrier();  // the partner's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t *>(&hdr->tmem_base);

    const long long my_tiles = (p.ntiles > group) ? (p.ntiles - group + ngroups - 1) / ngroups : 0;
    const long long my_units = my_tiles * p.nhalves;
    volatile int *abort_flag = &hdr->abort;
    const uint32_t stage_base = smem_u32(tc_smem + p.off_stage);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            // bytes that land per stage and phase on the barrier the MMA thread waits on: a
            // pair's loads all report to the leader's barrier
            const uint32_t stage_tx = static_cast<uint32_t>(kTcABytes + nb_cta * 128) * (PAIR ? 2u : 1u);
            int st = 0;
            uint32_t lap = 0;
            long long issued = 0;
            bool ok = true, stop = false;
            for (long long u = 0; u < my_units && !stop; ++u) {
                const long long tile = p.tile0 + group + (u / p.nhalves) * ngroups;
                const int half = static_cast<int>(u % p.nhalves);
                const int row_y = static_cast<int>(tile * kGroupRows + rank * kTcTileM);
                // a pair splits the N of this unit's MMA, not nb: the follower supplies the upper
                // half of the (rounded) queries this half really has
                const int nq_u = (p.s - half * p.nb < p.nb) ? (p.s - half * p.nb) : p.nb;
                const int query_y = half * p.nb + (PAIR ? static_cast<int>(rank) * (((nq_u + 31) & ~31) / 2) : 0);
                for (int c = 0; c < p.nchunks; ++c) {
                    ok = mbar_wait_bounded(smem_u32(&hdr->empty[st]), (lap & 1) ^ 1);
                    if (!ok || *abort_flag) {
                        stop = true;
                        break;
                    }
                    const uint32_t bar = smem_u32(&hdr->full[st]);
                    const uint32_t dst = stage_base + static_cast<uint32_t>(st) * p.stage_bytes;
                    if (PAIR) {
                        const uint32_t lead_bar = map_to_cta(bar, 0);
                        if (leader) mbar_arrive_expect_tx(bar, stage_tx);
                        tma_load_2d_pair(dst, &map_x, c * kTcChunkK, row_y, lead_bar);
                        tma_load_2d_pair(dst + kTcABytes, &map_q, c * kTcChunkK, query_y, lead_bar);
                    } else {
                        mbar_arrive_expect_tx(bar, stage_tx);
                        tma_load_2d(dst, &map_x, c * kTcChunkK, row_y, bar);
                        tma_load_2d(dst + kTcABytes, &map_q, c * kTcChunkK, query_y, bar);
                    }
                    ++issued;
                    if (++st == S) {
                        st = 0;
                        ++lap;
                    }
                }
            }
            if (!ok && !*abort_flag) {
                atomicMax(p.status, kStatusTimeout);
                *abort_flag = 1;
            }
            if (*abort_flag && (!PAIR || leader)) {
                // winding down early: let every copy already issued land before exit (a pair's
                // follower cannot watch the leader's barrier; its copies land in its own shared
                // memory, which stays allocated until both CTAs have passed the final barrier,
                // and a wait has already run out by then)
                const long long first = issued > S ? issued - S : 0;
                for (long long it = first; it < issued; ++it)
                    mbar_wait_bounded(smem_u32(&hdr->full[it % S]), static_cast<uint32_t>((it / S) & 1));
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && leader) {
            int st = 0;
            uint32_t lap = 0;
            bool ok = true;
            for (long long u = 0; u < my_units && ok; ++u) {
                const int half = static_cast<int>(u % p.nhalves);
                const int acc = static_cast<int>(u & 1);
                const int nq = (p.s - half * p.nb < p.nb) ? (p.s - half * p.nb) : p.nb;
                const int n_mma = PAIR ? ((nq + 31) & ~31) : ((nq + 15) & ~15);
                const uint32_t idesc = tc_idesc(n_mma, kGroupRows);
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kTcMaxN);
                // the selection warps must have drained this accumulator's previous unit
                ok = mbar_wait_bounded(smem_u32(&hdr->tmem_empty[acc]), static_cast<uint32_t>(((u >> 1) & 1) ^ 1));
                if (!ok || *abort_flag) break;
                tc_fence_after();
                for (int c = 0; c < p.nchunks; ++c) {
                    // (the mbarrier wait orders the TMA writes before the MMAs that read them; no
                    // tcgen05 fence here: it is only needed where tcgen05 work of other threads,
                    // the selection warps' loads, has to be ordered, as above)
                    ok = mbar_wait_bounded(smem_u32(&hdr->full[st]), lap & 1);
                    if (!ok || *abort_flag) break;
                    const uint32_t a_addr = stage_base + static_cast<uint32_t>(st) * p.stage_bytes;
                    const uint32_t b_addr = a_addr + kTcABytes;
#pragma unroll
                    for (int kk = 0; kk < kTcChunkK / 16; ++kk) {
                        if (PAIR)
                            tc_mma_f16_pair(d_tmem, tc_smem_desc(a_addr + kk * 32), tc_smem_desc(b_addr + kk * 32),
                                            idesc, (c | kk) != 0 ? 1u : 0u);
                        else
                            tc_mma_f16(d_tmem, tc_smem_desc(a_addr + kk * 32), tc_smem_desc(b_addr + kk * 32),
                                       idesc, (c | kk) != 0 ? 1u : 0u);
                    }
                    // stage reusable (in both CTAs of a pair) once these MMAs are done
                    if (PAIR) tc_commit_pair(smem_u32(&hdr->empty[st]));
                    else tc_commit(smem_u32(&hdr->empty[st]));
                    if (++st == S) {
                        st = 0;
                        ++lap;
                    }
                }
                if (!ok || *abort_flag) break;
                if (PAIR) tc_commit_pair(smem_u32(&hdr->tmem_full[acc]));
                else tc_commit(smem_u32(&hdr->tmem_full[acc]));
            }
            if (!ok && !*abort_flag) {
                atomicMax(p.status, kStatusTimeout);
                *abort_flag = 1;
            }
            // every MMA issued above must have completed before the TMEM is given back
            if (PAIR) tc_commit_pair(smem_u32(&hdr->drain));
            else tc_commit(smem_u32(&hdr->drain));
            mbar_wait_bounded(smem_u32(&hdr->drain), 0);
        }
    } else {
        // ------------------------------------------------------------------ selection
        const int ew = warp - 2;        // 0..3
        const int quarter = warp & 3;   // the TMEM lanes this warp may read: 32 * quarter ..
        uint64_t *my_cand = p.cand + static_cast<size_t>(blockIdx.x) * p.cand_q * kTcCap;
        bool ok = true;
        for (long long u = 0; u < my_units; ++u) {
            const long long tile = p.tile0 + group + (u / p.nhalves) * ngroups;
            const int half = static_cast<int>(u % p.nhalves);
            const int acc = static_cast<int>(u & 1);
            const int qb = half * p.nb;
            const int nq = (p.s - qb < p.nb) ? (p.s - qb) : p.nb;
            volatile int *dirty = &hdr->dirty[u % 3];
            if (ok && !*abort_flag) {
                int got = 0;
                if (lane == 0)
                    got = mbar_wait_bounded(smem_u32(&hdr->tmem_full[acc]), static_cast<uint32_t>((u >> 1) & 1)) ? 1 : 0;
                got = __shfl_sync(0xffffffffu, got, 0);
                if (!got) {
                    ok = false;
                    if (lane == 0) {
                        atomicMax(p.status, kStatusTimeout);
                        *abort_flag = 1;
                    }
                }
            }
            const bool live = ok && !*abort_flag;
            if (live) {
                tc_fence_after();
                const long long row = tile * kGroupRows + rank * kTcTileM + quarter * 32 + lane;
                const bool row_ok = row < p.N;
                const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                       static_cast<uint32_t>(acc * kTcMaxN);
                const float nx = (p.mode != 0 && row_ok) ? __ldg(p.norms + row) : 0.f;
                const float bound_sign = p.mode == 1 ? -1.0f : 1.0f;
                for (int j = 0; p.mode != 0 && j * 32 < nq; ++j) {
                    // L2: the same loop on the bound of -distance^2 (see TcParams::mode)
                    uint32_t v[32];
                    tmem_ld32(t_row + j * 32, v);
                    const float4 *t4 = reinterpret_cast<const float4 *>(thr + qb + j * 32);
                    const float4 *n4 = reinterpret_cast<const float4 *>(qn + qb + j * 32);
                    const float sl = bound_sign * p.slack;
                    bool p0 = false, p1 = false, p2 = false, p3 = false;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 th = t4[i];
                        const float4 nq4 = n4[i];
                        const float s0 = nx + nq4.x, s1 = nx + nq4.y, s2 = nx + nq4.z, s3 = nx + nq4.w;
                        p0 |= fmaf(sl, s0, fmaf(2.0f, __uint_as_float(v[4 * i + 0]), 0.0f - s0)) >= th.x;
                        p1 |= fmaf(sl, s1, fmaf(2.0f, __uint_as_float(v[4 * i + 1]), 0.0f - s1)) >= th.y;
                        p2 |= fmaf(sl, s2, fmaf(2.0f, __uint_as_float(v[4 * i + 2]), 0.0f - s2)) >= th.z;
                        p3 |= fmaf(sl, s3, fmaf(2.0f, __uint_as_float(v[4 * i + 3]), 0.0f - s3)) >= th.w;
                    }
                    if (__any_sync(0xffffffffu, row_ok && (p0 | p1 | p2 | p3)))
                        tc_append_chunk_l2(t_row + j * 32, thr + qb + j * 32, qn + qb + j * 32, cnt + qb + j * 32,
                                           my_cand + static_cast<size_t>(qb + j * 32) * kTcCap,
                                           static_cast<uint32_t>(row), row_ok, nx, p.slack, bound_sign, p.corpus,
                                           p.queries + static_cast<size_t>(qb + j * 32) * p.d, p.d, dirty, lane);
                }
                for (int j = 0; p.mode == 0 && j * 32 < nq; ++j) {
                    uint32_t v[32];
                    tmem_ld32(t_row + j * 32, v);
                    const float4 *t4 = reinterpret_cast<const float4 *>(thr + qb + j * 32);
                    // common case: nothing passes. Four independent predicate chains.
                    bool p0 = false, p1 = false, p2 = false, p3 = false;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 th = t4[i];
                        p0 |= __uint_as_float(v[4 * i + 0]) >= th.x;
                        p1 |= __uint_as_float(v[4 * i + 1]) >= th.y;
                        p2 |= __uint_as_float(v[4 * i + 2]) >= th.z;
                        p3 |= __uint_as_float(v[4 * i + 3]) >= th.w;
                    }
                    if (__any_sync(0xffffffffu, row_ok && (p0 | p1 | p2 | p3)))
                        tc_append_chunk(t_row + j * 32, thr + qb + j * 32, cnt + qb + j * 32,
                                        my_cand + static_cast<size_t>(qb + j * 32) * kTcCap,
                                        static_cast<uint32_t>(row), row_ok, dirty, lane);
                }
                // accumulator drained: hand it back to the MMA thread (the pair's leader)
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&hdr->tmem_empty[acc]), 0));
                    else mbar_arrive(smem_u32(&hdr->tmem_empty[acc]));
                }
            }
            // All four warps meet after every unit (also when winding down, so that nobody is
            // left waiting) so that every push of the unit is visible; each then reads the
            // unit's flag. Three flags in rotation make one barrier enough: unit u's flag is
            // written during unit u, read between the barriers that end units u and u + 1, and
            // cleared after the barrier that ends unit u + 1, well before unit u + 3 writes it.
            named_barrier(1, 128);
            const int need = *dirty;
            if (threadIdx.x == 64) *reinterpret_cast<volatile int *>(&hdr->dirty[(u + 2) % 3]) = 0;
            if (need) {
                for (int base = 0; base < p.s; base += 128) {
                    const int q = base + ew * 32 + lane;
                    unsigned m = __ballot_sync(0xffffffffu, q < p.s && cnt[q] >= kTcSoft);
                    while (m) {
                        const int b = __ffs(m) - 1;
                        m &= m - 1;
                        const int qq = base + ew * 32 + b;
                        tc_compact_query(my_cand + static_cast<size_t>(qq) * kTcCap, thr, cnt, sorted, qq, p.k, lane);
                    }
                }
                named_barrier(1, 128);  // thresholds and counts settled before the next unit's pushes
            }
        }
        // ---- CTA result: every list sorted and cut to k, written as this CTA's partial lists
        for (int base = 0; base < p.s; base += 128) {
            const int q0 = base + ew * 32;
            for (int b = 0; b < 32 && q0 + b < p.s; ++b) {
                const int q = q0 + b;
                uint64_t *list = my_cand + static_cast<size_t>(q) * kTcCap;
                if (cnt[q] != sorted[q]) tc_compact_query(list, thr, cnt, sorted, q, p.k, lane);
                const int n = cnt[q];
                uint64_t *dst = p.partial + (static_cast<size_t>(blockIdx.x) * p.s_total + p.q_base + q) * p.k;
                for (int i = lane; i < p.k; i += 32) dst[i] = (i < n) ? list[i] : 0ull;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // a pair leaves together: the leader's MMAs read the follower's shared memory and its
    // commits arrive on the follower's barriers
    if (PAIR) cluster_barrier();
    if (warp == 1) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols)
                         : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcTmemCols)
                         : "memory");
    }
}

}  // namespace ralm
