// Corpus scan for large query batches (up to 512 queries per pass; inner product, and L2 through
// the same inner-product tiles, see TcParams::mode) on the
// fifth-generation tensor cores: scores = corpus tile [128 rows] x queries^T [up to 256] with
// tcgen05.mma, fp16 operands, fp32 accumulators in tensor memory (TMEM), fused with the
// per-CTA top-k selection so that the N x s score matrix never exists in memory.
//
// One persistent CTA per SM, 6 warps:
//   warp 0      producer: issues the TMA tile loads. A K chunk is 64 fp16 = 128 bytes per row
//               (the 128-byte swizzle span) of 128 corpus rows and of up to 256 queries; a
//               stage holds up to two chunks; stages form a ring guarded by full/empty
//               mbarriers.
//   warp 1      MMA: issues tcgen05.mma (M = 128, N = 16..256, K = 16 per instruction, 4 per
//               chunk) and one tcgen05.commit per stage. A work unit is (row tile, half of
//               the queries); the two halves of TMEM (256 columns each) alternate between
//               units, so one accumulator is drained while the next is being filled.
//               Both warps run their loops with all 32 lanes converged and only the
//               instruction that starts the asynchronous work sits under an elected lane:
//               the waits, loop counters, addresses and descriptors then stay warp-uniform.
//               (Run by a single lane inside a divergent branch, the same loop took ~190
//               cycles per MMA and ~240 per wait + commit, whatever N was, and bounded the
//               kernel: 4 MMAs per commit cost 857 cycles against 572 converged; with 8 per
//               commit the converged loop is hidden behind the tensor pipe, 128 cycles per
//               M = 256, N = 256, K = 16 instruction.)
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
// Candidate lists per (CTA, query): `cap` slots; a list holding `soft` keys or more is compacted
// before the next unit, in which at most 128 more arrive (soft + 128 <= cap). k <= 64: 256 slots
// and soft 120, just under 128 so that the usual sort is one of 128 keys; k <= 256: 512 slots.
constexpr int kTcCapSmall = 256, kTcSoftSmall = 120, kTcSmallK = 64;
constexpr int kTcCapLarge = 512, kTcSoftLarge = 380;
constexpr int kTcMaxK = 256;
constexpr int kTcTmemCols = 512;

struct TcParams {
    uint64_t *partial;  // [gridDim.x][s_total][k] sorted keys, 0 = empty
    uint64_t *cand;     // [gridDim.x][cand_q][cap] candidate lists
    int cap, soft;      // slots per list; fill level that asks for a compaction (see kTcCapSmall)
    int *status;
    long long N;        // rows of this launch end here (the whole corpus, or the end of a sample)
    long long tile0;    // first row tile (of 128 rows, 256 for pairs) of this launch
    const float *thr_init;  // [s_total] starting thresholds (scores that k rows are known to reach), or null
    long long ntiles;   // row tiles of this launch
    int *tile_counter;  // zeroed before the launch: row tiles beyond the first of each CTA (pair) are handed out here
    int nchunks;        // ceil(d / 64)
    int s;              // queries in this pass (<= 512)
    int s_total;
    int q_base;
    int k;
    int nb;             // queries per accumulator (16..256; a multiple of 16, of 32 for CTA pairs);
                        // a CTA stages nb query rows per chunk, nb / 2 in a pair
    int nhalves;        // ceil(s / nb): 1 or 2
    int stages;
    int stage_chunks;   // K chunks per stage: 2, or 1 where the ring would otherwise be too short
    int chunk_bytes;    // kTcABytes + (staged query rows) * 128, a multiple of 1024
    int stage_bytes;    // stage_chunks * chunk_bytes
    int off_stage;      // shared-memory offset of the stage ring (1024-byte aligned)
    int cand_q;         // queries the candidate workspace was sized for (>= s)
    // mode 0: inner product, scores ranked as they are.
    // L2 (squared distance) runs on the same inner-product tiles: the tensor-core value
    // v = 2 x.q - |x|^2 - |q|^2 = -distance^2 cancels, so it is never ranked;
    // mode 2 (L2 main launch): a pair passes the filter when v + slack (|x|^2 + |q|^2) reaches the
    //         threshold, and is then scored again in the direct sum-of-squared-differences form
    //         from global memory; only that value is ranked and returned.
    // Sample launches (mode 3 inner product, mode 1 L2) keep no lists at all: every selection
    // warp keeps, per query, the best rank value among the rows it has seen (L2: the best LOWER
    // BOUND v - slack (|x|^2 + |q|^2)) and writes these maxima to gmax. The warps' rows are
    // disjoint, so the k-th largest of a query's maxima is a rank value that k different rows are
    // known to reach: the threshold the main launch starts from. The main launch then scans all
    // rows, the sample's too.
    int mode;
    float *gmax;        // sample launches: [gridDim.x * 4][s_total] maxima, -inf where a warp saw no row
    Extents ext;        // extents of the global arrays, for the debug build's checks
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
    uint64_t tile_full[32];  // tile_ring[i] holds the number of this CTA's (i + 32 n)-th row tile
    int tile_ring[32];
    int sel_tile[2];         // the selection warps' copy of their current tile number (even / odd tiles)
    uint32_t tmem_base;
    int abort;
    int dirty[3];  // [u % 3]: some candidate list reached the soft limit during unit u
};
constexpr int kTcHeaderBytes = 1024;
constexpr int kTcTileRing = 32;  // (a power of two; see scan_tc_kernel for why 32 is enough)
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
// One lane of a converged warp (the same one every time it is asked).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// Bounded wait that also gives up when another warp of the CTA has started winding down. The
// first probe is inline: the common case, a phase that completed long ago, costs one instruction.
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag || clock64() - t0 > kWaitCycleLimit) return false;
    }
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
                                                 int k, int cap, int lane) {
    const int n = cnt[q] < cap ? cnt[q] : cap;  // (the cap: see tc_append_octet)
    if (n <= 32) tc_compact_sorted<1>(list, thr, cnt, sorted, q, n, k, lane);
    else if (n <= 64) tc_compact_sorted<2>(list, thr, cnt, sorted, q, n, k, lane);
    else if (n <= 128) tc_compact_sorted<4>(list, thr, cnt, sorted, q, n, k, lane);
    else if (n <= 256) tc_compact_sorted<8>(list, thr, cnt, sorted, q, n, k, lane);
    else tc_compact_sorted<16>(list, thr, cnt, sorted, q, n, k, lane);
}

// Appending itself: every row (lane) whose bit b of `hit` is set stores key(v[b], row) in column
// b's list. Only columns with a hit anywhere in the warp are visited (a warp-uniform branch per
// column); each hit reserves its slot with its own shared-memory atomic.
__device__ __forceinline__ void tc_store_hits(const uint32_t (&v)[32], uint32_t hit, int *cnt_chunk,
                                              uint64_t *cand_chunk, uint32_t row, volatile int *dirty, int *status, int cap,
                                              int soft, long long room) {
    const uint32_t any_col = __reduce_or_sync(0xffffffffu, hit);
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        if (any_col & (1u << b)) {
            if ((hit >> b) & 1u) {
                const int slot = atomicAdd(&cnt_chunk[b], 1);
                if (slot + 1 >= soft) *dirty = 1;
                if (slot >= cap) atomicMax(status, kStatusInternal);
                else if (in_bounds(static_cast<long long>(b) * cap + slot, room, status))
                    cand_chunk[static_cast<size_t>(b) * cap + slot] = make_key(__uint_as_float(v[b]), row);
            }
        }
    }
}

// The rare part of the selection: some score among this warp's 32 rows x 8 columns (columns
// c0 .. c0 + 7 of a block of 32) passes its threshold. Out of line, so that the common path (no
// score passes) stays a short loop. thr_lane: the threshold of column `lane` of the block
// (thresholds travel by shuffle, not through shared memory, whose loads are slow while TMA and the
// tensor core keep it busy). Every row whose score passes stores key(score, row) in that
// column's list, reserving its slot with its own shared-memory atomic.
__device__ __noinline__ void tc_append_octet(uint32_t v0, uint32_t v1, uint32_t v2, uint32_t v3, uint32_t v4,
                                             uint32_t v5, uint32_t v6, uint32_t v7, int c0, float thr_lane,
                                             int *cnt_block, uint64_t *cand_block, uint32_t row, bool row_ok,
                                             volatile int *dirty, int *status, int cap, int soft,
                                             long long room) {
    // (room: keys between cand_block and the end of the list array; checked in the debug build)
    const uint32_t v[8] = {v0, v1, v2, v3, v4, v5, v6, v7};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float t = __shfl_sync(0xffffffffu, thr_lane, c0 + i);
        if (row_ok && __uint_as_float(v[i]) >= t) {
            const int slot = atomicAdd(&cnt_block[c0 + i], 1);
            if (slot + 1 >= soft) *dirty = 1;
            // (a list holds fewer than `soft` keys when a unit starts and gains at most 128 in
            // one, so slot < cap; should that ever fail the key is dropped and the status
            // word says so, rather than writing into the neighbouring list)
            if (slot >= cap)
                atomicMax(status, kStatusInternal);
            else if (in_bounds(static_cast<long long>(c0 + i) * cap + slot, room, status))
                cand_block[static_cast<size_t>(c0 + i) * cap + slot] = make_key(__uint_as_float(v[i]), row);
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

// The rare part of the selection for L2 (main launch): pairs whose upper bound of -distance^2
// reaches the threshold are scored again in the direct form and kept only if that value passes.
__device__ __noinline__ void tc_append_chunk_l2(uint32_t taddr, const float *thr_chunk, const float *qn_chunk,
                                                int *cnt_chunk, uint64_t *cand_chunk, uint32_t row, bool row_ok,
                                                float nx, float slack, const __half *corpus,
                                                const __half *queries_chunk, int d, volatile int *dirty,
                                                int *status, int cap, int soft, long long room, int lane) {
    uint32_t v[32];
    tmem_ld32(taddr, v);
    uint32_t hit = 0;
#pragma unroll
    for (int b = 0; b < 32; ++b) {
        const float s2 = nx + qn_chunk[b];
        const float val = fmaf(2.0f, __uint_as_float(v[b]), 0.0f - s2);
        hit |= (fmaf(slack, s2, val) >= thr_chunk[b] ? 1u : 0u) << b;
    }
    if (!row_ok) hit = 0;
    const uint32_t any_col = __reduce_or_sync(0xffffffffu, hit);
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
    tc_store_hits(v, hit, cnt_chunk, cand_chunk, row, dirty, status, cap, soft, room);
}

// One block of 32 queries of a sample launch: for every column the best rank value among this
// warp's 32 rows (as order-preserving bits, 0 = no row), folded into lane c's running maximum
// for column c.
__device__ __forceinline__ void tc_fold_block_maxima(const uint32_t (&v)[32], bool row_ok, uint32_t &best, int lane) {
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const uint32_t mine = row_ok ? ordered_bits(__uint_as_float(v[c]) + 0.0f) : 0u;
        const uint32_t m = __reduce_max_sync(0xffffffffu, mine);
        if (lane == c) best = m > best ? m : best;
    }
}

// Lane L's copy of the thresholds of queries L, L + 32, ... of both halves (+inf where there
// is none): tl[h][j] belongs to query h * nb + j * 32 + L.
__device__ __forceinline__ void tc_load_lane_thresholds(float (&tl)[2][kTcMaxN / 32], const float *thr, int nb,
                                                        int nhalves, int lane) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < kTcMaxN / 32; ++j) {
            const int q = h * nb + j * 32 + lane;
            tl[h][j] = (h < nhalves && j * 32 < nb && q < kTcMaxQueries) ? thr[q] : INFINITY;
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
// Arrival on a barrier of the pair's other CTA. The barrier only hands a TMEM accumulator back, and
// the reads it follows are ordered by tcgen05.wait::ld and the tcgen05 fence; the arrival's own release
// stays at CTA scope. (With cluster scope it also waited for this thread's earlier global stores to be
// visible across the cluster: about 2500 cycles per unit while TMA traffic is heavy, more than the
// scores take to read.)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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

// Remote store of one 32-bit value into the other CTA's shared memory that completes 4 bytes of
// the transaction count of an mbarrier there (so the value is visible to whoever that barrier lets through).
__device__ __forceinline__ void st_async_u32(uint32_t cluster_addr, uint32_t value, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(cluster_addr),
                 "r"(value), "r"(cluster_bar)
                 : "memory");
}

// Row tiles are handed out dynamically: CTAs (pairs) differ in speed by a few percent, and with a
// fixed assignment the slowest sets the launch's time. The leader's producer warp takes tile
// numbers from a global counter one tile ahead of its loads and publishes them in a small ring in
// shared memory (its own, and by st.async the follower's); every role reads its next tile there.
// The number of this CTA's seq-th tile, or -1 when there is none left (or the wait gave up). All
// lanes of the calling warp get the same value. `arm`: this warp is the follower's producer, whose
// elected lane makes the one arrival of the barrier's phase and announces the 4 bytes to come.
__device__ __forceinline__ long long tc_read_tile(TcHeader *hdr, long long seq, bool arm, bool elected,
                                                  volatile int *abort_flag, int *status, int lane) {
    const int slot = static_cast<int>(seq & (kTcTileRing - 1));
    const uint32_t bar = smem_u32(&hdr->tile_full[slot]);
    if (arm && elected) mbar_arrive_expect_tx(bar, 4);
    if (!tc_wait(bar, static_cast<uint32_t>((seq / kTcTileRing) & 1), abort_flag)) {
        if (lane == 0 && !*abort_flag) {
            atomicMax(status, kStatusTimeout);
            *abort_flag = 1;
        }
        return -1;
    }
    return *reinterpret_cast<volatile int *>(&hdr->tile_ring[slot]);
}

// PAIR = false: every CTA is on its own (M = 128 rows per MMA).
// PAIR = true: clusters of two CTAs. A row tile is 256 rows; CTA r of the pair stages rows
// 128 r .. 128 r + 127 and half of the query rows of each K chunk, the leader (rank 0) issues
// one M = 256 MMA for both, and each CTA finds the scores of its own 128 rows in its own
// TMEM. Per CTA and chunk this stages 16 KB + nb/2 query rows instead of 16 KB + nb.
// MODE: TcParams::mode as a compile-time constant, so that each launch carries only its own
// selection code (the loops over 32-column blocks are fully unrolled).
template <bool PAIR, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_q,
               const TcParams p) {
    extern __shared__ __align__(1024) unsigned char tc_smem[];
    TcHeader *hdr = reinterpret_cast<TcHeader *>(tc_smem);
    float *thr = reinterpret_cast<float *>(tc_smem + kTcOffThr);
    int *cnt = reinterpret_cast<int *>(tc_smem + kTcOffCnt);
    int *sorted = reinterpret_cast<int *>(tc_smem + kTcOffSorted);
    // (through a shuffle, so that the compiler knows the warp index to be the same in all lanes)
    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
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
        for (int i = 0; i < kTcTileRing; ++i) mbar_init(smem_u32(&hdr->tile_full[i]), 1);
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
    if (MODE == 1 || MODE == 2) {
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

    // (tile numbers: the ring of kTcTileRing slots is never overrun. A slot is rewritten 32 tiles
    // later; the publisher runs at most the stage ring (<= 12 tiles) plus one tile ahead of the MMA
    // warp, which runs at most two units ahead of the selection warps.)
    volatile int *abort_flag = &hdr->abort;
    const uint32_t stage_base = smem_u32(tc_smem + p.off_stage);

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        // All lanes run the loop; the elected lane issues the copies.
        const bool elected = elect_one();
        // bytes that land per chunk on the barrier the MMA warp waits on: a pair's loads all
        // report to the leader's barrier
        const uint32_t chunk_tx = static_cast<uint32_t>(kTcABytes + nb_cta * 128) * (PAIR ? 2u : 1u);
        const uint32_t chunk_bytes = static_cast<uint32_t>(p.chunk_bytes);
        const int nchunks = p.nchunks, SC = p.stage_chunks;
        int st = 0;
        uint32_t lap = 0;
        long long issued = 0;
        bool ok = true;
        // The leader publishes this CTA's (pair's) tile numbers: the first is fixed, the others come
        // from the launch's counter, each taken one tile before its loads are due.
        bool more = true;   // (leader's elected lane) the last number published was a tile
        auto publish = [&](long long seq, long long number) {
            const int slot = static_cast<int>(seq & (kTcTileRing - 1));
            const int value = number < p.ntiles ? static_cast<int>(number) : -1;
            more = value >= 0;
            *reinterpret_cast<volatile int *>(&hdr->tile_ring[slot]) = value;
            const uint32_t bar = smem_u32(&hdr->tile_full[slot]);
            mbar_arrive(bar);
            if (PAIR)
                st_async_u32(map_to_cta(smem_u32(&hdr->tile_ring[slot]), 1), static_cast<uint32_t>(value),
                             map_to_cta(bar, 1));
        };
        if (leader && elected) publish(0, group);
        long long tile = -1;
        for (long long u = 0; ok; ++u) {
            const int half = static_cast<int>(u % p.nhalves);
            if (half == 0) {
                const long long seq = u / p.nhalves;
                if (leader && elected && more) publish(seq + 1, ngroups + atomicAdd(p.tile_counter, 1));
                tile = tc_read_tile(hdr, seq, PAIR && !leader, elected, abort_flag, p.status, lane);
                if (tile < 0) break;
                tile += p.tile0;
            }
            const int row_y = static_cast<int>(tile * kGroupRows + rank * kTcTileM);
            // a pair splits the N of this unit's MMA, not nb: the follower supplies the upper
            // half of the (rounded) queries this half really has
            const int nq_u = (p.s - half * p.nb < p.nb) ? (p.s - half * p.nb) : p.nb;
            int query_y = half * p.nb + (PAIR ? static_cast<int>(rank) * (((nq_u + 31) & ~31) / 2) : 0);
            // With 16 queries or fewer in this half the follower's rows all lie beyond the last
            // query. A box that is out of range as a whole costs far more than its zeros are
            // worth (measured: the whole launch up to 20 % slower, depending on where the query
            // buffer sits), so the follower then stages the leader's rows once more: those
            // columns of the product belong to absent queries, which never pass.
            if (PAIR && query_y >= p.s) query_y = half * p.nb;
            for (int c = 0; c < nchunks; c += SC) {
                const int kc = (nchunks - c < SC) ? (nchunks - c) : SC;
                ok = tc_wait(smem_u32(&hdr->empty[st]), (lap & 1) ^ 1, abort_flag);
                if (!ok) break;
                if (elected) {
                    const uint32_t bar = smem_u32(&hdr->full[st]);
                    const uint32_t dst = stage_base + static_cast<uint32_t>(st) * p.stage_bytes;
                    if (PAIR) {
                        const uint32_t lead_bar = map_to_cta(bar, 0);
                        if (leader) mbar_arrive_expect_tx(bar, chunk_tx * kc);
                        for (int j = 0; j < kc; ++j) {
                            tma_load_2d_pair(dst + j * chunk_bytes, &map_x, (c + j) * kTcChunkK, row_y, lead_bar);
                            tma_load_2d_pair(dst + j * chunk_bytes + kTcABytes, &map_q, (c + j) * kTcChunkK, query_y,
                                             lead_bar);
                        }
                    } else {
                        mbar_arrive_expect_tx(bar, chunk_tx * kc);
                        for (int j = 0; j < kc; ++j) {
                            tma_load_2d(dst + j * chunk_bytes, &map_x, (c + j) * kTcChunkK, row_y, bar);
                            tma_load_2d(dst + j * chunk_bytes + kTcABytes, &map_q, (c + j) * kTcChunkK, query_y, bar);
                        }
                    }
                }
                ++issued;
                if (++st == S) {
                    st = 0;
                    ++lap;
                }
            }
        }
        if (!ok && lane == 0 && !*abort_flag) {
            atomicMax(p.status, kStatusTimeout);
            *abort_flag = 1;
        }
        __syncwarp();
        if (*abort_flag && (!PAIR || leader)) {
            // winding down early: let every copy already issued land before exit (a pair's
            // follower cannot watch the leader's barrier; its copies land in its own shared
            // memory, which stays allocated until both CTAs have passed the final barrier,
            // and a wait has already run out by then)
            const long long first = issued > S ? issued - S : 0;
            for (long long it = first; it < issued; ++it)
                mbar_wait_bounded(smem_u32(&hdr->full[it % S]), static_cast<uint32_t>((it / S) & 1));
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // The leader CTA's warp, all lanes converged; the elected lane issues MMAs and commits.
        if (leader) {
            const bool elected = elect_one();
            const uint64_t desc_fixed = tc_smem_desc(0);
            const uint32_t chunk_desc = static_cast<uint32_t>(p.chunk_bytes) >> 4;
            const int nchunks = p.nchunks, SC = p.stage_chunks;
            int st = 0;
            uint32_t lap = 0;
            bool ok = true;
            for (long long u = 0; ok; ++u) {
                const int half = static_cast<int>(u % p.nhalves);
                if (half == 0 && tc_read_tile(hdr, u / p.nhalves, false, elected, abort_flag, p.status, lane) < 0) break;
                const int acc = static_cast<int>(u & 1);
                const int nq = (p.s - half * p.nb < p.nb) ? (p.s - half * p.nb) : p.nb;
                const int n_mma = PAIR ? ((nq + 31) & ~31) : ((nq + 15) & ~15);
                const uint32_t idesc = tc_idesc(n_mma, kGroupRows);
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * kTcMaxN);
                // the selection warps must have drained this accumulator's previous unit
                ok = tc_wait(smem_u32(&hdr->tmem_empty[acc]), static_cast<uint32_t>(((u >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int c = 0; c < nchunks; c += SC) {
                    const int kc = (nchunks - c < SC) ? (nchunks - c) : SC;
                    // (the mbarrier wait orders the TMA writes before the MMAs that read them; no
                    // tcgen05 fence here: it is only needed where tcgen05 work of other threads,
                    // the selection warps' loads, has to be ordered, as above)
                    ok = tc_wait(smem_u32(&hdr->full[st]), lap & 1, abort_flag);
                    if (!ok) break;
                    if (elected) {
                        const uint32_t a_addr = stage_base + static_cast<uint32_t>(st) * p.stage_bytes;
                        const uint64_t a_desc = desc_fixed | ((a_addr & 0x3FFFFu) >> 4);
                        const uint64_t b_desc = desc_fixed | (((a_addr + kTcABytes) & 0x3FFFFu) >> 4);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            if (j < kc) {
#pragma unroll
                                for (int kk = 0; kk < kTcChunkK / 16; ++kk) {
                                    // (a K step of 16 is 32 bytes further along the 128-byte rows)
                                    const uint32_t step = j * chunk_desc + kk * 2;
                                    if (PAIR) tc_mma_f16_pair(d_tmem, a_desc + step, b_desc + step, idesc, accumulate);
                                    else tc_mma_f16(d_tmem, a_desc + step, b_desc + step, idesc, accumulate);
                                    accumulate = 1;
                                }
                            }
                        }
                        // stage reusable (in both CTAs of a pair) once these MMAs are done
                        if (PAIR) tc_commit_pair(smem_u32(&hdr->empty[st]));
                        else tc_commit(smem_u32(&hdr->empty[st]));
                    }
                    accumulate = 1;
                    if (++st == S) {
                        st = 0;
                        ++lap;
                    }
                }
                if (!ok) break;
                if (elected) {
                    if (PAIR) tc_commit_pair(smem_u32(&hdr->tmem_full[acc]));
                    else tc_commit(smem_u32(&hdr->tmem_full[acc]));
                }
            }
            if (!ok && lane == 0 && !*abort_flag) {
                atomicMax(p.status, kStatusTimeout);
                *abort_flag = 1;
            }
            __syncwarp();
            // every MMA issued above must have completed before the TMEM is given back
            if (elected) {
                if (PAIR) tc_commit_pair(smem_u32(&hdr->drain));
                else tc_commit(smem_u32(&hdr->drain));
            }
            mbar_wait_bounded(smem_u32(&hdr->drain), 0);
        }
    } else {
        // ------------------------------------------------------------------ selection
        const int ew = warp - 2;        // 0..3
        const int quarter = warp & 3;   // the TMEM lanes this warp may read: 32 * quarter ..
        uint64_t *my_cand = p.cand + static_cast<size_t>(blockIdx.x) * p.cand_q * p.cap;
        const long long cand_room = p.ext.lists - static_cast<long long>(blockIdx.x) * p.cand_q * p.cap;
        constexpr bool sample = MODE == 1 || MODE == 3;
        constexpr bool l2 = MODE == 1 || MODE == 2;
        bool ok = true;
        // Per-query values live in registers, spread over the lanes: lane L holds those of queries
        // L, L + 32, ... and column c's value reaches every row by a shuffle from lane c. The
        // common path then reads no shared memory, whose loads take several times longer while
        // TMA and the tensor core keep it busy (440 against 100 cycles per block of 32 queries).
        // tl: thresholds (main launches; reloaded after a compaction meeting, the only place where
        // they move). qnl: |q|^2 (L2). best: running maxima of a sample launch.
        float tl[2][kTcMaxN / 32], qnl[2][kTcMaxN / 32], al[2][kTcMaxN / 32];
        uint32_t best[2][kTcMaxN / 32];
        const float wide_slack = p.slack * 1.001f + 1.0f / 1048576.0f;
        tc_load_lane_thresholds(tl, thr, p.nb, p.nhalves, lane);
        if (l2) tc_load_lane_thresholds(qnl, qn, p.nb, p.nhalves, lane);
        // L2 main launch: the per-query side of the filter, thr / 2 + (1 - slack) |q|^2 / 2
        auto refresh_rhs = [&]() {
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int j = 0; j < kTcMaxN / 32; ++j) al[h][j] = fmaf(0.5f * (1.0f - wide_slack), qnl[h][j], 0.5f * tl[h][j]);
        };
        if (l2 && !sample) refresh_rhs();
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int j = 0; j < kTcMaxN / 32; ++j) best[h][j] = 0u;
        long long tile = -1;
        for (long long u = 0;; ++u) {
            const int half = static_cast<int>(u % p.nhalves);
            if (half == 0) {
                // One warp waits for the tile number and hands it to the others, so that all four
                // take the same decision (also when that wait gives up) and leave together: they
                // meet at named barriers that have no time limit.
                const long long seq = u / p.nhalves;
                if (ew == 0) {
                    const long long number = tc_read_tile(hdr, seq, false, false, abort_flag, p.status, lane);
                    if (lane == 0) *reinterpret_cast<volatile int *>(&hdr->sel_tile[seq & 1]) = static_cast<int>(number);
                }
                named_barrier(2, 128);
                tile = *reinterpret_cast<volatile int *>(&hdr->sel_tile[seq & 1]);
                if (tile < 0) break;
                tile += p.tile0;
            }
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
                const float nx = (l2 && row_ok && in_bounds(row, p.ext.rows, p.status)) ? __ldg(p.norms + row) : 0.f;
                // L2: this row's part of the bound (see below)
                const float row_part = sample ? 0.0f - (1.0f + wide_slack) * nx : 0.0f - 0.5f * (1.0f - wide_slack) * nx;
#pragma unroll
                for (int j = 0; j < kTcMaxN / 32; ++j) {
                    if (j * 32 < nq) {
                        uint32_t v[32];
                        tmem_ld32(t_row + j * 32, v);
                        if (sample) {
                            if (l2) {
                                // the part of the LOWER bound of -distance^2 that depends on the row:
                                // 2 x.q - (1 + slack) |x|^2; the query's part is subtracted at the end
#pragma unroll
                                for (int c = 0; c < 32; ++c)
                                    v[c] = __float_as_uint(fmaf(2.0f, __uint_as_float(v[c]), row_part));
                            }
                            if (half) tc_fold_block_maxima(v, row_ok, best[1][j], lane);
                            else tc_fold_block_maxima(v, row_ok, best[0][j], lane);
                        } else if (l2) {
                            // the UPPER bound of -distance^2 against the thresholds, rearranged so that
                            // the common path costs what the inner-product one does:
                            //   2 x.q - (1 - slack)(|x|^2 + |q|^2) >= thr
                            //   <=>  x.q - (1 - slack)|x|^2 / 2  >=  thr / 2 + (1 - slack)|q|^2 / 2
                            // (left: per row, right: per query, by shuffle from the lane that holds it;
                            // the slack used here is a little larger than the append routine's, so
                            // the rearrangement's own rounding cannot drop a pair that routine keeps)
                            const float my_rhs = half ? al[1][j] : al[0][j];
                            // (the row's part is added two columns per instruction)
                            const float2 row_part2 = make_float2(row_part, row_part);
#pragma unroll
                            for (int c = 0; c < 32; c += 2) {
                                const float2 t = __fadd2_rn(make_float2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), row_part2);
                                v[c] = __float_as_uint(t.x);
                                v[c + 1] = __float_as_uint(t.y);
                            }
                            bool p0 = false, p1 = false, p2 = false, p3 = false;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                p0 |= __uint_as_float(v[4 * i + 0]) >= __shfl_sync(0xffffffffu, my_rhs, 4 * i + 0);
                                p1 |= __uint_as_float(v[4 * i + 1]) >= __shfl_sync(0xffffffffu, my_rhs, 4 * i + 1);
                                p2 |= __uint_as_float(v[4 * i + 2]) >= __shfl_sync(0xffffffffu, my_rhs, 4 * i + 2);
                                p3 |= __uint_as_float(v[4 * i + 3]) >= __shfl_sync(0xffffffffu, my_rhs, 4 * i + 3);
                            }
                            if (__any_sync(0xffffffffu, row_ok && (p0 | p1 | p2 | p3)))
                                tc_append_chunk_l2(t_row + j * 32, thr + qb + j * 32, qn + qb + j * 32, cnt + qb + j * 32,
                                                   my_cand + static_cast<size_t>(qb + j * 32) * p.cap,
                                                   static_cast<uint32_t>(row), row_ok, nx, p.slack, p.corpus,
                                                   p.queries + static_cast<size_t>(qb + j * 32) * p.d, p.d, dirty, p.status, p.cap, p.soft,
                                                   cand_room - static_cast<long long>(qb + j * 32) * p.cap, lane);
                        } else {
                            // common case: nothing passes. Four independent predicate chains, one per
                            // eight columns, so that the rare case only revisits the eight it concerns.
                            const float my_thr = half ? tl[1][j] : tl[0][j];
                            bool p0 = false, p1 = false, p2 = false, p3 = false;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                p0 |= __uint_as_float(v[i]) >= __shfl_sync(0xffffffffu, my_thr, i);
                                p1 |= __uint_as_float(v[8 + i]) >= __shfl_sync(0xffffffffu, my_thr, 8 + i);
                                p2 |= __uint_as_float(v[16 + i]) >= __shfl_sync(0xffffffffu, my_thr, 16 + i);
                                p3 |= __uint_as_float(v[24 + i]) >= __shfl_sync(0xffffffffu, my_thr, 24 + i);
                            }
                            if (__any_sync(0xffffffffu, row_ok && (p0 | p1 | p2 | p3))) {
                                int *cnt_block = cnt + qb + j * 32;
                                uint64_t *cand_block = my_cand + static_cast<size_t>(qb + j * 32) * p.cap;
                                const long long room = cand_room - static_cast<long long>(qb + j * 32) * p.cap;
                                const uint32_t r32 = static_cast<uint32_t>(row);
                                if (__any_sync(0xffffffffu, row_ok && p0))
                                    tc_append_octet(v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], 0, my_thr, cnt_block,
                                                    cand_block, r32, row_ok, dirty, p.status, p.cap, p.soft, room);
                                if (__any_sync(0xffffffffu, row_ok && p1))
                                    tc_append_octet(v[8], v[9], v[10], v[11], v[12], v[13], v[14], v[15], 8, my_thr,
                                                    cnt_block, cand_block, r32, row_ok, dirty, p.status, p.cap, p.soft, room);
                                if (__any_sync(0xffffffffu, row_ok && p2))
                                    tc_append_octet(v[16], v[17], v[18], v[19], v[20], v[21], v[22], v[23], 16, my_thr,
                                                    cnt_block, cand_block, r32, row_ok, dirty, p.status, p.cap, p.soft, room);
                                if (__any_sync(0xffffffffu, row_ok && p3))
                                    tc_append_octet(v[24], v[25], v[26], v[27], v[28], v[29], v[30], v[31], 24, my_thr,
                                                    cnt_block, cand_block, r32, row_ok, dirty, p.status, p.cap, p.soft, room);
                            }
                        }
                    }
                }
                // accumulator drained: hand it back to the MMA warp (the pair's leader)
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (PAIR) mbar_arrive_cluster(map_to_cta(smem_u32(&hdr->tmem_empty[acc]), 0));
                    else mbar_arrive(smem_u32(&hdr->tmem_empty[acc]));
                }
            }
            if (sample) continue;   // no lists, nothing to compact
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
                    unsigned m = __ballot_sync(0xffffffffu, q < p.s && cnt[q] >= p.soft);
                    while (m) {
                        const int b = __ffs(m) - 1;
                        m &= m - 1;
                        const int qq = base + ew * 32 + b;
                        tc_compact_query(my_cand + static_cast<size_t>(qq) * p.cap, thr, cnt, sorted, qq, p.k, p.cap, lane);
                    }
                }
                named_barrier(1, 128);  // thresholds and counts settled before the next unit's pushes
                tc_load_lane_thresholds(tl, thr, p.nb, p.nhalves, lane);
                if (l2) refresh_rhs();
            }
        }
        if (sample) {
            // ---- this warp's best rank value per query (-inf if it saw no row)
            float *dst = p.gmax + (static_cast<size_t>(blockIdx.x) * 4 + ew) * p.s_total + p.q_base;
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int j = 0; j < kTcMaxN / 32; ++j) {
                    const int q = h * p.nb + j * 32 + lane;
                    if (h < p.nhalves && j * 32 < p.nb && q < p.s &&
                        in_bounds((static_cast<long long>(blockIdx.x) * 4 + ew) * p.s_total + p.q_base + q, p.ext.aux, p.status))
                        dst[q] = !best[h][j] ? -INFINITY
                                 : l2    ? __fmaf_rd(0.0f - (1.0f + wide_slack), qnl[h][j], from_ordered_bits(best[h][j]))
                                         : from_ordered_bits(best[h][j]);
                }
        } else {
            // ---- CTA result: every list sorted and cut to k, written as this CTA's partial lists
            for (int base = 0; base < p.s; base += 128) {
                const int q0 = base + ew * 32;
                for (int b = 0; b < 32 && q0 + b < p.s; ++b) {
                    const int q = q0 + b;
                    uint64_t *list = my_cand + static_cast<size_t>(q) * p.cap;
                    if (cnt[q] != sorted[q]) tc_compact_query(list, thr, cnt, sorted, q, p.k, p.cap, lane);
                    const int n = cnt[q];
                    const long long first = (static_cast<long long>(blockIdx.x) * p.s_total + p.q_base + q) * p.k;
                    uint64_t *dst = p.partial + first;
                    for (int i = lane; i < p.k; i += 32)
                        if (in_bounds(first + i, p.ext.partial, p.status)) dst[i] = (i < n) ? list[i] : 0ull;
                }
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
