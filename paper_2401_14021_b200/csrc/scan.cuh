// Corpus scan for small query batches (8 queries per pass; 16 or 32 for larger inner-product
// batches, as groups of 8 that share every staged tile): scores every corpus
// row against every query and keeps, per CTA and query, the best k rows.
//
// One persistent CTA per SM. Warp 0 is the producer: one thread streams tiles of whole rows
// of the row-major corpus (a tile is one contiguous block of memory) into shared-memory
// stages with 1-D bulk copies that complete on mbarriers. The consumer warps take the tiles
// round-robin, each through a private ring of stages: wait for the tile, score it, hand the
// stage back, keep candidates.
//
// Two ways of scoring a tile:
//   FMA flavour: each lane holds its slice of every query in registers (fp32, packed
//     pairs), converts its slice of a row and issues packed fp32 FMAs; per-lane partial
//     sums are combined with a transposing shuffle reduction. Serves both metrics (L2 in
//     the direct sum-of-squared-differences form, which has no cancellation).
//   warp-MMA flavour: m16n8k16 tensor-core tiles with the 16 corpus rows as M and the (up
//     to) 8 queries as N, fp32 accumulators. The k index is permuted (the same way for rows
//     and queries) so that each lane reads 16 contiguous bytes per row. For L2 the rows'
//     squared norms come from the index (or, without one, from the tensor cores: diagonals
//     of rows x rows products) and |x|^2 - 2 x.q + |q|^2 serves as a conservative filter;
//     every pair that passes is scored again from the staged tile in the direct form, and
//     only that value is ranked and returned.
//
// Selection: k == 1 keeps a running best key per thread. k > 1 uses a per-query threshold
// (the current k-th best of this CTA, or a better bound handed in by the caller) and a
// candidate buffer, in shared memory or, when large, in global memory with one shared sort
// scratch. A push that lands beyond the buffer's soft limit raises a flag; every consumer warp
// polls the flag while it waits for a tile and all of them meet to compact (sort, keep k, raise
// the threshold) the buffers, spread over the warps, before any buffer can overflow: after the
// flag is up each warp pushes at most the rest of the tile it is on.
//
// A launch covers the rows [row_begin, N) and may start from given thresholds: on large corpora
// the host scans a sample first, merges it, and starts the main launch from the sample's k-th
// values, so that few rows pass.
#pragma once

#include "common.cuh"

namespace ralm {

constexpr int kMaxStages = 24;
constexpr int kMaxConsumerWarps = 8;
constexpr int kScanMaxQueries = 8;       // queries of one MMA group (the N of m16n8k16)
constexpr int kScanMaxPassQueries = 32;  // queries per pass: up to four groups in the inner-product warp-MMA flavour
constexpr int kScanThreads = 32 * (kMaxConsumerWarps + 1);
constexpr int kQueryPadBytes = 64;

struct ScanParams {
    const __half *corpus;
    const __half *queries;  // [s][d] of this pass
    const float *norms;     // warp-MMA L2 with NRM: squared norm of every corpus row, fp32 [N]
                            // (8-bit scan: the per-row bound of its filter)
    const uint8_t *x8;      // 8-bit scan: the one-byte copy of the corpus, [N][d]
    const float *sqnorms;   // 8-bit scan, L2: squared norm of every corpus row, fp32 [N]
    uint64_t *partial;      // [gridDim.x][s_total][k] sorted keys, 0 = empty
    uint64_t *spill;        // large k: candidate lists in global memory, [gridDim.x][8][cap]; the
                            // shared-memory candidate area then holds one sort scratch of cap keys
    int *status;
    long long N;        // rows of this launch end here (the whole corpus, or the end of a sample)
    long long row_begin;  // first row of this launch (a multiple of tile_rows)
    const float *thr_init;  // k > 1: [s_total] starting thresholds (rank values that k rows are
                            // known to reach), or null
    long long ntiles;   // tiles of this launch
    int d;
    int s;        // queries in this pass (<= 8)
    int s_total;  // queries of the whole call (layout of `partial`)
    int q_base;   // index of this pass's first query in the call
    int k;
    int cap;         // candidate buffer capacity per query (power of two); unused when k == 1
    int soft_limit;  // a push into a slot >= soft_limit asks for a compaction
    int tile_rows;   // rows per tile (16 for the warp-MMA flavour)
    int nwarps;      // consumer warps; warp w owns stages w, w + nwarps, ... (a private ring)
    int depth;       // stages per consumer warp
    int stage_bytes;
    int off_q;  // shared-memory offsets (bytes)
    int off_cand;
    int off_stage;
    float l2_slack;  // warp-MMA L2: filter slack per unit of (|x|^2 + |q|^2)
    // Large k: thresholds shared between the CTAs of a launch. After every compaction a CTA
    // publishes, per query, the rank value of its pub_rank-th best row (as order-preserving bits,
    // 0 = nothing yet) in pub[blockIdx.x * s_total + q_base + q]. pub_rank * gridDim.x >= k, the
    // CTAs' rows are disjoint, so the lowest published value of a query is reached by k different
    // rows, and every CTA may raise its threshold to it. Null: off.
    uint32_t *pub;
    int pub_rank;
    // Sample launch for large k (TOP1 instantiations only): instead of one best key per CTA and
    // query, every consumer warp writes the best rank value among ITS rows to
    // gmax[group * s_total + q_base + q] (-inf: it saw no row). The warps'
    // rows are disjoint, so the k-th largest of a query's maxima is reached by k different rows.
    // A warp keeps gmax_slots groups, taking its tiles in turn, so that a launch has
    // gridDim.x * nwarps * gmax_slots of them (large k needs many more groups than k for the
    // threshold to be tight): group (blockIdx.x * nwarps + warp) * gmax_slots + slot.
    // The bests live in shared memory at off_cand (nwarps x gmax_slots x 32 keys). Null: off.
    float *gmax;
    int gmax_slots;
    long long gmax_len;  // elements of gmax (debug build)
    Extents ext;     // extents of the global arrays, for the debug build's checks
};

struct ScanHeader {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    unsigned long long best[kScanMaxPassQueries];
    float thr[kScanMaxPassQueries];
    int cnt[kScanMaxPassQueries];
    int abort;
    int flag;  // some query's candidate buffer is nearly full: everyone meet and compact
    int done;  // consumer warps that have finished their tiles
};
constexpr int kScanHeaderBytes = 1024;
static_assert(sizeof(ScanHeader) <= kScanHeaderBytes, "header too large");

// Sort query q's candidates, keep the best k, raise the threshold. Called by a group of
// `nthr` threads with ranks `tid`, synchronised through group_sync(bar_id). With a scratch
// area the list (which then lives in global memory) is sorted there and its head copied back.
struct PubCtx {
    uint32_t *mine;   // this CTA's row of published values (indexed by the pass's query), or null
    int rank;         // which of its best rows a CTA publishes
};

__device__ inline void compact_query(ScanHeader *hdr, uint64_t *cand, uint64_t *scratch, int cap, int q,
                                     int k, int tid, int nthr, int bar_id, PubCtx pub = PubCtx{nullptr, 0}) {
    uint64_t *list = cand + static_cast<size_t>(q) * cap;
    uint64_t *a = scratch ? scratch : list;
    const int n = hdr->cnt[q] < cap ? hdr->cnt[q] : cap;  // (cap: see push_candidate)
    const int P = next_pow2(n > 1 ? n : 2);
    if (scratch) {
        for (int i = tid; i < P; i += nthr) a[i] = (i < n) ? list[i] : 0ull;
    } else {
        for (int i = n + tid; i < P; i += nthr) a[i] = 0;
    }
    group_sync(bar_id, nthr);
    bitonic_sort_desc(a, P, tid, nthr, bar_id);
    if (scratch) {
        const int keep = n < k ? n : k;
        for (int i = tid; i < keep; i += nthr) list[i] = a[i];
    }
    if (tid == 0) {
        hdr->cnt[q] = n < k ? n : k;
        // (never below a threshold taken over from the other CTAs)
        const float kth = (n >= k) ? key_value(a[k - 1]) : -INFINITY;
        hdr->thr[q] = fmaxf(hdr->thr[q], kth);
        if (pub.mine && n >= pub.rank)
            *reinterpret_cast<volatile uint32_t *>(pub.mine + q) = ordered_bits(key_value(a[pub.rank - 1]));
    }
    group_sync(bar_id, nthr);
}

// Large k: raise every query's threshold to the lowest value the CTAs of the launch have
// published for it (see ScanParams::pub), once all of them have published one. Called by one
// warp between the barriers of a compaction meeting.
__device__ inline void adopt_published_thresholds(ScanHeader *hdr, const uint32_t *pub, int nblocks, int s_total,
                                                  int q_base, int s, int lane) {
    for (int q = 0; q < s; ++q) {
        uint32_t lowest = 0xFFFFFFFFu;
        for (int c = lane; c < nblocks; c += 32) {
            const uint32_t v = __ldcg(pub + static_cast<size_t>(c) * s_total + q_base + q);
            lowest = v < lowest ? v : lowest;
        }
        lowest = __reduce_min_sync(0xffffffffu, lowest);
        if (lane == 0 && lowest != 0u) hdr->thr[q] = fmaxf(hdr->thr[q], from_ordered_bits(lowest));
    }
    __syncwarp();
}

// All W consumer warps (this one is w) compact every query that holds more than `min_count`
// candidates; the queries are spread over groups of warps that sort in parallel. Must be
// called by all W * 32 consumer threads, with no push in flight.
__device__ inline void compact_all(ScanHeader *hdr, uint64_t *cand, uint64_t *scratch, int cap, int s,
                                   int k, int min_count, int w, int lane, int W, PubCtx pub = PubCtx{nullptr, 0}) {
    int list[kScanMaxPassQueries];
    int nq = 0;
#pragma unroll
    for (int q = 0; q < kScanMaxPassQueries; ++q)
        if (q < s && hdr->cnt[q] > min_count) list[nq++] = q;
    // nobody may start rewriting cnt[] before everybody has taken the same snapshot of it
    named_barrier(1, W * 32);
    if (nq == 0) return;
    // one scratch area: one group, the queries one after the other
    const int ngroups = scratch ? 1 : (nq < W ? nq : W);
    const int G = W / ngroups;  // warps per group
    const int group = w / G;
    if (group >= ngroups) return;
    const int tid = (w - group * G) * 32 + lane;
    const int bar_id = (G == 1) ? -2 : 2 + group;
    for (int i = group; i < nq; i += ngroups) {
        int q = 0;
#pragma unroll
        for (int j = 0; j < kScanMaxPassQueries; ++j)
            if (j == i) q = list[j];
        compact_query(hdr, cand, scratch, cap, q, k, tid, G * 32, bar_id, pub);
    }
}

// The meeting itself: barrier, compact, lower the flag, barrier.
__device__ __forceinline__ void compaction_meeting(ScanHeader *hdr, uint64_t *cand, uint64_t *scratch,
                                                   const int cap, const int s, const int k, int w,
                                                   int lane, int W, const ScanParams &p) {
    named_barrier(1, W * 32);
    PubCtx pub{p.pub ? p.pub + static_cast<size_t>(blockIdx.x) * p.s_total + p.q_base : nullptr, p.pub_rank};
    // (with shared thresholds every list that can already publish is sorted, not only the full ones)
    compact_all(hdr, cand, scratch, cap, s, k, p.pub ? p.pub_rank - 1 : k, w, lane, W, pub);
    if (p.pub) {
        named_barrier(1, W * 32);   // every compaction of this meeting has written its threshold
        if (w == 0) adopt_published_thresholds(hdr, p.pub, gridDim.x, p.s_total, p.q_base, s, lane);
    }
    if (w == 0 && lane == 0) *reinterpret_cast<volatile int *>(&hdr->flag) = 0;
    named_barrier(1, W * 32);
}

// FMA flavour: transposing shuffle reduction. On entry every lane holds V partial sums
// (V = 16); on exit a[0] of lanes 2v and 2v+1 is the full sum of value index v.
template <int V>
__device__ __forceinline__ void transpose_reduce(float (&a)[V], int lane) {
    int off = 16;
#pragma unroll
    for (int n = V; n > 1; n >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float keep = upper ? a[i + n / 2] : a[i];
            const float send = upper ? a[i] : a[i + n / 2];
            a[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
        off >>= 1;
    }
#pragma unroll
    for (int o = 16 / V; o > 0; o >>= 1) a[0] += __shfl_xor_sync(0xffffffffu, a[0], o);
}

// Shared-memory banks, warp-MMA flavour: a lane reads 16 bytes of two rows per step and the
// lanes of a quarter warp hold two different rows, which collide when a row is a multiple of 128
// bytes long (768 and 1024 dimensions both are). So a tile is staged as two copies of 8 rows,
// the second shifted by kTileShiftBytes, and MMA row m takes its data from staged row
// staged_row(m), which alternates between the two groups (rows m and m + 1 then sit 64 bytes
// apart modulo 128).
constexpr int kTileShiftBytes = 64;
__host__ __device__ __forceinline__ int staged_row(int m) {
    return ((m & 1) << 3) + ((m & 8) >> 1) + ((m & 7) >> 1);
}
__host__ __device__ __forceinline__ int staged_row_offset(int row, int row_bytes) {
    return row * row_bytes + ((row & 8) ? kTileShiftBytes : 0);
}

__device__ __forceinline__ void mma_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                             uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr));
    return v;
}

__device__ __forceinline__ float2 h2_to_f2(uint32_t h2) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&h2));
}

// The host sizes the lists so that slot < cap always holds (every warp pushes at most the rest of
// its tile after the flag is up). Should that ever fail, the key is dropped and the status word
// says so, rather than writing into the neighbouring list.
__device__ __forceinline__ void push_candidate(ScanHeader *hdr, uint64_t *cand, int cap, int soft,
                                               int q, uint64_t key, int *status, long long list_room = 1LL << 62) {
    const int slot = atomicAdd(&hdr->cnt[q], 1);
    // (list_room: keys between `cand` and the end of the global list array; debug build only)
    if (slot < cap && in_bounds(static_cast<long long>(q) * cap + slot, list_room, status))
        cand[static_cast<size_t>(q) * cap + slot] = key;
    else atomicMax(status, kStatusInternal);
    if (slot >= soft) *reinterpret_cast<volatile int *>(&hdr->flag) = 1;
}


// Warp-MMA L2 flavour, exact part: squared distance between one staged corpus row and one
// query (both fp16 in shared memory), computed by the whole warp in the direct
// sum-of-squared-differences form (no cancellation). Every lane returns the full sum.
__device__ __forceinline__ float warp_direct_l2(uint32_t row_addr, uint32_t q_addr, int d, int lane) {
    float2 sum = make_float2(0.f, 0.f);
    for (int piece = lane; piece * 8 < d; piece += 32) {
        const uint4 xr = lds128(row_addr + piece * 16);
        const uint4 qr = lds128(q_addr + piece * 16);
        const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
        const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 x = h2_to_f2(xw[e]), q = h2_to_f2(qw[e]);
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

// ------------------------------------------------------------------------------------
// The kernel. MMA: warp-MMA flavour or FMA flavour. L2: metric (the warp-MMA flavour uses
// the tensor-core value of |x|^2 - 2 x.q + |q|^2 as a filter and ranks the direct form). SQ: queries held per lane (1 or 4; FMA flavour).
// DP: 16-byte pieces of a row per lane (d <= 256 * DP; FMA flavour). TOP1: k == 1.
// NRM (warp-MMA L2): the rows' squared norms come from p.norms instead of extra MMAs.
// ------------------------------------------------------------------------------------
template <bool MMA, bool L2, int SQ, int DP, bool TOP1, bool NRM = false>
__global__ void __launch_bounds__(MMA ? kScanThreads : kScanThreads - 32, 1)
scan_kernel(const ScanParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    ScanHeader *hdr = reinterpret_cast<ScanHeader *>(smem);
    uint64_t *scratch = p.spill ? reinterpret_cast<uint64_t *>(smem + p.off_cand) : nullptr;
    uint64_t *cand = p.spill ? p.spill + static_cast<size_t>(blockIdx.x) * kScanMaxPassQueries * p.cap
                             : reinterpret_cast<uint64_t *>(smem + p.off_cand);
    const long long list_room = p.spill ? p.ext.lists - static_cast<long long>(blockIdx.x) * kScanMaxPassQueries * p.cap
                                        : 1LL << 62;
    const int W = p.nwarps;
    const int S = W * p.depth;
    const int T = p.tile_rows;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int d = p.d;

    if (threadIdx.x == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(smem_u32(&hdr->full[i]), 1);
            mbar_init(smem_u32(&hdr->empty[i]), 1);
        }
        mbar_fence_init();
        hdr->abort = 0;
        hdr->flag = 0;
        hdr->done = 0;
    }
    if (threadIdx.x < kScanMaxPassQueries) {
        hdr->thr[threadIdx.x] = (p.thr_init && threadIdx.x < p.s) ? p.thr_init[p.q_base + threadIdx.x] : -INFINITY;
        hdr->cnt[threadIdx.x] = 0;
        hdr->best[threadIdx.x] = 0ull;
    }
    if (TOP1 && p.gmax)
        for (int i = threadIdx.x; i < p.nwarps * p.gmax_slots * kScanMaxPassQueries; i += blockDim.x)
            reinterpret_cast<unsigned long long *>(smem + p.off_cand)[i] = 0ull;
    if (MMA) {
        // queries as fp16 [8][d] in shared memory, rows >= s zeroed; rows are padded by
        // kQueryPadBytes so that the eight query rows do not all start on the same bank
        const uint4 *qg = reinterpret_cast<const uint4 *>(p.queries);
        const int per_row = d / 8;
        for (int i = threadIdx.x; i < (MMA ? SQ : kScanMaxQueries) * per_row; i += blockDim.x) {
            const int row = i / per_row, col = i - row * per_row;
            *reinterpret_cast<uint4 *>(smem + p.off_q + row * (d * 2 + kQueryPadBytes) + col * 16) =
                (row < p.s) ? qg[i] : make_uint4(0, 0, 0, 0);
        }
    }
    __syncthreads();

    const long long my_tiles =
        (p.ntiles > blockIdx.x) ? (p.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    volatile int *abort_flag = &hdr->abort;
    volatile int *compact_flag = &hdr->flag;
    volatile int *done_count = &hdr->done;

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        // All 32 lanes run the loop (waits, counters and addresses stay warp-uniform); one elected
        // lane issues the copies.
        uint32_t elected;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "elect.sync _|p, 0xffffffff;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(elected));
        long long issued = 0;
        bool ok = true;
        // tile `it` belongs to consumer warp cw = it % W; it is that warp's (it / W)-th
        // tile and goes to slot (it / W) % depth of the warp's private ring, for the
        // use-th time. The counters advance incrementally: no division on this path.
        int cw = 0, slot = 0;
        uint32_t use = 0;
        long long row0 = p.row_begin + static_cast<long long>(blockIdx.x) * T;
        const long long row_step = static_cast<long long>(gridDim.x) * T;
        const uint32_t stage_base = smem_u32(smem + p.off_stage);
        const uint32_t row_bytes = static_cast<uint32_t>(d * 2);
        for (long long it = 0; it < my_tiles; ++it) {
            const int st = cw + slot * W;
            if (use > 0) {
                const uint32_t ebar = smem_u32(&hdr->empty[st]);
                if (!mbar_try_wait(ebar, (use - 1) & 1)) ok = mbar_wait_bounded(ebar, (use - 1) & 1);
                if (!ok) break;
            }
            if (*abort_flag) break;
            if (elected) {
                const long long rows = (p.N - row0 < T) ? (p.N - row0) : T;
                const uint32_t bytes = static_cast<uint32_t>(rows) * row_bytes;
                const uint32_t bar = smem_u32(&hdr->full[st]);
                const uint32_t dst = stage_base + static_cast<uint32_t>(st) * p.stage_bytes;
                const long long src_row = in_bounds(row0 + rows - 1, p.ext.rows, p.status) ? row0 : 0;
                mbar_arrive_expect_tx(bar, bytes);
                if (MMA) {
                    // rows 0..7 and rows 8..15 as two copies, the second kTileShiftBytes further
                    const uint32_t first = rows < 8 ? bytes : 8u * row_bytes;
                    bulk_load(dst, p.corpus + src_row * d, first, bar);
                    if (bytes > first)
                        bulk_load(dst + first + kTileShiftBytes, p.corpus + (src_row + 8) * d, bytes - first, bar);
                } else {
                    bulk_load(dst, p.corpus + src_row * d, bytes, bar);
                }
            }
            issued = it + 1;
            row0 += row_step;
            if (++cw == W) {
                cw = 0;
                if (++slot == p.depth) {
                    slot = 0;
                    ++use;
                }
            }
        }
        if (!ok && lane == 0) {
            atomicMax(p.status, kStatusTimeout);
            *abort_flag = 1;
        }
        __syncwarp();
        if (*abort_flag) {
            // winding down early: let every copy already issued land before exit
            for (long long it = (issued > S ? issued - S : 0); it < issued; ++it) {
                const long long local = it / W;
                mbar_wait_bounded(smem_u32(&hdr->full[(it % W) + (local % p.depth) * W]),
                                  (local / p.depth) & 1);
            }
        }
    } else if (warp - 1 < W) {
        // ---------------------------------------------------------------- consumers
        const int w = warp - 1;
        const int ctid = threadIdx.x - 32;
        const int cthreads = W * 32;
        const int g = lane >> 2, t = lane & 3;

        // warp-MMA flavour: SQ / 8 groups of 8 queries share every tile
        constexpr int NG = MMA ? SQ / 8 : 1;
        uint64_t bestA[NG], bestB[NG];
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) bestA[grp] = bestB[grp] = 0;
        // FMA flavour: this lane's slice of every query as fp32 pairs (negated for L2 so
        // that the difference is one packed add)
        constexpr int DPR = MMA ? 1 : DP;
        constexpr int SQR = MMA ? 1 : SQ;
        float2 qreg[SQR][DPR][4];
        if (!MMA) {
#pragma unroll
            for (int j = 0; j < SQR; ++j)
#pragma unroll
                for (int i = 0; i < DPR; ++i) {
                    const int piece = lane + 32 * i;
                    uint4 raw = make_uint4(0, 0, 0, 0);
                    if (j < p.s && piece * 8 < d)
                        raw = *reinterpret_cast<const uint4 *>(p.queries +
                                                               static_cast<size_t>(j) * d + piece * 8);
                    const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float2 v = h2_to_f2(words[e]);
                        if (L2) {
                            v.x = -v.x;
                            v.y = -v.y;
                        }
                        qreg[j][i][e] = v;
                    }
                }
        }

        // warp-MMA flavour: where the queries sit in shared memory; for L2 also the squared
        // norms of this lane's two queries (2t, 2t+1), summed in fp32
        const uint32_t q_pitch = static_cast<uint32_t>(d * 2 + kQueryPadBytes);
        const uint32_t q_base_addr = smem_u32(smem + p.off_q);
        float qn0[NG], qn1[NG];
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) {
            qn0[grp] = qn1[grp] = 0.f;
            if (MMA && L2) {
                const int row_a = grp * kScanMaxQueries + 2 * t;
                const __half *qa = reinterpret_cast<const __half *>(smem + p.off_q + row_a * q_pitch);
                const __half *qb = reinterpret_cast<const __half *>(smem + p.off_q + (row_a + 1) * q_pitch);
                for (int i = 0; i < d; ++i) {
                    const float a = __half2float(qa[i]), b = __half2float(qb[i]);
                    qn0[grp] = fmaf(a, a, qn0[grp]);
                    qn1[grp] = fmaf(b, b, qn1[grp]);
                }
            }
        }

        const int ph_lo = staged_row(g), ph_hi = staged_row(g + 8);
        // k == 1: where the best key of every query is kept: the CTA's, or (sample launch for large
        // k, see ScanParams::gmax) this warp's own
        unsigned long long *const warp_bests =
            reinterpret_cast<unsigned long long *>(smem + p.off_cand) + w * p.gmax_slots * kScanMaxPassQueries;
        unsigned long long *bestq = (TOP1 && p.gmax) ? warp_bests : hdr->best;
        int gslot = 0;
        int slot = 0;         // position in this warp's private ring
        uint32_t parity = 0;  // phase parity of the ring's current lap
        long long row0 =
            p.row_begin + (static_cast<long long>(blockIdx.x) + static_cast<long long>(w) * gridDim.x) * T;
        const long long row_step = static_cast<long long>(gridDim.x) * W * T;
        // shared thresholds (large k): lists fill too slowly to call meetings by themselves, so the
        // first consumer warp calls one after 64, 128, 256, ... of its tiles
        long long tiles_done = 0, next_meeting = 64;
        for (long long it = w; it < my_tiles; it += W, row0 += row_step) {
            if (*abort_flag) continue;
            if (!TOP1 && p.pub && w == 0 && ++tiles_done == next_meeting) {
                next_meeting *= 2;
                if (lane == 0) *compact_flag = 1;
            }
            // this warp's private ring: only this warp ever waits on these stages, in order,
            // so a parity wait can never be satisfied by an older phase
            const int st = w + slot * W;
            const uint32_t full_bar = smem_u32(&hdr->full[st]);
            const uint32_t my_parity = parity;
            // (MMA rows g and g + 8 are the tile's rows ph_lo and ph_hi: see staged_row)
            float pn_lo = 0.f, pn_hi = 0.f;  // stored norms of those rows, in flight during the wait
            if (MMA && L2 && NRM) {
                if (row0 + ph_lo < p.N && in_bounds(row0 + ph_lo, p.ext.rows, p.status)) pn_lo = __ldg(p.norms + row0 + ph_lo);
                if (row0 + ph_hi < p.N && in_bounds(row0 + ph_hi, p.ext.rows, p.status)) pn_hi = __ldg(p.norms + row0 + ph_hi);
            }
            if (++slot == p.depth) {
                slot = 0;
                parity ^= 1;
            }
            // Wait for the tile. Lane 0 polls; a raised compaction flag takes priority over a
            // ready tile (after the flag is up a warp finishes at most the tile it is on), and
            // a warp still waiting for its tile joins the meeting instead of blocking it.
            bool have_tile = false;
            {
                const long long t0 = clock64();
                int spins = 0;
                while (!have_tile) {
                    int state = 0;  // 1 tile ready, 2 compaction requested, 3 gave up
                    if (lane == 0) {
                        if (!TOP1 && *compact_flag) state = 2;
                        else if (mbar_try_wait(full_bar, my_parity)) state = 1;
                        else if ((++spins & 1023) == 0 && clock64() - t0 > kWaitCycleLimit) state = 3;
                    }
                    state = __shfl_sync(0xffffffffu, state, 0);
                    if (state == 1) {
                        while (!mbar_try_wait(full_bar, my_parity)) {}  // completed: returns at once
                        have_tile = true;
                    } else if (state == 2) {
                        compaction_meeting(hdr, cand, scratch, p.cap, p.s, p.k, w, lane, W, p);
                    } else if (state == 3) {
                        if (lane == 0) {
                            atomicMax(p.status, kStatusTimeout);
                            *abort_flag = 1;
                        }
                        break;
                    }
                }
            }
            if (!have_tile) continue;
            const uint32_t stage_addr =
                smem_u32(smem + p.off_stage + static_cast<size_t>(st) * p.stage_bytes);
            const uint32_t empty_bar = smem_u32(&hdr->empty[st]);
            if (TOP1 && p.gmax) {
                // sample launch by maxima: this tile's rows count for the warp's next group
                if (MMA) {
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        const int gq = grp * kScanMaxQueries + 2 * t;
                        if (bestA[grp]) atomicMax(&bestq[gq], static_cast<unsigned long long>(bestA[grp]));
                        if (bestB[grp]) atomicMax(&bestq[gq + 1], static_cast<unsigned long long>(bestB[grp]));
                        bestA[grp] = bestB[grp] = 0;
                    }
                }
                __syncwarp();
                bestq = warp_bests + gslot * kScanMaxPassQueries;
                if (++gslot == p.gmax_slots) gslot = 0;
            }
            if (MMA) {
                // ---- 16 rows x 8 queries on tensor cores; two accumulator sets halve the
                // dependent chain. For L2 two more products per step, rows x rows, put the
                // rows' squared norms on the diagonals of nlo (rows 0..7) and nhi (rows 8..15).
                float acc[NG][4], acc_b[NG][4];
#pragma unroll
                for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[grp][i] = acc_b[grp][i] = 0.f;
                float nlo[4] = {0.f, 0.f, 0.f, 0.f}, nlo_b[4] = {0.f, 0.f, 0.f, 0.f};
                float nhi[4] = {0.f, 0.f, 0.f, 0.f}, nhi_b[4] = {0.f, 0.f, 0.f, 0.f};
                const int nchunks = (d + 31) >> 5;
                const uint32_t q_addr = q_base_addr + g * q_pitch;
                const uint32_t a_lo_addr = stage_addr + staged_row_offset(ph_lo, d * 2);
                const uint32_t a_hi_addr = stage_addr + staged_row_offset(ph_hi, d * 2);
#pragma unroll 4
                for (int c = 0; c < nchunks; ++c) {
                    // logical k (2t, 2t+1, 2t+8, 2t+9 of two MMAs) <- physical halves
                    // off..off+7, the same permutation for every row and query
                    const int off = c * 32 + t * 8;
                    uint4 lo = make_uint4(0, 0, 0, 0), hi = lo;
                    if (off < d) {  // ragged last chunk: absent pieces stay zero
                        lo = lds128(a_lo_addr + off * 2);
                        hi = lds128(a_hi_addr + off * 2);
                    }
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        uint4 b = make_uint4(0, 0, 0, 0);
                        if (off < d) b = lds128(q_addr + grp * kScanMaxQueries * q_pitch + off * 2);
                        mma_m16n8k16(acc[grp], lo.x, hi.x, lo.y, hi.y, b.x, b.y);
                        mma_m16n8k16(acc_b[grp], lo.z, hi.z, lo.w, hi.w, b.z, b.w);
                    }
                    if (L2 && !NRM) {
                        mma_m16n8k16(nlo, lo.x, hi.x, lo.y, hi.y, lo.x, lo.y);
                        mma_m16n8k16(nhi, lo.x, hi.x, lo.y, hi.y, hi.x, hi.y);
                        mma_m16n8k16(nlo_b, lo.z, hi.z, lo.w, hi.w, lo.z, lo.w);
                        mma_m16n8k16(nhi_b, lo.z, hi.z, lo.w, hi.w, hi.z, hi.w);
                    }
                }
#pragma unroll
                for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[grp][i] += acc_b[grp][i];
                if (!L2) {  // the L2 flavour still needs the rows: it hands the stage back below
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar);
                }
                // acc[0]: (row g, query 2t)     acc[1]: (row g, query 2t+1)
                // acc[2]: (row g+8, query 2t)   acc[3]: (row g+8, query 2t+1)
                const long long r_lo = row0 + ph_lo, r_hi = row0 + ph_hi;
                const int q0 = 2 * t;  // this lane's first query within a group; the second is q0 + 1
                if (L2) {
                    // |x|^2 - 2 x.q + |q|^2 from the tensor cores is only a FILTER (it cancels):
                    // a pair passes when it could still beat the threshold given the slack that
                    // bounds the filter's rounding error, and is then scored again in the direct
                    // form, which is the value that is ranked and returned.
                    float n_lo = pn_lo, n_hi = pn_hi;
                    if (!NRM) {
                        // the diagonal entry of row g (and g + 8) is held by the lane with t == g / 2
                        const float d_lo = (g & 1) ? (nlo[1] + nlo_b[1]) : (nlo[0] + nlo_b[0]);
                        const float d_hi = (g & 1) ? (nhi[3] + nhi_b[3]) : (nhi[2] + nhi_b[2]);
                        const int diag_lane = (lane & ~3) | (g >> 1);
                        n_lo = __shfl_sync(0xffffffffu, d_lo, diag_lane);
                        n_hi = __shfl_sync(0xffffffffu, d_hi, diag_lane);
                    }
                    const float sl = p.l2_slack;
                    if (TOP1 && p.gmax) {
                        // Sample launch by maxima: the filter value minus its slack is a LOWER bound
                        // of the rank value the direct form would give, and a threshold only has to
                        // be a value that k different rows are known to reach. So nothing is scored
                        // again here: the warp keeps the best lower bound per query and group (the
                        // slack is widened a little to cover the rounding of these few operations).
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty_bar);
                        const float ws = fmaf(sl, 1.001f, 9.5367431640625e-7f);
#pragma unroll
                        for (int grp = 0; grp < NG; ++grp) {
                            const float a0 = qn0[grp], a1 = qn1[grp];
                            if (r_lo < p.N) {
                                const uint64_t k0 = make_key(fmaf(-ws, n_lo + a0, (2.f * acc[grp][0] - n_lo) - a0), static_cast<uint32_t>(r_lo));
                                const uint64_t k1 = make_key(fmaf(-ws, n_lo + a1, (2.f * acc[grp][1] - n_lo) - a1), static_cast<uint32_t>(r_lo));
                                bestA[grp] = k0 > bestA[grp] ? k0 : bestA[grp];
                                bestB[grp] = k1 > bestB[grp] ? k1 : bestB[grp];
                            }
                            if (r_hi < p.N) {
                                const uint64_t k0 = make_key(fmaf(-ws, n_hi + a0, (2.f * acc[grp][2] - n_hi) - a0), static_cast<uint32_t>(r_hi));
                                const uint64_t k1 = make_key(fmaf(-ws, n_hi + a1, (2.f * acc[grp][3] - n_hi) - a1), static_cast<uint32_t>(r_hi));
                                bestA[grp] = k0 > bestA[grp] ? k0 : bestA[grp];
                                bestB[grp] = k1 > bestB[grp] ? k1 : bestB[grp];
                            }
                        }
                    } else {
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        const int gq0 = grp * kScanMaxQueries + q0, gq1 = gq0 + 1;
                        float th0, th1;
                        if (TOP1) {
                            const unsigned long long b0 = *reinterpret_cast<volatile unsigned long long *>(&bestq[gq0]);
                            const unsigned long long b1 = *reinterpret_cast<volatile unsigned long long *>(&bestq[gq1]);
                            th0 = b0 ? key_value(b0) : -INFINITY;
                            th1 = b1 ? key_value(b1) : -INFINITY;
                        } else {
                            th0 = *reinterpret_cast<volatile float *>(&hdr->thr[gq0]);
                            th1 = *reinterpret_cast<volatile float *>(&hdr->thr[gq1]);
                        }
                        const float a0 = qn0[grp], a1 = qn1[grp];
                        bool pass[4];
                        pass[0] = r_lo < p.N && gq0 < p.s && (2.f * acc[grp][0] - n_lo - a0) + sl * (n_lo + a0) >= th0;
                        pass[1] = r_lo < p.N && gq1 < p.s && (2.f * acc[grp][1] - n_lo - a1) + sl * (n_lo + a1) >= th1;
                        pass[2] = r_hi < p.N && gq0 < p.s && (2.f * acc[grp][2] - n_hi - a0) + sl * (n_hi + a0) >= th0;
                        pass[3] = r_hi < p.N && gq1 < p.s && (2.f * acc[grp][3] - n_hi - a1) + sl * (n_hi + a1) >= th1;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            unsigned m = __ballot_sync(0xffffffffu, pass[i]);
                            while (m) {
                                const int src = __ffs(m) - 1;
                                m &= m - 1;
                                const int row_local = staged_row((src >> 2) + ((i & 2) ? 8 : 0));
                                const int q = grp * kScanMaxQueries + 2 * (src & 3) + (i & 1);
                                const float dist = warp_direct_l2(stage_addr + staged_row_offset(row_local, d * 2),
                                                                  q_base_addr + q * q_pitch, d, lane);
                                if (lane == 0) {
                                    const float val = 0.0f - dist;
                                    const uint64_t key = make_key(val, static_cast<uint32_t>(row0 + row_local));
                                    if (TOP1) {
                                        atomicMax(&bestq[q], static_cast<unsigned long long>(key));
                                    } else if (val >= *reinterpret_cast<volatile float *>(&hdr->thr[q])) {
                                        push_candidate(hdr, cand, p.cap, p.soft_limit, q, key, p.status, list_room);
                                    }
                                }
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar);
                    }
                } else {
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) {
                    const int gq0 = grp * kScanMaxQueries + q0, gq1 = gq0 + 1;
                    if (TOP1) {
                        if (r_lo < p.N) {
                            const uint64_t k0 = make_key(acc[grp][0], static_cast<uint32_t>(r_lo));
                            const uint64_t k1 = make_key(acc[grp][1], static_cast<uint32_t>(r_lo));
                            bestA[grp] = k0 > bestA[grp] ? k0 : bestA[grp];
                            bestB[grp] = k1 > bestB[grp] ? k1 : bestB[grp];
                        }
                        if (r_hi < p.N) {
                            const uint64_t k0 = make_key(acc[grp][2], static_cast<uint32_t>(r_hi));
                            const uint64_t k1 = make_key(acc[grp][3], static_cast<uint32_t>(r_hi));
                            bestA[grp] = k0 > bestA[grp] ? k0 : bestA[grp];
                            bestB[grp] = k1 > bestB[grp] ? k1 : bestB[grp];
                        }
                    } else {
                        const float th0 = hdr->thr[gq0], th1 = hdr->thr[gq1];
                        if (r_lo < p.N) {
                            if (gq0 < p.s && acc[grp][0] >= th0)
                                push_candidate(hdr, cand, p.cap, p.soft_limit, gq0,
                                               make_key(acc[grp][0], static_cast<uint32_t>(r_lo)), p.status, list_room);
                            if (gq1 < p.s && acc[grp][1] >= th1)
                                push_candidate(hdr, cand, p.cap, p.soft_limit, gq1,
                                               make_key(acc[grp][1], static_cast<uint32_t>(r_lo)), p.status, list_room);
                        }
                        if (r_hi < p.N) {
                            if (gq0 < p.s && acc[grp][2] >= th0)
                                push_candidate(hdr, cand, p.cap, p.soft_limit, gq0,
                                               make_key(acc[grp][2], static_cast<uint32_t>(r_hi)), p.status, list_room);
                            if (gq1 < p.s && acc[grp][3] >= th1)
                                push_candidate(hdr, cand, p.cap, p.soft_limit, gq1,
                                               make_key(acc[grp][3], static_cast<uint32_t>(r_hi)), p.status, list_room);
                        }
                    }
                }
                }
            } else {
                // ---- FMA flavour: RG rows at a time, RG * SQ = 16 partial sums
                constexpr int RG = 16 / SQR;
                constexpr int V = 16;
#pragma unroll 1
                for (int rg = 0; rg < T; rg += RG) {
                    float2 acc2[RG][SQR];
#pragma unroll
                    for (int r = 0; r < RG; ++r)
#pragma unroll
                        for (int jq = 0; jq < SQR; ++jq) acc2[r][jq] = make_float2(0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < DPR; ++i) {
                        const int piece = lane + 32 * i;
                        if (piece * 8 < d) {
#pragma unroll
                            for (int r = 0; r < RG; ++r) {
                                const uint4 raw = lds128(stage_addr + ((rg + r) * d + piece * 8) * 2);
                                const uint32_t words[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float2 x = h2_to_f2(words[e]);
#pragma unroll
                                    for (int jq = 0; jq < SQR; ++jq) {
                                        if (L2) {
                                            const float2 df = __fadd2_rn(x, qreg[jq][i][e]);
                                            acc2[r][jq] = __ffma2_rn(df, df, acc2[r][jq]);
                                        } else {
                                            acc2[r][jq] = __ffma2_rn(x, qreg[jq][i][e], acc2[r][jq]);
                                        }
                                    }
                                }
                            }
                        }
                    }
                    if (rg + RG >= T) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty_bar);
                    }
                    float a[V];
#pragma unroll
                    for (int r = 0; r < RG; ++r)
#pragma unroll
                        for (int jq = 0; jq < SQR; ++jq) a[r * SQR + jq] = acc2[r][jq].x + acc2[r][jq].y;
                    transpose_reduce<V>(a, lane);
                    // lanes 2v and 2v+1 hold value v = r * SQ + jq
                    const int v = lane >> 1;
                    const int r = v / SQR, jq = v % SQR;
                    const long long row = row0 + rg + r;
                    const float val = L2 ? (0.0f - a[0]) : a[0];
                    if ((lane & 1) == 0 && row < p.N && jq < p.s) {
                        if (TOP1) {
                            const uint64_t key = make_key(val, static_cast<uint32_t>(row));
                            bestA[0] = key > bestA[0] ? key : bestA[0];
                        } else if (val >= hdr->thr[jq]) {
                            push_candidate(hdr, cand, p.cap, p.soft_limit, jq,
                                           make_key(val, static_cast<uint32_t>(row)), p.status, list_room);
                        }
                    }
                }
            }
        }

        // ------------------------------------------------------------ CTA result
        if (TOP1) {
            if (MMA) {
                // (the L2 flavour of a main launch has put its keys into hdr->best as it went)
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) {
                    const int gq = grp * kScanMaxQueries + 2 * t;
                    if (bestA[grp]) atomicMax(&bestq[gq], static_cast<unsigned long long>(bestA[grp]));
                    if (bestB[grp]) atomicMax(&bestq[gq + 1], static_cast<unsigned long long>(bestB[grp]));
                }
            } else {
                const int jq = (lane >> 1) % SQR;
                if (bestA[0]) atomicMax(&bestq[jq], static_cast<unsigned long long>(bestA[0]));
            }
            if (p.gmax) {
                // this warp's maxima, group by group (lane q writes query q's)
                __syncwarp();
                for (int sl = 0; sl < p.gmax_slots; ++sl) {
                    const unsigned long long best = warp_bests[sl * kScanMaxPassQueries + lane];
                    const long long at = ((static_cast<long long>(blockIdx.x) * W + w) * p.gmax_slots + sl) * p.s_total +
                                         p.q_base + lane;
                    if (lane < p.s && in_bounds(at, p.gmax_len, p.status)) p.gmax[at] = best ? key_value(best) : -INFINITY;
                }
            } else {
                named_barrier(1, cthreads);
                if (ctid < p.s && in_bounds(static_cast<long long>(blockIdx.x) * p.s_total + p.q_base + ctid, p.ext.partial, p.status))
                    p.partial[static_cast<size_t>(blockIdx.x) * p.s_total + p.q_base + ctid] =
                        hdr->best[ctid];
            }
        } else {
            // this warp is out of tiles; keep answering compaction calls until every warp is
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                atomicAdd(&hdr->done, 1);
            }
            for (;;) {
                int state = 0;  // 1: compaction requested, 2: everybody finished
                if (lane == 0) {
                    if (*compact_flag) {
                        state = 1;
                    } else if (*done_count >= W) {
                        // the flag is raised before `done` is incremented: look again
                        __threadfence_block();
                        state = *compact_flag ? 1 : 2;
                    }
                }
                state = __shfl_sync(0xffffffffu, state, 0);
                if (state == 1) compaction_meeting(hdr, cand, scratch, p.cap, p.s, p.k, w, lane, W, p);
                else if (state == 2) break;
            }
            named_barrier(1, cthreads);
            compact_all(hdr, cand, scratch, p.cap, p.s, p.k, 0, w, lane, W);
            named_barrier(1, cthreads);
            for (int q = 0; q < p.s; ++q) {
                const int n = hdr->cnt[q];
                const long long first = (static_cast<long long>(blockIdx.x) * p.s_total + p.q_base + q) * p.k;
                uint64_t *dst = p.partial + first;
                for (int i = ctid; i < p.k; i += cthreads)
                    if (in_bounds(first + i, p.ext.partial, p.status))
                        dst[i] = (i < n) ? cand[static_cast<size_t>(q) * p.cap + i] : 0ull;
            }
        }
    }
}

}  // namespace ralm
