// Inner-product corpus scan over an 8-bit copy of the corpus, with exact results.
//
// The small-batch scan is bound by the bytes of the corpus it streams. This variant streams a
// one-byte-per-element copy instead (E5M2: the upper byte of the fp16 value after rounding to
// two mantissa bits, so a byte becomes an fp16 operand by placing it in the upper half of a
// 16-bit lane) and uses the tensor-core score of the rounded row only as a FILTER:
//
//     |q.x - q.x8| <= |q| |x - x8|                      (Cauchy-Schwarz)
//
// so with e_j >= |x_j - x8_j| + (rounding slack of the fp32 accumulation) stored per row,
// U = q.x8_j + |q| e_j is an upper bound of the true score. A (row, query) pair whose U cannot
// reach the query's threshold (a score that k rows are already known to reach exactly) is
// dropped; every pair that passes is scored again by the whole warp from the fp16 row in
// global memory, and only that value is compared, kept and returned. The result is therefore
// the same as the fp16 scan's, at half the streamed bytes plus the rows that pass.
//
// Shared-memory banks: a lane reads 16 bytes of two rows per step, and the lanes of a quarter
// warp hold two different rows, which collide when d is a multiple of 128 bytes. So a tile is
// staged as two copies of 8 rows, the second shifted by 64 bytes, and MMA row m takes its data
// from staged row q8_phys_row(m), which alternates between the two groups; the staged queries
// get a pitch of 16 bytes modulo 128 for the same reason.
//
// L2 (squared distance) uses the same filter on x.q: with the rows' stored squared norms,
//     -|x - q|^2 = 2 x.q - |x|^2 - |q|^2 <= 2 (q.x8 + |q| e_j) - |x|^2 - |q|^2
// (plus the slack that bounds the rounding of the stored norms, as in the fp16 L2 scan), and a
// pair that passes is scored again in the direct sum-of-squared-differences form from the fp16
// row, which is the only value ranked and returned.
//
// Structure (producer warp, private stage rings per consumer warp, candidate buffers, compaction
// meetings) is that of scan_kernel; the tile is 16 rows of d bytes. The host starts this kernel
// from the thresholds of an fp16 scan of a small sample, without which nearly every pair would
// pass until the lists fill.
#pragma once

#include "scan.cuh"

namespace ralm {

// staged row (0..15, rows 8..15 sit 64 bytes further) that feeds MMA row m
__host__ __device__ __forceinline__ int q8_phys_row(int m) {
    return ((m & 1) << 3) + ((m & 8) >> 1) + ((m & 7) >> 1);
}
__host__ __device__ __forceinline__ int q8_row_offset(int phys_row, int d) {
    return phys_row * d + ((phys_row & 8) << 3);
}
// bytes between staged queries: 2 d rounded up to 16 modulo 128
__host__ __device__ __forceinline__ int q8_query_pitch(int d) { return 2 * d + (144 - (2 * d) % 128) % 128; }
constexpr int kQ8TileBytesExtra = 64;

// fp16 -> E5M2 byte, round to nearest even, saturating at the largest finite value (inputs are
// finite). Exposed to the quantisation kernel only.
__device__ __forceinline__ uint32_t half_bits_to_e5m2(uint32_t h) {
    uint32_t r = (h + 0x7fu + ((h >> 8) & 1u)) >> 8;
    if ((r & 0x7fu) >= 0x7cu) r = (r & 0x80u) | 0x7bu;
    return r & 0xffu;
}

// One warp per row: x8[row] = E5M2(x[row]); bound[row] = |x - x8| (1 + 2^-10)
// + d 2^-21 |x8| (1 + 2^-10): the quantisation error plus a bound on the rounding of d fp32
// accumulation steps of the tensor-core product, per unit of |q|.
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const __half *__restrict__ corpus, long long N, int d, uint8_t *__restrict__ x8,
                     float *__restrict__ bound) {
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long row = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); row < N;
         row += warps) {
        const uint4 *src = reinterpret_cast<const uint4 *>(corpus + row * d);
        uint2 *dst = reinterpret_cast<uint2 *>(x8 + row * d);
        float err2 = 0.f, n2 = 0.f;
        for (int piece = lane; piece * 8 < d; piece += 32) {
            const uint4 raw = __ldg(src + piece);
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t out[2] = {0u, 0u};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t h = (w[e >> 1] >> ((e & 1) * 16)) & 0xffffu;
                const uint32_t b = half_bits_to_e5m2(h);
                out[e >> 2] |= b << ((e & 3) * 8);
                const float x = __half2float(__ushort_as_half(static_cast<unsigned short>(h)));
                const float xq = __half2float(__ushort_as_half(static_cast<unsigned short>(b << 8)));
                const float df = x - xq;
                err2 = fmaf(df, df, err2);
                n2 = fmaf(xq, xq, n2);
            }
            dst[piece] = make_uint2(out[0], out[1]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            err2 += __shfl_xor_sync(0xffffffffu, err2, o);
            n2 += __shfl_xor_sync(0xffffffffu, n2, o);
        }
        if (lane == 0) {
            const float up = 1.0f + 1.0f / 1024.0f;
            bound[row] = __fadd_ru(__fmul_ru(__fsqrt_ru(err2), up),
                                   __fmul_ru(__fmul_ru(__fsqrt_ru(n2), up), static_cast<float>(d) * (1.0f / 2097152.0f)));
        }
    }
}

// One fp16 corpus row (global memory) against one staged query, by the whole warp: the exact
// inner product, or for L2 the squared distance in the direct sum-of-squared-differences form.
// The staged query has every group of four elements stored as (e0, e2, e1, e3). The row is not
// in any cache (only its one-byte copy was streamed), so the loads of four steps are issued
// together: one DRAM latency per 1024 elements instead of four.
template <bool L2>
__device__ __forceinline__ float warp_exact_score(const __half *row, uint32_t q_addr, int d, int lane) {
    float2 sum = make_float2(0.f, 0.f);
    const uint4 *src = reinterpret_cast<const uint4 *>(row);
    const int pieces = d >> 3;
    for (int base = 0; base < pieces; base += 128) {
        uint4 xr[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int piece = base + u * 32 + lane;
            xr[u] = piece < pieces ? __ldg(src + piece) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int piece = base + u * 32 + lane;
            if (piece < pieces) {
                const uint4 qr = lds128(q_addr + piece * 16);
                const uint32_t xw[4] = {xr[u].x, xr[u].y, xr[u].z, xr[u].w};
                const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float2 x01 = h2_to_f2(xw[2 * e]), x23 = h2_to_f2(xw[2 * e + 1]);
                    const float2 q02 = h2_to_f2(qw[2 * e]), q13 = h2_to_f2(qw[2 * e + 1]);
                    if (L2) {
                        const float d0 = x01.x - q02.x, d1 = x01.y - q13.x, d2 = x23.x - q02.y, d3 = x23.y - q13.y;
                        sum.x = fmaf(d0, d0, sum.x);
                        sum.y = fmaf(d1, d1, sum.y);
                        sum.x = fmaf(d2, d2, sum.x);
                        sum.y = fmaf(d3, d3, sum.y);
                    } else {
                        sum.x = fmaf(x01.x, q02.x, sum.x);
                        sum.y = fmaf(x01.y, q13.x, sum.y);
                        sum.x = fmaf(x23.x, q02.y, sum.x);
                        sum.y = fmaf(x23.y, q13.y, sum.y);
                    }
                }
            }
        }
    }
    float v = sum.x + sum.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// p.x8: the 8-bit copy; p.norms: the per-row bound e_j; p.corpus: the fp16 rows (rescoring).
// L2: squared distance (p.sqnorms: the rows' squared norms; p.l2_slack as in the fp16 L2 scan).
// p.spill: candidate lists in global memory with one sort scratch in shared memory (large k).
// NG groups of 8 queries per pass share every staged tile (NG = 1 or 2); p.tile_rows == 16;
// d % 16 == 0.
template <bool TOP1, int NG, bool L2 = false>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_q8_kernel(const ScanParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    ScanHeader *hdr = reinterpret_cast<ScanHeader *>(smem);
    uint64_t *scratch = p.spill ? reinterpret_cast<uint64_t *>(smem + p.off_cand) : nullptr;
    uint64_t *cand = p.spill ? p.spill + static_cast<size_t>(blockIdx.x) * kScanMaxPassQueries * p.cap
                             : reinterpret_cast<uint64_t *>(smem + p.off_cand);
    const long long list_room = p.spill ? p.ext.lists - static_cast<long long>(blockIdx.x) * kScanMaxPassQueries * p.cap
                                        : 1LL << 62;
    const int W = p.nwarps;
    const int S = W * p.depth;
    constexpr int T = 16;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int d = p.d;
    const uint32_t q_pitch = static_cast<uint32_t>(q8_query_pitch(d));

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
    {
        // queries as fp16 [8 NG][d] in shared memory, rows >= s zeroed, every group of four elements
        // stored as (e0, e2, e1, e3): the order in which a 32-bit word of the 8-bit rows unpacks
        const uint2 *qg = reinterpret_cast<const uint2 *>(p.queries);
        const int per_row = d / 4;
        for (int i = threadIdx.x; i < NG * kScanMaxQueries * per_row; i += blockDim.x) {
            const int row = i / per_row, col = i - row * per_row;
            uint2 v = make_uint2(0u, 0u);
            if (row < p.s) {
                const uint2 src = qg[i];   // (e0, e1), (e2, e3)
                v.x = __byte_perm(src.x, src.y, 0x5410);
                v.y = __byte_perm(src.x, src.y, 0x7632);
            }
            *reinterpret_cast<uint2 *>(smem + p.off_q + row * q_pitch + col * 8) = v;
        }
    }
    __syncthreads();

    const long long my_tiles = (p.ntiles > blockIdx.x) ? (p.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    volatile int *abort_flag = &hdr->abort;
    volatile int *compact_flag = &hdr->flag;
    volatile int *done_count = &hdr->done;

    // Every consumer warp streams its own tiles: its lane 0 refills a stage as soon as the warp has
    // read it (a single producer thread could not issue tiles of this size fast enough). Warp 0
    // only takes part in the set-up above.
    if (warp >= 1 && warp - 1 < W) {
        // ---------------------------------------------------------------- consumers
        const int w = warp - 1;
        const int ctid = threadIdx.x - 32;
        const int cthreads = W * 32;
        const int g = lane >> 2, t = lane & 3;
        const uint32_t q_base_addr = smem_u32(smem + p.off_q);

        long long row0 = p.row_begin + (static_cast<long long>(blockIdx.x) + static_cast<long long>(w) * gridDim.x) * T;
        const long long row_step = static_cast<long long>(gridDim.x) * W * T;

        // |q| of this lane's two queries (2t, 2t + 1), rounded up (and |q|^2 for L2)
        float qn0[NG], qn1[NG], qs0[NG], qs1[NG];
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) {
            const int row_a = grp * kScanMaxQueries + 2 * t;
            const __half *qa = reinterpret_cast<const __half *>(smem + p.off_q + row_a * q_pitch);
            const __half *qb = reinterpret_cast<const __half *>(smem + p.off_q + (row_a + 1) * q_pitch);
            float a2 = 0.f, b2 = 0.f;
            for (int i = 0; i < d; ++i) {
                const float a = __half2float(qa[i]), b = __half2float(qb[i]);
                a2 = fmaf(a, a, a2);
                b2 = fmaf(b, b, b2);
            }
            const float up = 1.0f + 1.0f / 1024.0f;
            qn0[grp] = __fmul_ru(__fsqrt_ru(a2), up);
            qn1[grp] = __fmul_ru(__fsqrt_ru(b2), up);
            qs0[grp] = a2;
            qs1[grp] = b2;
        }

        int slot = 0;
        uint32_t parity = 0;
        // this warp's tiles: the CTA's tiles w, w + W, ...; the j-th goes to slot j % depth of the
        // warp's private ring (stage w + slot * W)
        const long long n_mine = (my_tiles > w) ? (my_tiles - w + W - 1) / W : 0;
        const uint32_t stage_base = smem_u32(smem + p.off_stage);
        auto issue_tile = [&](long long first_row, int slot_) {   // lane 0 only
            const long long rows = (p.N - first_row < T) ? (p.N - first_row) : T;
            const uint32_t bytes = static_cast<uint32_t>(rows) * static_cast<uint32_t>(d);
            const int st_ = w + slot_ * W;
            const uint32_t bar = smem_u32(&hdr->full[st_]);
            mbar_arrive_expect_tx(bar, bytes);
            // rows 0..7 and rows 8..15 as two copies, the second 64 bytes further
            const uint32_t first = rows < 8 ? bytes : static_cast<uint32_t>(8 * d);
            const uint32_t dst = stage_base + static_cast<uint32_t>(st_) * p.stage_bytes;
            const long long src_row = in_bounds(first_row + rows - 1, p.ext.rows, p.status) ? first_row : 0;
            bulk_load(dst, p.x8 + src_row * d, first, bar);
            if (bytes > first)
                bulk_load(dst + first + kQ8TileBytesExtra, p.x8 + (src_row + 8) * d, bytes - first, bar);
        };
        long long issued = 0, landed = 0;   // of this warp's tiles (lane 0 issues; all lanes count alike)
        for (; issued < p.depth && issued < n_mine; ++issued)
            if (lane == 0) issue_tile(row0 + issued * row_step, static_cast<int>(issued));

        // The rows' bounds are fetched one tile ahead: the tile itself is usually resident by the
        // time its turn comes, and a load issued only then would stall the warp for a DRAM latency.
        const int ph_lo = q8_phys_row(g), ph_hi = q8_phys_row(g + 8);
        float e_lo_next = 0.f, e_hi_next = 0.f, n_lo_next = 0.f, n_hi_next = 0.f;
        if (w < my_tiles) {
            if (row0 + ph_lo < p.N) e_lo_next = __ldg(p.norms + row0 + ph_lo);
            if (row0 + ph_hi < p.N) e_hi_next = __ldg(p.norms + row0 + ph_hi);
            if (L2 && row0 + ph_lo < p.N) n_lo_next = __ldg(p.sqnorms + row0 + ph_lo);
            if (L2 && row0 + ph_hi < p.N) n_hi_next = __ldg(p.sqnorms + row0 + ph_hi);
        }
        long long tiles_done = 0, next_meeting = 64;
        for (long long it = w; it < my_tiles; it += W, row0 += row_step) {
            const float e_lo = e_lo_next, e_hi = e_hi_next, n_lo = n_lo_next, n_hi = n_hi_next;
            e_lo_next = e_hi_next = n_lo_next = n_hi_next = 0.f;
            if (it + W < my_tiles) {
                const long long nrow = row0 + row_step;
                if (nrow + ph_lo < p.N) e_lo_next = __ldg(p.norms + nrow + ph_lo);
                if (nrow + ph_hi < p.N) e_hi_next = __ldg(p.norms + nrow + ph_hi);
                if (L2 && nrow + ph_lo < p.N) n_lo_next = __ldg(p.sqnorms + nrow + ph_lo);
                if (L2 && nrow + ph_hi < p.N) n_hi_next = __ldg(p.sqnorms + nrow + ph_hi);
            }
            if (*abort_flag) continue;
            // (shared thresholds, large k: meetings after 64, 128, 256, ... tiles, as in scan_kernel)
            if (!TOP1 && p.pub && w == 0 && ++tiles_done == next_meeting) {
                next_meeting *= 2;
                if (lane == 0) *compact_flag = 1;
            }
            const int st = w + slot * W;
            const int cur_slot = slot;
            const uint32_t full_bar = smem_u32(&hdr->full[st]);
            const uint32_t my_parity = parity;
            if (++slot == p.depth) {
                slot = 0;
                parity ^= 1;
            }
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
            ++landed;
            const uint32_t stage_addr = smem_u32(smem + p.off_stage + static_cast<size_t>(st) * p.stage_bytes);

            // ---- 16 rows x 8 queries on tensor cores. Per step a lane takes 16 bytes of rows g
            // and g + 8 (16 elements) and the same 16 elements of query g; each 32-bit word of a
            // row unpacks into the fp16 pairs (e0, e2) and (e1, e3), which is how the query is stored.
            // several accumulator sets per group shorten the chain of dependent MMAs
            constexpr int NA = NG == 1 ? 4 : 2;
            float accs[NG][NA][4];
#pragma unroll
            for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                for (int i = 0; i < NA; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) accs[grp][i][j] = 0.f;
            const int nchunks = (d + 63) >> 6;
            const uint32_t q_addr = q_base_addr + g * q_pitch;
            const uint32_t grp_pitch = kScanMaxQueries * q_pitch;
            const uint32_t a_lo_addr = stage_addr + q8_row_offset(ph_lo, d);
            const uint32_t a_hi_addr = stage_addr + q8_row_offset(ph_hi, d);
            // (the loads of step c + 1 are issued before the MMAs of step c)
            uint4 lo = make_uint4(0, 0, 0, 0), hi = lo;
            uint4 b0[NG], b1[NG];
#pragma unroll
            for (int grp = 0; grp < NG; ++grp) b0[grp] = b1[grp] = lo;
            if (t * 16 < d) {
                lo = lds128(a_lo_addr + t * 16);
                hi = lds128(a_hi_addr + t * 16);
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) {
                    b0[grp] = lds128(q_addr + grp * grp_pitch + t * 32);
                    b1[grp] = lds128(q_addr + grp * grp_pitch + t * 32 + 16);
                }
            }
#pragma unroll 4
            for (int c = 0; c < nchunks; ++c) {
                const int off = (c + 1) * 64 + t * 16;
                uint4 nlo = make_uint4(0, 0, 0, 0), nhi = nlo;
                uint4 nb0[NG], nb1[NG];
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) nb0[grp] = nb1[grp] = nlo;
                if (off < d) {  // ragged last chunk: absent pieces stay zero (the MMAs are warp-wide)
                    nlo = lds128(a_lo_addr + off);
                    nhi = lds128(a_hi_addr + off);
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        nb0[grp] = lds128(q_addr + grp * grp_pitch + off * 2);
                        nb1[grp] = lds128(q_addr + grp * grp_pitch + off * 2 + 16);
                    }
                }
                const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w};
                const uint32_t hw[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t l02 = __byte_perm(lw[i], 0u, 0x2404), l13 = lw[i] & 0xff00ff00u;
                    const uint32_t h02 = __byte_perm(hw[i], 0u, 0x2404), h13 = hw[i] & 0xff00ff00u;
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        const uint32_t bw[8] = {b0[grp].x, b0[grp].y, b0[grp].z, b0[grp].w,
                                                b1[grp].x, b1[grp].y, b1[grp].z, b1[grp].w};
                        mma_m16n8k16(accs[grp][i % NA], l02, h02, l13, h13, bw[2 * i], bw[2 * i + 1]);
                    }
                }
                lo = nlo;
                hi = nhi;
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) {
                    b0[grp] = nb0[grp];
                    b1[grp] = nb1[grp];
                }
            }
            float acc[NG][4];
#pragma unroll
            for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[grp][i] = accs[grp][0][i] + accs[grp][1][i];
                    if (NA == 4) acc[grp][i] += accs[grp][2 % NA][i] + accs[grp][3 % NA][i];
                }
            // every lane has read the stage, since the MMAs above have consumed what it loaded (the
            // rest works from registers and global memory):
            // refill it with this warp's tile `depth` further on
            __syncwarp();
            if (issued < n_mine && !*abort_flag) {
                if (lane == 0) issue_tile(row0 + static_cast<long long>(p.depth) * row_step, cur_slot);
                ++issued;
            }

            // acc[0]: (MMA row g, query 2t)     acc[1]: (MMA row g, query 2t+1)
            // acc[2]: (MMA row g+8, query 2t)   acc[3]: (MMA row g+8, query 2t+1)
            const long long r_lo = row0 + ph_lo, r_hi = row0 + ph_hi;
#pragma unroll
            for (int grp = 0; grp < NG; ++grp) {
                const int q0 = grp * kScanMaxQueries + 2 * t, q1 = q0 + 1;
                float th0 = *reinterpret_cast<volatile float *>(&hdr->thr[q0]);
                float th1 = *reinterpret_cast<volatile float *>(&hdr->thr[q1]);
                if (TOP1) {
                    const unsigned long long k0 = *reinterpret_cast<volatile unsigned long long *>(&hdr->best[q0]);
                    const unsigned long long k1 = *reinterpret_cast<volatile unsigned long long *>(&hdr->best[q1]);
                    if (k0) th0 = fmaxf(th0, key_value(k0));
                    if (k1) th1 = fmaxf(th1, key_value(k1));
                }
                // upper bounds of the rank value: the score itself, or for L2 of -distance^2
                float u[4];
                u[0] = __fmaf_ru(qn0[grp], e_lo, acc[grp][0]);
                u[1] = __fmaf_ru(qn1[grp], e_lo, acc[grp][1]);
                u[2] = __fmaf_ru(qn0[grp], e_hi, acc[grp][2]);
                u[3] = __fmaf_ru(qn1[grp], e_hi, acc[grp][3]);
                if (L2) {
                    const float sl = p.l2_slack;
                    const float s00 = n_lo + qs0[grp], s01 = n_lo + qs1[grp], s10 = n_hi + qs0[grp], s11 = n_hi + qs1[grp];
                    u[0] = __fmaf_ru(2.0f, u[0], __fmaf_ru(sl, s00, 0.0f - s00));
                    u[1] = __fmaf_ru(2.0f, u[1], __fmaf_ru(sl, s01, 0.0f - s01));
                    u[2] = __fmaf_ru(2.0f, u[2], __fmaf_ru(sl, s10, 0.0f - s10));
                    u[3] = __fmaf_ru(2.0f, u[3], __fmaf_ru(sl, s11, 0.0f - s11));
                }
                bool pass[4];
                pass[0] = r_lo < p.N && q0 < p.s && u[0] >= th0;
                pass[1] = r_lo < p.N && q1 < p.s && u[1] >= th1;
                pass[2] = r_hi < p.N && q0 < p.s && u[2] >= th0;
                pass[3] = r_hi < p.N && q1 < p.s && u[3] >= th1;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    unsigned m = __ballot_sync(0xffffffffu, pass[i]);
                    while (m) {
                        const int src = __ffs(m) - 1;
                        m &= m - 1;
                        const int row_local = q8_phys_row((src >> 2) + ((i & 2) ? 8 : 0));
                        const int q = grp * kScanMaxQueries + 2 * (src & 3) + (i & 1);
                        const long long row = row0 + row_local;
                        if (!in_bounds(row, p.ext.rows, p.status)) continue;
                        const float exact = warp_exact_score<L2>(p.corpus + row * d, q_base_addr + q * q_pitch, d, lane);
                        const float val = L2 ? 0.0f - exact : exact;
                        if (lane == 0) {
                            const uint64_t key = make_key(val, static_cast<uint32_t>(row));
                            if (TOP1) {
                                if (val >= *reinterpret_cast<volatile float *>(&hdr->thr[q]))
                                    atomicMax(&hdr->best[q], static_cast<unsigned long long>(key));
                            } else if (val >= *reinterpret_cast<volatile float *>(&hdr->thr[q])) {
                                push_candidate(hdr, cand, p.cap, p.soft_limit, q, key, p.status, list_room);
                            }
                        }
                    }
                }
            }
        }

        // winding down early: let every copy this warp has issued land before the CTA exits
        if (lane == 0)
            for (long long j = landed; j < issued; ++j)
                mbar_wait_bounded(smem_u32(&hdr->full[w + static_cast<int>(j % p.depth) * W]),
                                  static_cast<uint32_t>((j / p.depth) & 1));

        // ------------------------------------------------------------ CTA result
        if (TOP1) {
            named_barrier(1, cthreads);
            if (ctid < p.s && in_bounds(static_cast<long long>(blockIdx.x) * p.s_total + p.q_base + ctid, p.ext.partial, p.status))
                p.partial[static_cast<size_t>(blockIdx.x) * p.s_total + p.q_base + ctid] = hdr->best[ctid];
        } else {
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
