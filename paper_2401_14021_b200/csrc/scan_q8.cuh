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
// Structure (producer warp, private stage rings per consumer warp, candidate buffers, compaction
// meetings) is that of scan_kernel; the tile is 16 rows of d bytes. The host starts this kernel
// from the thresholds of an fp16 scan of a small sample, without which nearly every pair would
// pass until the lists fill.
#pragma once

#include "scan.cuh"

namespace ralm {

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

// Exact inner product of one fp16 corpus row (global memory) with one staged query, by the
// whole warp. The staged query has every group of four elements stored as (e0, e2, e1, e3).
__device__ __forceinline__ float warp_exact_ip(const __half *row, uint32_t q_addr, int d, int lane) {
    float2 sum = make_float2(0.f, 0.f);
    const uint4 *src = reinterpret_cast<const uint4 *>(row);
    for (int piece = lane; piece * 8 < d; piece += 32) {
        const uint4 xr = __ldg(src + piece);
        const uint4 qr = lds128(q_addr + piece * 16);
        const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
        const uint32_t qw[4] = {qr.x, qr.y, qr.z, qr.w};
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float2 x01 = h2_to_f2(xw[2 * e]), x23 = h2_to_f2(xw[2 * e + 1]);
            const float2 q02 = h2_to_f2(qw[2 * e]), q13 = h2_to_f2(qw[2 * e + 1]);
            sum.x = fmaf(x01.x, q02.x, sum.x);
            sum.y = fmaf(x01.y, q13.x, sum.y);
            sum.x = fmaf(x23.x, q02.y, sum.x);
            sum.y = fmaf(x23.y, q13.y, sum.y);
        }
    }
    float v = sum.x + sum.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// p.x8: the 8-bit copy; p.norms: the per-row bound e_j; p.corpus: the fp16 rows (rescoring).
// Up to 8 queries per pass; p.tile_rows == 16; d % 16 == 0.
template <bool TOP1>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_q8_kernel(const ScanParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    ScanHeader *hdr = reinterpret_cast<ScanHeader *>(smem);
    uint64_t *cand = reinterpret_cast<uint64_t *>(smem + p.off_cand);
    const int W = p.nwarps;
    const int S = W * p.depth;
    constexpr int T = 16;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int d = p.d;
    const uint32_t q_pitch = static_cast<uint32_t>(d * 2 + kQueryPadBytes);

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
        // queries as fp16 [8][d] in shared memory, rows >= s zeroed, every group of four elements
        // stored as (e0, e2, e1, e3): the order in which a 32-bit word of the 8-bit rows unpacks
        const uint2 *qg = reinterpret_cast<const uint2 *>(p.queries);
        const int per_row = d / 4;
        for (int i = threadIdx.x; i < kScanMaxQueries * per_row; i += blockDim.x) {
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

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        if (lane == 0) {
            long long issued = 0;
            bool ok = true;
            int cw = 0, slot = 0;
            uint32_t use = 0;
            long long row0 = p.row_begin + static_cast<long long>(blockIdx.x) * T;
            const long long row_step = static_cast<long long>(gridDim.x) * T;
            const uint32_t stage_base = smem_u32(smem + p.off_stage);
            for (long long it = 0; it < my_tiles; ++it) {
                const int st = cw + slot * W;
                if (use > 0) {
                    ok = mbar_wait_bounded(smem_u32(&hdr->empty[st]), (use - 1) & 1);
                    if (!ok) break;
                }
                if (*abort_flag) break;
                const long long rows = (p.N - row0 < T) ? (p.N - row0) : T;
                const uint32_t bytes = static_cast<uint32_t>(rows) * static_cast<uint32_t>(d);
                const uint32_t bar = smem_u32(&hdr->full[st]);
                mbar_arrive_expect_tx(bar, bytes);
                bulk_load(stage_base + static_cast<uint32_t>(st) * p.stage_bytes, p.x8 + row0 * d, bytes, bar);
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
            if (!ok) {
                atomicMax(p.status, kStatusTimeout);
                *abort_flag = 1;
            }
            if (*abort_flag) {
                // winding down early: let every copy already issued land before exit
                for (long long it = (issued > S ? issued - S : 0); it < issued; ++it) {
                    const long long local = it / W;
                    mbar_wait_bounded(smem_u32(&hdr->full[(it % W) + (local % p.depth) * W]), (local / p.depth) & 1);
                }
            }
        }
    } else if (warp - 1 < W) {
        // ---------------------------------------------------------------- consumers
        const int w = warp - 1;
        const int ctid = threadIdx.x - 32;
        const int cthreads = W * 32;
        const int g = lane >> 2, t = lane & 3;
        const uint32_t q_base_addr = smem_u32(smem + p.off_q);

        // |q| of this lane's two queries (2t, 2t + 1), rounded up
        float qn0 = 0.f, qn1 = 0.f;
        {
            const __half *qa = reinterpret_cast<const __half *>(smem + p.off_q + (2 * t) * q_pitch);
            const __half *qb = reinterpret_cast<const __half *>(smem + p.off_q + (2 * t + 1) * q_pitch);
            for (int i = 0; i < d; ++i) {
                const float a = __half2float(qa[i]), b = __half2float(qb[i]);
                qn0 = fmaf(a, a, qn0);
                qn1 = fmaf(b, b, qn1);
            }
            const float up = 1.0f + 1.0f / 1024.0f;
            qn0 = __fmul_ru(__fsqrt_ru(qn0), up);
            qn1 = __fmul_ru(__fsqrt_ru(qn1), up);
        }

        int slot = 0;
        uint32_t parity = 0;
        long long row0 = p.row_begin + (static_cast<long long>(blockIdx.x) + static_cast<long long>(w) * gridDim.x) * T;
        const long long row_step = static_cast<long long>(gridDim.x) * W * T;
        for (long long it = w; it < my_tiles; it += W, row0 += row_step) {
            if (*abort_flag) continue;
            const int st = w + slot * W;
            const uint32_t full_bar = smem_u32(&hdr->full[st]);
            const uint32_t my_parity = parity;
            // the rows' bounds, in flight during the wait
            float e_lo = 0.f, e_hi = 0.f;
            if (row0 + g < p.N) e_lo = __ldg(p.norms + row0 + g);
            if (row0 + g + 8 < p.N) e_hi = __ldg(p.norms + row0 + g + 8);
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
                        compaction_meeting(hdr, cand, nullptr, p.cap, p.s, p.k, w, lane, W);
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
            const uint32_t stage_addr = smem_u32(smem + p.off_stage + static_cast<size_t>(st) * p.stage_bytes);
            const uint32_t empty_bar = smem_u32(&hdr->empty[st]);

            // ---- 16 rows x 8 queries on tensor cores. Per step a lane takes 16 bytes of rows g
            // and g + 8 (16 elements) and the same 16 elements of query g; each 32-bit word of a
            // row unpacks into the fp16 pairs (e0, e2) and (e1, e3), which is how the query is stored.
            float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc_b[4] = {0.f, 0.f, 0.f, 0.f};
            const int nchunks = (d + 63) >> 6;
            const uint32_t q_addr = q_base_addr + g * q_pitch;
            const uint32_t a_lo_addr = stage_addr + g * d;
            const uint32_t a_hi_addr = stage_addr + (g + 8) * d;
#pragma unroll 2
            for (int c = 0; c < nchunks; ++c) {
                const int off = c * 64 + t * 16;
                uint4 lo = make_uint4(0, 0, 0, 0), hi = lo, b0 = lo, b1 = lo;
                if (off < d) {  // ragged last chunk: absent pieces stay zero (the MMAs are warp-wide)
                    lo = lds128(a_lo_addr + off);
                    hi = lds128(a_hi_addr + off);
                    b0 = lds128(q_addr + off * 2);
                    b1 = lds128(q_addr + off * 2 + 16);
                }
                const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w};
                const uint32_t hw[4] = {hi.x, hi.y, hi.z, hi.w};
                const uint32_t bw[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t l02 = __byte_perm(lw[i], 0u, 0x2404), l13 = lw[i] & 0xff00ff00u;
                    const uint32_t h02 = __byte_perm(hw[i], 0u, 0x2404), h13 = hw[i] & 0xff00ff00u;
                    if (i & 1) mma_m16n8k16(acc_b, l02, h02, l13, h13, bw[2 * i], bw[2 * i + 1]);
                    else mma_m16n8k16(acc, l02, h02, l13, h13, bw[2 * i], bw[2 * i + 1]);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] += acc_b[i];
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);  // the rest works from registers and global memory

            // acc[0]: (row g, query 2t)     acc[1]: (row g, query 2t+1)
            // acc[2]: (row g+8, query 2t)   acc[3]: (row g+8, query 2t+1)
            const long long r_lo = row0 + g, r_hi = row0 + g + 8;
            const int q0 = 2 * t, q1 = q0 + 1;
            float th0 = *reinterpret_cast<volatile float *>(&hdr->thr[q0]);
            float th1 = *reinterpret_cast<volatile float *>(&hdr->thr[q1]);
            if (TOP1) {
                const unsigned long long k0 = *reinterpret_cast<volatile unsigned long long *>(&hdr->best[q0]);
                const unsigned long long k1 = *reinterpret_cast<volatile unsigned long long *>(&hdr->best[q1]);
                if (k0) th0 = fmaxf(th0, key_value(k0));
                if (k1) th1 = fmaxf(th1, key_value(k1));
            }
            bool pass[4];
            pass[0] = r_lo < p.N && q0 < p.s && __fmaf_ru(qn0, e_lo, acc[0]) >= th0;
            pass[1] = r_lo < p.N && q1 < p.s && __fmaf_ru(qn1, e_lo, acc[1]) >= th1;
            pass[2] = r_hi < p.N && q0 < p.s && __fmaf_ru(qn0, e_hi, acc[2]) >= th0;
            pass[3] = r_hi < p.N && q1 < p.s && __fmaf_ru(qn1, e_hi, acc[3]) >= th1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                unsigned m = __ballot_sync(0xffffffffu, pass[i]);
                while (m) {
                    const int src = __ffs(m) - 1;
                    m &= m - 1;
                    const int row_local = (src >> 2) + ((i & 2) ? 8 : 0);
                    const int q = 2 * (src & 3) + (i & 1);
                    const long long row = row0 + row_local;
                    const float val = warp_exact_ip(p.corpus + row * d, q_base_addr + q * q_pitch, d, lane);
                    if (lane == 0) {
                        const uint64_t key = make_key(val, static_cast<uint32_t>(row));
                        if (TOP1) {
                            if (val >= *reinterpret_cast<volatile float *>(&hdr->thr[q]))
                                atomicMax(&hdr->best[q], static_cast<unsigned long long>(key));
                        } else if (val >= *reinterpret_cast<volatile float *>(&hdr->thr[q])) {
                            push_candidate(hdr, cand, p.cap, p.soft_limit, q, key);
                        }
                    }
                }
            }
        }

        // ------------------------------------------------------------ CTA result
        if (TOP1) {
            named_barrier(1, cthreads);
            if (ctid < p.s)
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
                if (state == 1) compaction_meeting(hdr, cand, nullptr, p.cap, p.s, p.k, w, lane, W);
                else if (state == 2) break;
            }
            named_barrier(1, cthreads);
            compact_all(hdr, cand, nullptr, p.cap, p.s, p.k, 0, w, lane, W);
            named_barrier(1, cthreads);
            for (int q = 0; q < p.s; ++q) {
                const int n = hdr->cnt[q];
                uint64_t *dst = p.partial + (static_cast<size_t>(blockIdx.x) * p.s_total + p.q_base + q) * p.k;
                for (int i = ctid; i < p.k; i += cthreads)
                    dst[i] = (i < n) ? cand[static_cast<size_t>(q) * p.cap + i] : 0ull;
            }
        }
    }
}

}  // namespace ralm
