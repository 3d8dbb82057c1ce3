// Shared device helpers: ranking keys, bounded mbarrier waits, bulk copies, bitonic sort.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ralm {

// Device status word values (match ralm_status_t).
constexpr int kStatusTimeout = 4;
constexpr int kStatusBadCacheId = 6;
constexpr int kStatusInternal = 8;  // a candidate list was asked to hold more than its capacity

// ---------------------------------------------------------------------------------
// Debug build (-DRALM_DEBUG_BOUNDS, `python -m paper_2401_14021_b200.build --debug`): every index
// into a global array that a scan computes is checked against the array's extent; a violation
// records kStatusInternal in the status word, a store is skipped and a load is redirected to
// element 0. Nothing traps. The release build compiles the checks away.
// ---------------------------------------------------------------------------------
struct Extents {
    long long rows;     // rows of the whole corpus (norms, bounds and the 8-bit copy have as many)
    long long partial;  // keys in the partial-list array
    long long lists;    // keys in the candidate lists that live in global memory (0: none)
    long long aux;      // elements of the sample launch's maxima (tcgen05 scan)
};
#ifdef RALM_DEBUG_BOUNDS
__device__ __forceinline__ bool in_bounds(long long i, long long n, int *status) {
    if (i >= 0 && i < n) return true;
    atomicMax(status, kStatusInternal);
    return false;
}
#else
__device__ __forceinline__ bool in_bounds(long long, long long, int *) { return true; }
#endif

// ---------------------------------------------------------------------------------
// Ranking keys. Every candidate is one 64-bit key whose unsigned order IS the ranking:
//   high 32 bits: order-preserving image of the "rank value" v (larger v ranks first),
//                 v = score for inner product, v = -distance^2 for L2;
//   low 32 bits:  0xFFFFFFFF - row id, so that among equal v the lower id is larger.
// Key 0 is below every real key and marks an empty slot.
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ordered_bits(float v) {
    const uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}
__device__ __forceinline__ uint64_t make_key(float v, uint32_t row) {
    v += 0.0f;  // -0.0 -> +0.0 so equal values have equal bits
    return (static_cast<uint64_t>(ordered_bits(v)) << 32) | (0xFFFFFFFFu - row);
}
__device__ __forceinline__ float key_value(uint64_t key) {
    return from_ordered_bits(static_cast<uint32_t>(key >> 32));
}
__device__ __forceinline__ uint32_t key_row(uint64_t key) {
    return 0xFFFFFFFFu - static_cast<uint32_t>(key);
}

// ---------------------------------------------------------------------------------
// mbarrier + bulk-copy wrappers (shared::cta addresses as 32-bit).
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Every wait is bounded: about two seconds of SM clock, after which the caller records
// kStatusTimeout and winds down instead of spinning forever.
constexpr long long kWaitCycleLimit = 4000000000LL;
__device__ __forceinline__ bool mbar_wait_bounded_for(uint32_t bar, uint32_t parity, long long limit_cycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit_cycles) return false;
    }
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    return mbar_wait_bounded_for(bar, parity, kWaitCycleLimit);
}
// 1-D bulk copy global -> shared, completion signalled on an mbarrier (no multicast).
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes,
                                          uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void named_barrier(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ---------------------------------------------------------------------------------
// Bitonic sort (descending) of P = 2^n keys in shared memory by a group of `nthr`
// threads with ranks `tid`, synchronised through group_sync(bar_id). All threads of the
// group must call it.
// ---------------------------------------------------------------------------------
// bar_id >= 0: named barrier over nthr threads; -1: the whole CTA; -2: one warp.
__device__ __forceinline__ void group_sync(int bar_id, int nthr) {
    if (bar_id >= 0) named_barrier(bar_id, nthr);
    else if (bar_id == -1) __syncthreads();
    else __syncwarp();
}
template <typename Key>
__device__ inline void bitonic_sort_desc(Key *a, int P, int tid, int nthr, int bar_id) {
    for (int size = 2; size <= P; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = tid; i < (P >> 1); i += nthr) {
                const int lo = 2 * i - (i & (stride - 1));
                const int hi = lo + stride;
                const bool desc = (lo & size) == 0;
                const Key x = a[lo], y = a[hi];
                if ((x < y) == desc) {
                    a[lo] = y;
                    a[hi] = x;
                }
            }
            group_sync(bar_id, nthr);
        }
    }
}
// Merge step only: `a` is a bitonic sequence of P keys; leaves it sorted descending.
__device__ inline void bitonic_merge_desc(uint64_t *a, int P, int tid, int nthr, int bar_id) {
    for (int stride = P >> 1; stride > 0; stride >>= 1) {
        for (int i = tid; i < (P >> 1); i += nthr) {
            const int lo = 2 * i - (i & (stride - 1));
            const int hi = lo + stride;
            const uint64_t x = a[lo], y = a[hi];
            if (x < y) {
                a[lo] = y;
                a[hi] = x;
            }
        }
        group_sync(bar_id, nthr);
    }
}

__host__ __device__ inline int next_pow2(int v) {
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

}  // namespace ralm
