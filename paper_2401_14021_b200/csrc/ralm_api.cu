// Host side of the C ABI declared in include/ralm.h: argument checks, workspace, variant
// dispatch and launches. All device work is in the kernels included below.
#include "../../include/ralm.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "aux_kernels.cuh"
#include "scan.cuh"
#include "scan_q8.cuh"
#include "scan_tc.cuh"

using namespace ralm;

struct ralm_index {
    const __half *corpus;
    int64_t N;
    int32_t d;
    ralm_metric_t metric;
    int32_t max_s, max_k;
    int device;
    int num_sms;
    int smem_optin;
    int variant;  // 0 auto, 1 FMA, 2 warp-MMA, 3 tcgen05
    int tune_warps, tune_depth, tune_rows;  // 0 = library default
    uint64_t *partial;   // [num_sms][max_s][max_k]
    long long partial_keys;  // keys the array holds
    uint64_t *merge_tmp;   // two-level final merge: [kMergeGroups][kMergeTwoLevelMaxS][max_k] keys, or null
    uint64_t *cache_keys;  // [RALM_MAX_CACHE_KEYS]
    uint64_t *spill;       // large k: candidate lists of the small-batch scan, [num_sms][8][spill_cap]
    int spill_cap;
    uint32_t *pub;         // large k: thresholds the scan CTAs publish to each other, [num_sms][max_s]
    float *scan_gmax;      // large k: per-warp maxima of the small-batch scan's sample launch, [num_sms * 8][max_s]
    float *norms;          // L2: squared norm of every corpus row (fp32 [N]), or null
    uint8_t *x8;           // inner product, optional: one-byte (E5M2) copy of the corpus, [N][d]
    float *x8_bound;       // per row: bound on |q.x - q.x8| per unit of |q| (see scan_q8.cuh)
    bool x8_force;         // use the copy also on corpora too small for a sample phase (testing aid)
    float *tc_thr;         // thresholds from the sample phase of a two-phase scan, [max_s]
    float *tc_gmax;        // tcgen05 scan, sample launch: [num_sms * 4][max_s] maxima per selection warp
    int *tc_tile_counter;  // tcgen05 scan: the launch's row-tile counter
    bool tc_two_phase;     // sample phase enabled (tuning aid)
    int tc_clusters;       // CTA pairs the device runs at once (-1 = not asked yet)
    uint64_t *tc_cand;     // tcgen05 scan: [num_sms][tc_cand_q][tc_cand_cap] candidate lists, or null
    int tc_cand_q, tc_cand_cap;
    int *status;
    // staging for the host-buffer entry point
    __half *h_queries;
    int64_t *h_ids;
    float *h_scores;
    int64_t launches;
    // what the last search ran (ralm_index_last_dispatch)
    int last_kernel, last_passes, last_phases;
    int64_t last_sample_rows;
    // optional per-launch timing of the scan kernel (events on the caller's stream)
    bool timing;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timed;   // recorded, not yet read
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> spare;   // reusable
};

namespace {

struct ScanPlan {
    int nwarps, depth, tile_rows, stage_bytes, cap, soft_limit, off_q, off_cand, off_stage, smem_bytes;
    bool spill;  // candidate lists in global memory, one sort scratch in shared memory
};

constexpr int kSmemCandBytes = 32 * 1024;  // candidate lists larger than this leave shared memory
constexpr int kPubMinK = 128;              // from this k on the scan CTAs share thresholds (ScanParams::pub)
constexpr int kGmaxSlots = 4;              // groups per warp in a sample launch by maxima (ScanParams::gmax_slots)
constexpr int kMergeGroups = 16;           // two-level final merge: groups of lists merged side by side first
constexpr int kMergeTwoLevelMaxS = 16;     // ... for batches up to this size (larger ones have CTAs enough)

int align_up(int v, int a) { return (v + a - 1) / a * a; }

// Extents of an index's global arrays (checked by the debug build's kernels).
Extents index_extents(const ralm_index *idx, long long list_keys) {
    Extents e;
    e.rows = idx->N;
    e.partial = idx->partial_keys;
    e.lists = list_keys;
    e.aux = idx->tc_gmax ? static_cast<long long>(idx->num_sms) * 4 * idx->max_s : 0;
    return e;
}

// Every device allocation of the library goes through here, so that a test can make the n-th
// one fail (ralm_debug_fail_allocation) and check that creation reports it and frees the rest.
std::atomic<int> g_fail_allocation_in{0};
template <typename T>
cudaError_t device_alloc(T **ptr, size_t bytes) {
    int n = g_fail_allocation_in.load();
    while (n > 0 && !g_fail_allocation_in.compare_exchange_weak(n, n - 1)) {}
    if (n == 1) {
        *ptr = nullptr;
        return cudaErrorMemoryAllocation;
    }
    return cudaMalloc(reinterpret_cast<void **>(ptr), bytes);
}

// Shared-memory layout of one scan CTA. Returns false if not even two stages fit.
bool plan_scan(const ralm_index *idx, bool mma, int s_pass, int k, ScanPlan *pl, bool maxima = false) {
    // warp-MMA tiles are 16 rows (the M of m16n8k16). The FMA flavour is bound by its
    // arithmetic, so it wants many small tiles: several being scored while more are in flight.
    pl->nwarps = mma ? kMaxConsumerWarps : kMaxConsumerWarps - 1;
    pl->tile_rows = mma ? 16 : (s_pass == 1 ? 16 : 4);
    if (idx->tune_warps > 0) pl->nwarps = std::min(idx->tune_warps, pl->nwarps);
    if (idx->tune_rows > 0 && !mma) {
        const int unit = s_pass == 1 ? 16 : 4;  // rows per reduction group of the FMA flavour
        pl->tile_rows = std::max(unit, idx->tune_rows / unit * unit);
    }
    pl->stage_bytes = align_up(pl->tile_rows * idx->d * 2 + (mma ? kTileShiftBytes : 0), 128);
    pl->off_q = kScanHeaderBytes;
    // (the warp-MMA flavour stages 8 query rows, or 16 when a pass carries more than 8)
    const int q_rows = s_pass > 16 ? 32 : (s_pass > kScanMaxQueries ? 16 : kScanMaxQueries);
    int off = pl->off_q + (mma ? align_up(q_rows * (idx->d * 2 + kQueryPadBytes), 128) : 0);
    pl->off_cand = off;
    pl->cap = 0;
    pl->soft_limit = 0;
    pl->spill = false;
    if (k > 1) {
        // after the flag is raised every warp may still finish the tile it is on
        // (256 slots up to k = 64: with 512 the lists of 8 queries take 32 KB of shared memory, one
        // stage of the ring, and the scan runs on seven consumer warps instead of eight)
        pl->cap = k <= 64 ? 256 : std::max(512, 2 * next_pow2(k));
        // (a tuned tile height must leave that room: k kept keys plus one tile from every warp)
        const int unit = mma ? 16 : (s_pass == 1 ? 16 : 4);
        const int max_rows = (pl->cap - k) / (kMaxConsumerWarps + 1) / unit * unit;
        if (pl->tile_rows > max_rows) {
            pl->tile_rows = std::max(unit, max_rows);
            pl->stage_bytes = align_up(pl->tile_rows * idx->d * 2 + (mma ? kTileShiftBytes : 0), 128);
        }
        // compact before the buffer is full, and already at about 4 k entries: a threshold only
        // rises when its list is compacted, and until then every push costs a shared atomic
        pl->soft_limit = std::min(pl->cap - (kMaxConsumerWarps + 1) * pl->tile_rows, std::max(4 * k, 64));
        // the stage ring needs the room more than large lists do: those go to global memory
        // (they are touched rarely) and only the scratch they are sorted in stays here
        pl->spill = s_pass * pl->cap * 8 > kSmemCandBytes && idx->spill && pl->cap <= idx->spill_cap;
        off += (pl->spill ? 1 : s_pass) * pl->cap * 8;
    } else if (maxima) {
        off += kMaxConsumerWarps * kGmaxSlots * kScanMaxPassQueries * 8;  // the warps' best keys (ScanParams::gmax)
    }
    pl->off_stage = align_up(off, 128);
    const int room = idx->smem_optin - pl->off_stage;
    const int fit = std::min(kMaxStages, room / pl->stage_bytes);
    if (fit < 2) return false;
    // every consumer warp owns `depth` stages; fewer warps when the stages are large
    pl->nwarps = std::min(pl->nwarps, fit);
    pl->depth = std::min(fit / pl->nwarps, idx->tune_depth > 0 ? idx->tune_depth : 3);
    pl->smem_bytes = pl->off_stage + pl->nwarps * pl->depth * pl->stage_bytes;
    return true;
}

// Shared-memory layout of one CTA of the 8-bit scan: 16-row tiles of d bytes, 8 or 16 staged
// queries, candidate lists in shared memory: k <= kQ8MaxK for up to 8 queries, k <= kQ8MaxKWide
// (lists of 256 slots) for 9..16, which keeps them within kSmemCandBytes. Larger k (up to 8
// queries) keeps the lists in global memory, as the fp16 scan does, when the index has them.
constexpr int kQ8MaxK = 256;
constexpr int kQ8MaxKWide = 64;
constexpr int kQ8MaxQueries = 2 * kScanMaxQueries;
bool plan_scan_q8(const ralm_index *idx, int s_pass, int k, ScanPlan *pl) {
    const int q_rows = s_pass > kScanMaxQueries ? kQ8MaxQueries : kScanMaxQueries;
    // (lists beyond 256 slots go to global memory whenever the index has room for them there: with
    // 512 slots in shared memory the stage ring loses a consumer warp, and this scan is bound by
    // those; with more, the lists do not fit at all)
    const bool spill = q_rows == kScanMaxQueries && k > kQ8MaxKWide && idx->spill &&
                       std::max(512, 2 * next_pow2(k)) <= idx->spill_cap;
    if (s_pass > kQ8MaxQueries || (k > (q_rows > kScanMaxQueries ? kQ8MaxKWide : kQ8MaxK) && !spill)) return false;
    pl->tile_rows = 16;
    pl->stage_bytes = align_up(pl->tile_rows * idx->d + kQ8TileBytesExtra, 128);
    pl->off_q = kScanHeaderBytes;
    int off = pl->off_q + align_up(q_rows * q8_query_pitch(idx->d), 128);
    pl->off_cand = off;
    pl->cap = 0;
    pl->soft_limit = 0;
    pl->spill = false;
    if (k > 1) {
        // (lists of 256 slots wherever k allows: with 512 the stage ring has room for only seven
        // consumer warps, and this scan is bound by them: 2.59 against 2.35 ms on 21 M x 768)
        pl->cap = (q_rows > kScanMaxQueries || k <= kQ8MaxKWide) ? 256 : std::max(512, 2 * next_pow2(k));
        pl->soft_limit = std::min(pl->cap - (kMaxConsumerWarps + 1) * pl->tile_rows, std::max(4 * k, 64));
        pl->spill = spill;
        off += (spill ? 1 : q_rows) * pl->cap * 8;   // spilled lists: one sort scratch stays here
    }
    pl->off_stage = align_up(off, 128);
    const int fit = std::min(kMaxStages, (idx->smem_optin - pl->off_stage) / pl->stage_bytes);
    if (fit < 2) return false;
    // two stages per consumer warp before an eighth warp: a warp that is scoring a row again
    // from global memory must not hold up the producer
    pl->depth = fit >= 3 * kMaxConsumerWarps ? 3 : (fit >= 4 ? 2 : 1);
    pl->nwarps = std::min(kMaxConsumerWarps, fit / pl->depth);
    if (idx->tune_warps > 0 && idx->tune_depth > 0 && idx->tune_warps * idx->tune_depth <= fit) {
        pl->nwarps = std::min(idx->tune_warps, kMaxConsumerWarps);
        pl->depth = idx->tune_depth;
    }
    pl->smem_bytes = pl->off_stage + pl->nwarps * pl->depth * pl->stage_bytes;
    return true;
}

template <bool MMA, bool L2, int SQ, int DP, bool TOP1, bool NRM = false>
cudaError_t launch_scan(const ScanParams &p, int grid, int smem, cudaStream_t st) {
    auto kern = scan_kernel<MMA, L2, SQ, DP, TOP1, NRM>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, 32 * (p.nwarps + 1), smem, st>>>(p);
    return cudaGetLastError();
}

template <bool L2, int SQ, bool TOP1>
cudaError_t launch_fma_dp(const ScanParams &p, int grid, int smem, cudaStream_t st) {
    if (p.d <= 256) return launch_scan<false, L2, SQ, 1, TOP1>(p, grid, smem, st);
    if (p.d <= 768) return launch_scan<false, L2, SQ, 3, TOP1>(p, grid, smem, st);
    return launch_scan<false, L2, SQ, 4, TOP1>(p, grid, smem, st);
}

template <bool L2>
cudaError_t launch_fma(const ScanParams &p, int grid, int smem, cudaStream_t st) {
    const bool top1 = p.k == 1;
    if (p.s == 1)
        return top1 ? launch_fma_dp<L2, 1, true>(p, grid, smem, st)
                    : launch_fma_dp<L2, 1, false>(p, grid, smem, st);
    return top1 ? launch_fma_dp<L2, 4, true>(p, grid, smem, st)
                : launch_fma_dp<L2, 4, false>(p, grid, smem, st);
}

constexpr int kFmaMaxD = 1024;
constexpr int kFmaQueriesPerPass = 4;

// Which scan serves a small batch on this index: 1 = FMA, 2 = warp-MMA (the default).
int resolve_variant(const ralm_index *idx) {
    if (idx->variant == 1 || idx->variant == 2) return idx->variant;
    return 2;
}


using TimedEvents = std::pair<cudaEvent_t, cudaEvent_t>;

// Optional timing of the scan launches of one pass: a pair of events recorded on the caller's
// stream directly around them, kept until ralm_index_read_timing collects the durations.
bool timing_begin(ralm_index *idx, cudaStream_t st, TimedEvents *ev) {
    if (!idx->timing) return true;
    if (!idx->spare.empty()) {
        *ev = idx->spare.back();
        idx->spare.pop_back();
    } else if (cudaEventCreate(&ev->first) != cudaSuccess || cudaEventCreate(&ev->second) != cudaSuccess) {
        return false;
    }
    return cudaEventRecord(ev->first, st) == cudaSuccess;
}
void timing_end(ralm_index *idx, cudaStream_t st, const TimedEvents &ev) {
    if (!idx->timing) return;
    cudaEventRecord(ev.second, st);
    idx->timed.push_back(ev);
}

// ---- tcgen05 scan (large batches, inner product) -------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The tensor-map encoder lives in the driver; it is looked up once through the runtime so that
// the library does not link against the driver library.
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(sym);
    }();
    return fn;
}

// fp16 [rows][d] row-major, tiles of box_rows x 64 elements, 128-byte swizzle, zero fill
// outside the tensor.
bool encode_rows_map(CUtensorMap *map, const void *base, long long rows, int d, int box_rows) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kTcChunkK), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_can_serve(const ralm_index *idx, int k) {
    return (idx->metric == RALM_IP || idx->norms != nullptr) && idx->tc_cand != nullptr && k <= kTcMaxK &&
           (k <= kTcSmallK || idx->tc_cand_cap >= kTcCapLarge) &&
           idx->d >= kTcChunkK;
}

bool alloc_tc_workspace(ralm_index *idx, int queries) {
    if (idx->tc_cand && idx->tc_cand_q >= queries) return true;
    if (idx->tc_cand) cudaFree(idx->tc_cand);
    idx->tc_cand = nullptr;
    idx->tc_cand_q = 0;
    const int cap = idx->max_k > kTcSmallK ? kTcCapLarge : kTcCapSmall;
    const size_t bytes = sizeof(uint64_t) * idx->num_sms * static_cast<size_t>(queries) * cap;
    if (!idx->tc_thr && device_alloc(&idx->tc_thr, sizeof(float) * idx->max_s) != cudaSuccess) {
        idx->tc_thr = nullptr;
        return false;
    }
    if (!idx->tc_gmax &&
        device_alloc(&idx->tc_gmax, sizeof(float) * idx->num_sms * 4 * static_cast<size_t>(idx->max_s)) != cudaSuccess) {
        idx->tc_gmax = nullptr;
        return false;
    }
    if (!idx->tc_tile_counter && device_alloc(&idx->tc_tile_counter, sizeof(int)) != cudaSuccess) {
        idx->tc_tile_counter = nullptr;
        return false;
    }
    if (device_alloc(&idx->tc_cand, bytes) != cudaSuccess) {
        idx->tc_cand = nullptr;
        return false;
    }
    idx->tc_cand_q = queries;
    idx->tc_cand_cap = cap;
    return true;
}

// One pass of up to min(512, workspace) queries. `pair`: clusters of two CTAs that share each
// MMA (half the query bytes staged per CTA); falls back to single CTAs when no cluster fits.
ralm_status_t launch_tc_pass(ralm_index *idx, const __half *queries, int sp, int s_total, int q0, int k,
                             bool pair, long long row_begin, long long row_end, const float *thr_init,
                             int mode, int *grid_out, cudaStream_t st) {
    TcParams p;
    p.partial = idx->partial;
    p.cand = idx->tc_cand;
    p.cand_q = idx->tc_cand_q;
    // (lists of 256 slots whenever k allows, also in a workspace sized for more)
    p.cap = k > kTcSmallK ? kTcCapLarge : kTcCapSmall;
    p.soft = k > kTcSmallK ? kTcSoftLarge : kTcSoftSmall;
    p.status = idx->status;
    p.N = row_end;
    p.thr_init = thr_init;
    p.mode = mode;
    p.gmax = idx->tc_gmax;
    p.tile_counter = idx->tc_tile_counter;
    if (cudaMemsetAsync(idx->tc_tile_counter, 0, sizeof(int), st) != cudaSuccess) return RALM_ERR_CUDA;
    p.ext = index_extents(idx, static_cast<long long>(idx->num_sms) * idx->tc_cand_q * idx->tc_cand_cap);
    p.d = idx->d;
    p.slack = static_cast<float>(idx->d) * (1.0f / 2097152.0f);  // as in the small-batch L2 scan
    p.norms = idx->norms;
    p.corpus = idx->corpus;
    p.queries = queries;
    p.nchunks = (idx->d + kTcChunkK - 1) / kTcChunkK;
    p.s = sp;
    p.s_total = s_total;
    p.q_base = q0;
    p.k = k;
    p.off_stage = align_up(kTcOffEnd, 1024);
    CUtensorMap map_x, map_q;
    if (!encode_rows_map(&map_x, idx->corpus, idx->N, idx->d, kTcTileM)) return RALM_ERR_CUDA;
    for (;;) {
        const int group_rows = pair ? 2 * kTcTileM : kTcTileM;
        p.tile0 = row_begin / group_rows;  // row_begin is a multiple of 256
        p.ntiles = (row_end - row_begin + group_rows - 1) / group_rows;
        p.nb = sp > kTcMaxN ? kTcMaxN : align_up(sp, pair ? 32 : 16);
        p.nhalves = (sp + p.nb - 1) / p.nb;
        const int nb_cta = pair ? p.nb / 2 : p.nb;
        p.chunk_bytes = kTcABytes + nb_cta * 128;
        // two K chunks per stage (half as many waits and commits per MMA) wherever the ring then
        // still has three stages
        const int room = idx->smem_optin - p.off_stage;
        p.stage_chunks = (p.nchunks >= 2 && room / (2 * p.chunk_bytes) >= 3) ? 2 : 1;
        p.stage_bytes = p.stage_chunks * p.chunk_bytes;
        p.stages = std::min(kTcMaxStages, room / p.stage_bytes);
        if (p.stages < 2) return RALM_ERR_UNSUPPORTED;
        const int smem = p.off_stage + p.stages * p.stage_bytes;
        if (!encode_rows_map(&map_q, queries, sp, idx->d, nb_cta)) return RALM_ERR_CUDA;
        void (*single)(CUtensorMap, CUtensorMap, TcParams) =
            mode == 0 ? scan_tc_kernel<false, 0> : mode == 1 ? scan_tc_kernel<false, 1>
            : mode == 2 ? scan_tc_kernel<false, 2> : scan_tc_kernel<false, 3>;
        void (*paired)(CUtensorMap, CUtensorMap, TcParams) =
            mode == 0 ? scan_tc_kernel<true, 0> : mode == 1 ? scan_tc_kernel<true, 1>
            : mode == 2 ? scan_tc_kernel<true, 2> : scan_tc_kernel<true, 3>;
        if (!pair) {
            const int grid = static_cast<int>(std::min<long long>(idx->num_sms, p.ntiles));
            if (cudaFuncSetAttribute(single, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
                return RALM_ERR_CUDA;
            single<<<grid, kTcThreads, smem, st>>>(map_x, map_q, p);
            *grid_out = grid;
            return cudaGetLastError() == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
        }
        if (cudaFuncSetAttribute(paired, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return RALM_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.gridDim = dim3(2, 1, 1);
        cfg.blockDim = dim3(kTcThreads, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (idx->tc_clusters < 0) {
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, paired, &cfg) != cudaSuccess) {
                cudaGetLastError();
                n = 0;
            }
            idx->tc_clusters = std::min(n, idx->num_sms / 2);
        }
        if (idx->tc_clusters < 1) {  // no room for a pair on this device: single CTAs
            pair = false;
            continue;
        }
        const int clusters = static_cast<int>(std::min<long long>(idx->tc_clusters, p.ntiles));
        cfg.gridDim = dim3(2 * clusters, 1, 1);
        *grid_out = 2 * clusters;
        return cudaLaunchKernelEx(&cfg, paired, map_x, map_q, p) == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
    }
}

constexpr int kTcAutoMinQueries = 9;     // batches the 8-query scan cannot serve in one pass
// From how many queries the automatic variant takes the tcgen05 scan (measured on 21 M x 768 and
// 50 M x 1024): inner product, k = 1: 16 queries 4.42 against 4.34 ms for the two-group warp-MMA
// pass, 24 queries 4.44 against 5.3 ms; k = 20: 12 queries 4.42 against 4.74 ms; L2 9 queries 14.9
// against 16.4 ms. On corpora too small for a sample launch the small-batch scan keeps batches of
// up to 32 inner-product queries.
constexpr int kTcAutoMinQueriesIp = 17;      // k == 1
constexpr int kTcAutoMinQueriesIpTopK = 9;   // k > 1
constexpr int kTcAutoMinQueriesIpSmall = 33;
constexpr int kTcAutoMinQueriesL2 = 9;

// Final merge of `lists` partial lists per query into ids and scores. One CTA per query walks
// through its lists one after the other; with few queries and long lists (4 queries, 148 lists of
// 1024 keys: 0.33 ms) the lists are first merged in kMergeGroups groups side by side, then the
// groups' results.
ralm_status_t final_merge(ralm_index *idx, int lists, int s, int k, bool l2, int64_t *ids, float *scores,
                          int extra_slot, cudaStream_t st) {
    const int all_lists = lists + (extra_slot >= 0 ? 1 : 0);
    if (idx->merge_tmp && s <= kMergeTwoLevelMaxS && all_lists >= 4 * kMergeGroups &&
        static_cast<long long>(all_lists) * k > kMergeSortMax) {
        merge_kernel<<<dim3(s, kMergeGroups), kMergeThreads, 0, st>>>(idx->partial, lists, s, k, l2 ? 1 : 0, nullptr, nullptr,
                                                                   idx->merge_tmp, nullptr, extra_slot);
        if (cudaGetLastError() != cudaSuccess) return RALM_ERR_CUDA;
        merge_kernel<<<s, kMergeThreads, 0, st>>>(idx->merge_tmp, kMergeGroups, s, k, l2 ? 1 : 0, ids, scores, nullptr,
                                                  nullptr, -1);
        if (cudaGetLastError() != cudaSuccess) return RALM_ERR_CUDA;
        idx->launches += 2;
        return RALM_OK;
    }
    merge_kernel<<<s, kMergeThreads, 0, st>>>(idx->partial, lists, s, k, l2 ? 1 : 0, ids, scores, nullptr, nullptr, extra_slot);
    if (cudaGetLastError() != cudaSuccess) return RALM_ERR_CUDA;
    idx->launches++;
    return RALM_OK;
}

ralm_status_t search_device(ralm_index *idx, const __half *queries, int s, int k, int64_t *ids,
                            float *scores, cudaStream_t st) {
    if (s == 0) return RALM_OK;
    // (rows too long for two 16-row stages of the small-batch scan also go to the tcgen05 scan,
    // whose stages hold 64 columns at a time)
    ScanPlan probe;
    const bool small_scan_fits = plan_scan(idx, true, kScanMaxQueries, k, &probe);
    // L2 on this path always runs sample first (the sample is what keeps its exact rescoring
    // rare), so it needs a corpus large enough for one
    const long long tc_rows = 2 * kTcTileM;
    // (a larger sample for large k: the k-th largest of the launch's 4 maxima per CTA is a tighter
    // threshold when each maximum is taken over more rows, and at k = 256 the rows that still pass
    // it in the main launch cost more than the longer sample launch)
    long long tc_sample = std::max<long long>(idx->N / (k > kTcSmallK ? 16 : 64), 4LL * idx->num_sms * kTcTileM);
    tc_sample = (tc_sample + tc_rows - 1) / tc_rows * tc_rows;
    const bool tc_two_phase = tc_sample * 8 <= idx->N && idx->tc_two_phase;
    const bool l2 = idx->metric == RALM_L2;
    // (L2 rows too long for the small-batch scan take this path on any corpus: without a sample
    // every pair passes the filter and is scored again, which is slow but small corpora are small)
    const int tc_from = l2 ? kTcAutoMinQueriesL2
                           : (tc_two_phase ? (k > 1 ? kTcAutoMinQueriesIpTopK : kTcAutoMinQueriesIp) : kTcAutoMinQueriesIpSmall);
    const bool tc_auto = !small_scan_fits || ((tc_two_phase || !l2) && s >= tc_from);
    const bool tc = tc_can_serve(idx, k) && (!l2 || tc_two_phase || !small_scan_fits) &&
                    (idx->variant == 3 || idx->variant == 4 || (idx->variant == 0 && tc_auto));
    if (tc) {
        // Large corpora are scanned in two phases: a small sample first, which gives every query a
        // score that k rows are known to reach; the scan proper then starts from those thresholds,
        // so that hardly any score passes and the selection stays off the critical path.
        const long long sample = tc_sample;
        const bool two_phase = tc_two_phase;
        int grid = 0;
        const int per_pass = std::min(kTcMaxQueries, idx->tc_cand_q);
        idx->last_kernel = idx->variant == 4 ? 4 : 3;
        idx->last_passes = (s + per_pass - 1) / per_pass;
        idx->last_phases = two_phase ? 3 : 1;
        idx->last_sample_rows = two_phase ? sample : 0;
        for (int q0 = 0; idx->N > 0 && q0 < s; q0 += per_pass) {
            const int sp = std::min(per_pass, s - q0);
            const __half *qp = queries + static_cast<size_t>(q0) * idx->d;
            TimedEvents ev{nullptr, nullptr};
            if (!timing_begin(idx, st, &ev)) return RALM_ERR_CUDA;
            ralm_status_t rs = RALM_OK;
            if (two_phase) {
                int grid1 = 0;
                // the sample launch keeps no lists: its selection warps write their best rank value
                // per query (L2: best lower bound), and the k-th largest of a query's maxima is the
                // threshold; the main launch then scans every row, the sample's too
                rs = launch_tc_pass(idx, qp, sp, s, q0, k, idx->variant != 4, 0, sample, nullptr, l2 ? 1 : 3,
                                    &grid1, st);
                if (rs == RALM_OK) {
                    kth_of_maxima_kernel<<<sp, kMergeThreads, 0, st>>>(idx->tc_gmax + q0, grid1 * 4, s, k,
                                                                       idx->tc_thr + q0);
                    if (cudaGetLastError() != cudaSuccess) rs = RALM_ERR_CUDA;
                }
                if (rs == RALM_OK)
                    rs = launch_tc_pass(idx, qp, sp, s, q0, k, idx->variant != 4, 0, idx->N, idx->tc_thr,
                                        l2 ? 2 : 0, &grid, st);
                idx->launches += 2;
            } else {
                rs = launch_tc_pass(idx, qp, sp, s, q0, k, idx->variant != 4, 0, idx->N, nullptr, l2 ? 2 : 0, &grid, st);
            }
            timing_end(idx, st, ev);
            if (rs != RALM_OK) return rs;
            idx->launches++;
        }
        return final_merge(idx, grid, s, k, l2, ids, scores, -1, st);
    }
    const int variant = resolve_variant(idx);
    const bool mma = variant == 2;
    if (!mma && idx->d > kFmaMaxD) return RALM_ERR_UNSUPPORTED;
    // warp-MMA flavour: up to four groups of 8 queries share every staged tile when the batch
    // has more than 8 (the tile is read from HBM once)
    const bool wide = mma && s > kScanMaxQueries && (idx->metric == RALM_IP || idx->norms != nullptr);
    // (L2 stops at two groups: with four, its filter and rescoring cost more than a second pass)
    const int wide_pass = idx->metric == RALM_L2 ? 16 : kScanMaxPassQueries;
    // An index with an 8-bit copy (ralm_index_enable_q8) streams that copy for batches of up to 16
    // queries and scores again, exactly, what its filter lets through; the sample is scanned in
    // fp16 also for k == 1, since the filter needs thresholds to be of any use.
    ScanPlan pl8;
    // (only where a sample phase is possible: without thresholds nearly every pair passes the filter)
    const long long q8_sample = (std::max<long long>(idx->N / 128, 4LL * idx->num_sms * kTcTileM) + 255) / 256 * 256;
    // (two query groups only pay at k == 1: 16 queries 3.6 ms against 4.3; at k = 20 4.8 against 4.7 fp16)
    const bool use_q8 = idx->x8 && (idx->metric == RALM_IP || idx->norms) && idx->variant == 0 && s <= kQ8MaxQueries &&
                        (s <= kScanMaxQueries || k == 1 || idx->x8_force) &&
                        (idx->x8_force || (idx->tc_thr && idx->tc_two_phase && q8_sample * 32 <= idx->N)) &&
                        plan_scan_q8(idx, s, k, &pl8);
    const int per_pass = use_q8 ? kQ8MaxQueries : mma ? (wide ? wide_pass : kScanMaxQueries) : kFmaQueriesPerPass;
    // k > 1 on a large corpus: scan a sample first and start the rest from the sample's merged
    // k-th scores (see the large-batch path above); the sample's list is block num_sms of `partial`
    // (1/128 of the rows here: measured best for this scan; the large-batch scan prefers 1/64)
    long long sample = std::max<long long>(idx->N / 128, 4LL * idx->num_sms * kTcTileM);
    sample = (sample + 255) / 256 * 256;
    // (two more launches: only worth it when the scan itself takes a millisecond or more)
    const bool two_phase = (k > 1 || use_q8) && idx->tc_thr && idx->tc_two_phase && sample * 32 <= idx->N;
    // large k: the sample launch only takes per-warp maxima (needs the stored norms for L2, and as
    // many warps in the sample launch as k asks for)
    const bool maxima_sample = two_phase && mma && k >= kPubMinK && idx->scan_gmax &&
                               (idx->metric == RALM_IP || idx->norms) &&
                               k <= std::min<long long>(idx->num_sms, sample / 16) * 4 * kGmaxSlots &&
                               idx->num_sms * kMaxConsumerWarps * kGmaxSlots <= kMaximaSortMax;
    int grid = 0;
    idx->last_kernel = use_q8 ? 5 : (mma ? 2 : 1);
    idx->last_passes = (s + per_pass - 1) / per_pass;
    idx->last_phases = two_phase ? (maxima_sample ? 3 : 2) : 1;
    idx->last_sample_rows = two_phase ? sample : 0;
    for (int q0 = 0; idx->N > 0 && q0 < s; q0 += per_pass) {
        const int sp = std::min(per_pass, s - q0);
        ScanPlan pl;
        if (!plan_scan(idx, mma, sp, k, &pl)) return RALM_ERR_UNSUPPORTED;
        ScanParams p;
        p.corpus = idx->corpus;
        p.queries = queries + static_cast<size_t>(q0) * idx->d;
        p.norms = idx->norms;
        p.x8 = nullptr;
        p.sqnorms = nullptr;
        p.pub = nullptr;
        p.pub_rank = 0;
        p.gmax = nullptr;
        p.gmax_slots = 1;
        p.gmax_len = 0;
        p.ext = index_extents(idx, idx->spill ? static_cast<long long>(idx->num_sms) * kScanMaxPassQueries * idx->spill_cap : 0);
        p.spill = pl.spill ? idx->spill : nullptr;
        p.partial = idx->partial;
        p.status = idx->status;
        p.d = idx->d;
        p.s = sp;
        p.s_total = s;
        p.q_base = q0;
        p.k = k;
        p.cap = pl.cap;
        p.soft_limit = pl.soft_limit;
        p.tile_rows = pl.tile_rows;
        p.nwarps = pl.nwarps;
        p.depth = pl.depth;
        p.stage_bytes = pl.stage_bytes;
        p.off_q = pl.off_q;
        p.off_cand = pl.off_cand;
        p.off_stage = pl.off_stage;
        // bound on the rounding error of the tensor-core |x|^2 - 2 x.q + |q|^2 relative to
        // |x|^2 + |q|^2: d accumulation steps of at most 2^-22 each, on terms that sum to
        // at most twice that scale
        p.l2_slack = static_cast<float>(idx->d) * (1.0f / 2097152.0f);
        // one launch over rows [begin, end) starting from the given thresholds
        auto scan_rows = [&](long long begin, long long end, const float *thr_init, int *grid_out) -> cudaError_t {
            p.row_begin = begin;
            p.N = end;
            p.thr_init = thr_init;
            p.ntiles = (end - begin + pl.tile_rows - 1) / pl.tile_rows;
            // the same grid whatever the tile height of the pass: the merge reads one list per CTA
            const int g = static_cast<int>(std::min<long long>(idx->num_sms, (end - begin + 15) / 16));
            *grid_out = g;
            p.pub = (idx->pub && k >= kPubMinK && g > 1) ? idx->pub : nullptr;
            p.pub_rank = p.pub ? (k + g - 1) / g : 0;
            if (p.pub && cudaMemsetAsync(idx->pub, 0, sizeof(uint32_t) * idx->num_sms * static_cast<size_t>(idx->max_s), st) !=
                             cudaSuccess)
                return cudaErrorUnknown;
            if (mma && idx->metric == RALM_L2 && idx->norms && sp > kScanMaxQueries)
                return (k == 1) ? launch_scan<true, true, 16, 1, true, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, true, 16, 1, false, true>(p, g, pl.smem_bytes, st);
            if (mma && idx->metric == RALM_L2 && idx->norms)
                return (k == 1) ? launch_scan<true, true, 8, 1, true, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, true, 8, 1, false, true>(p, g, pl.smem_bytes, st);
            if (mma && idx->metric == RALM_L2)
                return (k == 1) ? launch_scan<true, true, 8, 1, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, true, 8, 1, false>(p, g, pl.smem_bytes, st);
            if (mma && sp > 16)
                return (k == 1) ? launch_scan<true, false, 32, 1, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, false, 32, 1, false>(p, g, pl.smem_bytes, st);
            if (mma && sp > kScanMaxQueries)
                return (k == 1) ? launch_scan<true, false, 16, 1, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, false, 16, 1, false>(p, g, pl.smem_bytes, st);
            if (mma)
                return (k == 1) ? launch_scan<true, false, 8, 1, true>(p, g, pl.smem_bytes, st)
                                : launch_scan<true, false, 8, 1, false>(p, g, pl.smem_bytes, st);
            return idx->metric == RALM_L2 ? launch_fma<true>(p, g, pl.smem_bytes, st)
                                          : launch_fma<false>(p, g, pl.smem_bytes, st);
        };
        // Sample launch for large k: the k == 1 kernels over rows [0, end), every consumer warp writing
        // the best rank value of its rows (ScanParams::gmax); then the k-th largest of a query's maxima
        // becomes its threshold. No lists, no merge: a fraction of what the sample costs otherwise at
        // k = 1024 (1.1 ms of scan and 0.3 ms of merge on 50 M x 1024).
        auto sample_by_maxima = [&](long long end) -> cudaError_t {
            ScanPlan ps;
            if (!plan_scan(idx, true, sp, 1, &ps, true)) return cudaErrorUnknown;
            ScanParams q = p;
            q.spill = nullptr;
            q.k = 1;
            q.cap = 0;
            q.soft_limit = 0;
            q.tile_rows = ps.tile_rows;
            q.nwarps = ps.nwarps;
            q.depth = ps.depth;
            q.stage_bytes = ps.stage_bytes;
            q.off_q = ps.off_q;
            q.off_cand = ps.off_cand;
            q.off_stage = ps.off_stage;
            q.row_begin = 0;
            q.N = end;
            q.thr_init = nullptr;
            q.ntiles = (end + ps.tile_rows - 1) / ps.tile_rows;
            q.gmax = idx->scan_gmax;
            q.gmax_slots = kGmaxSlots;
            q.gmax_len = static_cast<long long>(idx->num_sms) * kMaxConsumerWarps * kGmaxSlots * idx->max_s;
            const int g = static_cast<int>(std::min<long long>(idx->num_sms, (end + 15) / 16));
            cudaError_t ke;
            if (idx->metric == RALM_L2 && sp > kScanMaxQueries) ke = launch_scan<true, true, 16, 1, true, true>(q, g, ps.smem_bytes, st);
            else if (idx->metric == RALM_L2) ke = launch_scan<true, true, 8, 1, true, true>(q, g, ps.smem_bytes, st);
            else if (sp > 16) ke = launch_scan<true, false, 32, 1, true>(q, g, ps.smem_bytes, st);
            else if (sp > kScanMaxQueries) ke = launch_scan<true, false, 16, 1, true>(q, g, ps.smem_bytes, st);
            else ke = launch_scan<true, false, 8, 1, true>(q, g, ps.smem_bytes, st);
            if (ke != cudaSuccess) return ke;
            kth_of_maxima_kernel<<<sp, kMergeThreads, 0, st>>>(idx->scan_gmax + q0, g * ps.nwarps * kGmaxSlots, s, k,
                                                               idx->tc_thr + q0);
            return cudaGetLastError();
        };
        auto scan_rows_q8 = [&](long long begin, long long end, const float *thr_init, int *grid_out) -> cudaError_t {
            ScanParams p8 = p;
            p8.x8 = idx->x8;
            p8.norms = idx->x8_bound;
            p8.sqnorms = idx->norms;
            p8.spill = pl8.spill ? idx->spill : nullptr;
            p8.cap = pl8.cap;
            p8.soft_limit = pl8.soft_limit;
            p8.tile_rows = pl8.tile_rows;
            p8.nwarps = pl8.nwarps;
            p8.depth = pl8.depth;
            p8.stage_bytes = pl8.stage_bytes;
            p8.off_q = pl8.off_q;
            p8.off_cand = pl8.off_cand;
            p8.off_stage = pl8.off_stage;
            p8.row_begin = begin;
            p8.N = end;
            p8.thr_init = thr_init;
            p8.ntiles = (end - begin + pl8.tile_rows - 1) / pl8.tile_rows;
            const int g = static_cast<int>(std::min<long long>(idx->num_sms, (end - begin + 15) / 16));
            *grid_out = g;
            p8.pub = (idx->pub && k >= kPubMinK && g > 1) ? idx->pub : nullptr;
            p8.pub_rank = p8.pub ? (k + g - 1) / g : 0;
            if (p8.pub && cudaMemsetAsync(idx->pub, 0, sizeof(uint32_t) * idx->num_sms * static_cast<size_t>(idx->max_s), st) !=
                              cudaSuccess)
                return cudaErrorUnknown;
            auto kern = (k == 1) ? scan_q8_kernel<true, 1> : scan_q8_kernel<false, 1>;
            if (sp > kScanMaxQueries) kern = (k == 1) ? scan_q8_kernel<true, 2> : scan_q8_kernel<false, 2>;
            if (idx->metric == RALM_L2) {
                kern = (k == 1) ? scan_q8_kernel<true, 1, true> : scan_q8_kernel<false, 1, true>;
                if (sp > kScanMaxQueries) kern = (k == 1) ? scan_q8_kernel<true, 2, true> : scan_q8_kernel<false, 2, true>;
            }
            cudaError_t ke = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, pl8.smem_bytes);
            if (ke != cudaSuccess) return ke;
            kern<<<g, 32 * (pl8.nwarps + 1), pl8.smem_bytes, st>>>(p8);
            return cudaGetLastError();
        };
        cudaError_t e;
        TimedEvents ev{nullptr, nullptr};
        if (!timing_begin(idx, st, &ev)) return RALM_ERR_CUDA;
        if (maxima_sample) {
            // (the scan proper then covers every row, the sample's too)
            e = sample_by_maxima(sample);
            if (e == cudaSuccess) e = use_q8 ? scan_rows_q8(0, idx->N, idx->tc_thr, &grid) : scan_rows(0, idx->N, idx->tc_thr, &grid);
            idx->launches += 2;
        } else if (use_q8) {
            if (two_phase) {
                int grid1 = 0;
                e = scan_rows(0, sample, nullptr, &grid1);
                if (e == cudaSuccess) {
                    merge_kernel<<<sp, kMergeThreads, 0, st>>>(
                        idx->partial + static_cast<size_t>(q0) * k, grid1, s, k, 0, nullptr, nullptr,
                        idx->partial + (static_cast<size_t>(idx->num_sms) * s + q0) * k, idx->tc_thr + q0);
                    e = cudaGetLastError();
                }
                if (e == cudaSuccess) e = scan_rows_q8(sample, idx->N, idx->tc_thr, &grid);
                idx->launches += 2;
            } else {
                e = scan_rows_q8(0, idx->N, nullptr, &grid);
            }
        } else if (two_phase) {
            int grid1 = 0;
            e = scan_rows(0, sample, nullptr, &grid1);
            if (e == cudaSuccess) {
                merge_kernel<<<sp, kMergeThreads, 0, st>>>(
                    idx->partial + static_cast<size_t>(q0) * k, grid1, s, k, idx->metric == RALM_L2, nullptr,
                    nullptr, idx->partial + (static_cast<size_t>(idx->num_sms) * s + q0) * k, idx->tc_thr + q0);
                e = cudaGetLastError();
            }
            if (e == cudaSuccess) e = scan_rows(sample, idx->N, idx->tc_thr, &grid);
            idx->launches += 2;
        } else {
            e = scan_rows(0, idx->N, nullptr, &grid);
        }
        timing_end(idx, st, ev);
        if (e != cudaSuccess) return RALM_ERR_CUDA;
        idx->launches++;
    }
    return final_merge(idx, grid, s, k, idx->metric == RALM_L2, ids, scores,
                       (two_phase && !maxima_sample) ? idx->num_sms : -1, st);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// ---------------------------------------------------------------------------------------
// Scratch for ralm_search_static. It lives in the library image itself: every GPU that loads
// the library holds these bytes until the process exits, whether or not the call is used.
// Layout: [blocks][s][k] sorted partial top-k keys, exactly what the scan hands to the merge.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned long long
    g_static_partial[RALM_STATIC_MAX_BLOCKS * RALM_STATIC_MAX_S * RALM_STATIC_MAX_K];
static __device__ __align__(256) int g_static_status[64];

namespace {

constexpr int kStaticMaxDevices = 64;

struct StaticDeviceState {
    bool ready = false;
    uint64_t *partial = nullptr;  // device address of g_static_partial on this device
    int *status = nullptr;        // device address of g_static_status on this device
    int num_sms = 0;
    int smem_optin = 0;
    int cc_major = 0;
};
StaticDeviceState g_static_state[kStaticMaxDevices];
std::mutex g_static_mutex;

// One-time set-up per device, with that device current. In host code the array names above
// are only handles; the addresses a kernel can use come from cudaGetSymbolAddress.
ralm_status_t static_state_for_current_device(StaticDeviceState **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RALM_ERR_CUDA;
    if (dev < 0 || dev >= kStaticMaxDevices) return RALM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState &st = g_static_state[dev];
    if (!st.ready) {
        void *partial = nullptr, *status = nullptr;
        if (cudaGetSymbolAddress(&partial, g_static_partial) != cudaSuccess) return RALM_ERR_CUDA;
        if (cudaGetSymbolAddress(&status, g_static_status) != cudaSuccess) return RALM_ERR_CUDA;
        int sms = 0, smem = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return RALM_ERR_CUDA;
        st.partial = static_cast<uint64_t *>(partial);
        st.status = static_cast<int *>(status);
        st.num_sms = sms;
        st.smem_optin = smem;
        st.cc_major = major;
        st.ready = true;
    }
    *out = &st;
    return RALM_OK;
}

}  // namespace

extern "C" {

ralm_status_t ralm_index_create(const void *corpus, int64_t N, int32_t d, ralm_metric_t metric,
                                int32_t max_s, int32_t max_k, ralm_index_t **out) {
    if (!out) return RALM_ERR_INVALID_ARG;
    *out = nullptr;
    if (N < 0 || N >= (int64_t{1} << 31)) return RALM_ERR_INVALID_ARG;
    if (!corpus && N > 0) return RALM_ERR_INVALID_ARG;
    if (!aligned16(corpus)) return RALM_ERR_INVALID_ARG;
    if (d < 8 || d > RALM_MAX_D || d % 8 != 0) return RALM_ERR_INVALID_ARG;
    if (metric != RALM_IP && metric != RALM_L2) return RALM_ERR_INVALID_ARG;
    if (max_s < 1 || max_s > RALM_MAX_QUERIES || max_k < 1 || max_k > RALM_MAX_K)
        return RALM_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RALM_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return RALM_ERR_CUDA;
    if (prop.major != 10) return RALM_ERR_UNSUPPORTED;
    ralm_index *idx = new (std::nothrow) ralm_index();
    if (!idx) return RALM_ERR_OOM;
    idx->corpus = static_cast<const __half *>(corpus);
    idx->N = N;
    idx->d = d;
    idx->metric = metric;
    idx->max_s = max_s;
    idx->max_k = max_k;
    idx->device = dev;
    idx->num_sms = prop.multiProcessorCount;
    idx->smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    idx->variant = 0;
    idx->tune_warps = idx->tune_depth = idx->tune_rows = 0;
    idx->launches = 0;
    idx->timing = false;
    idx->last_kernel = idx->last_passes = idx->last_phases = 0;
    idx->last_sample_rows = 0;
    // one list per scan CTA and query, plus one more block for the list of a sample phase
    const size_t partial_bytes = sizeof(uint64_t) * (idx->num_sms + 1) * max_s * static_cast<size_t>(max_k);
    const size_t sk = static_cast<size_t>(max_s) * max_k;
    idx->tc_cand = nullptr;
    idx->tc_cand_q = 0;
    idx->tc_cand_cap = 0;
    idx->tc_clusters = -1;
    idx->tc_thr = nullptr;
    idx->tc_gmax = nullptr;
    idx->tc_tile_counter = nullptr;
    idx->tc_two_phase = true;
    idx->norms = nullptr;
    idx->x8 = nullptr;
    idx->x8_bound = nullptr;
    idx->x8_force = false;
    idx->spill = nullptr;
    idx->spill_cap = 0;
    idx->pub = nullptr;
    idx->scan_gmax = nullptr;
    idx->merge_tmp = nullptr;
    cudaError_t first_error = cudaSuccess;
    auto alloc = [&first_error](auto **ptr, size_t bytes) {
        if (first_error == cudaSuccess) first_error = device_alloc(ptr, bytes);
    };
    alloc(&idx->partial, partial_bytes);
    idx->partial_keys = static_cast<long long>(partial_bytes / sizeof(uint64_t));
    alloc(&idx->tc_thr, sizeof(float) * max_s);
    if (static_cast<long long>(idx->num_sms + 1) * max_k > kMergeSortMax)
        alloc(&idx->merge_tmp, sizeof(uint64_t) * kMergeGroups * kMergeTwoLevelMaxS * static_cast<size_t>(max_k));
    const int pass_queries = std::min(max_s, kScanMaxPassQueries);
    if (max_k > 1 && std::max(512, 2 * next_pow2(max_k)) * 8 * pass_queries > kSmemCandBytes) {
        idx->spill_cap = std::max(512, 2 * next_pow2(max_k));
        alloc(&idx->spill, sizeof(uint64_t) * idx->num_sms * kScanMaxPassQueries * static_cast<size_t>(idx->spill_cap));
    }
    if (max_k >= kPubMinK) alloc(&idx->pub, sizeof(uint32_t) * idx->num_sms * static_cast<size_t>(max_s));
    if (max_k >= kPubMinK)
        alloc(&idx->scan_gmax, sizeof(float) * idx->num_sms * kMaxConsumerWarps * kGmaxSlots * static_cast<size_t>(max_s));
    if (metric == RALM_L2 && N > 0) alloc(&idx->norms, sizeof(float) * N);
    ScanPlan probe;
    const bool small_scan_fits = plan_scan(idx, true, kScanMaxQueries, 1, &probe);
    if ((max_s >= kTcAutoMinQueries || !small_scan_fits) && d >= kTcChunkK &&
        first_error == cudaSuccess &&
        !alloc_tc_workspace(idx, std::min(kTcMaxQueries, align_up(max_s, 16))))
        first_error = cudaErrorMemoryAllocation;
    alloc(&idx->cache_keys, sizeof(uint64_t) * RALM_MAX_CACHE_KEYS);
    alloc(&idx->status, sizeof(int));
    alloc(&idx->h_queries, static_cast<size_t>(max_s) * d * 2);
    alloc(&idx->h_ids, sk * sizeof(int64_t));
    alloc(&idx->h_scores, sk * sizeof(float));
    if (first_error != cudaSuccess) {
        cudaGetLastError();  // clear the runtime's sticky copy of an allocation failure
        ralm_index_destroy(idx);
        return first_error == cudaErrorMemoryAllocation ? RALM_ERR_OOM : RALM_ERR_CUDA;
    }
    if (cudaMemset(idx->status, 0, sizeof(int)) != cudaSuccess) {
        ralm_index_destroy(idx);
        return RALM_ERR_CUDA;
    }
    if (idx->norms) {
        // one pass over the corpus; the filter of the L2 scan reads these instead of recomputing
        const int blocks = static_cast<int>(std::min<long long>((N + 7) / 8, 32LL * idx->num_sms));
        row_norm_kernel<<<blocks, 256>>>(idx->corpus, N, d, idx->norms);
        if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
            ralm_index_destroy(idx);
            return RALM_ERR_CUDA;
        }
    }
    // benchmarking aid: RALM_FORCE_VARIANT=<n> pins the scan variant of every new index, as
    // ralm_index_set_variant(n) would (ignored when that variant cannot serve the index)
    if (const char *forced = std::getenv("RALM_FORCE_VARIANT")) {
        const int v = std::atoi(forced);
        if (v >= 1 && v <= 4) ralm_index_set_variant(idx, v);
    }
    *out = idx;
    return RALM_OK;
}

ralm_status_t ralm_index_destroy(ralm_index_t *idx) {
    if (!idx) return RALM_OK;
    cudaFree(idx->partial);
    cudaFree(idx->cache_keys);
    cudaFree(idx->merge_tmp);
    cudaFree(idx->tc_cand);
    cudaFree(idx->tc_thr);
    cudaFree(idx->tc_gmax);
    cudaFree(idx->tc_tile_counter);
    cudaFree(idx->norms);
    cudaFree(idx->x8);
    cudaFree(idx->x8_bound);
    cudaFree(idx->spill);
    cudaFree(idx->pub);
    cudaFree(idx->scan_gmax);
    cudaFree(idx->status);
    cudaFree(idx->h_queries);
    cudaFree(idx->h_ids);
    cudaFree(idx->h_scores);
    for (auto *list : {&idx->timed, &idx->spare})
        for (auto &ev : *list) {
            cudaEventDestroy(ev.first);
            cudaEventDestroy(ev.second);
        }
    delete idx;
    return RALM_OK;
}

ralm_status_t ralm_search(ralm_index_t *idx, const void *queries, int32_t s, int32_t k,
                          int64_t *ids, float *scores, void *stream) {
    if (!idx || s < 0 || s > idx->max_s || k < 1 || k > idx->max_k) return RALM_ERR_INVALID_ARG;
    if (s == 0) return RALM_OK;
    if (!queries || !ids || !scores || !aligned16(queries)) return RALM_ERR_INVALID_ARG;
    return search_device(idx, static_cast<const __half *>(queries), s, k, ids, scores,
                         static_cast<cudaStream_t>(stream));
}

ralm_status_t ralm_search_host(ralm_index_t *idx, const void *queries_host, int32_t s, int32_t k,
                               int64_t *ids_host, float *scores_host, void *stream) {
    if (!idx || s < 0 || s > idx->max_s || k < 1 || k > idx->max_k) return RALM_ERR_INVALID_ARG;
    if (s == 0) return RALM_OK;
    if (!queries_host || !ids_host || !scores_host) return RALM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t sk = static_cast<size_t>(s) * k;
    if (cudaMemcpyAsync(idx->h_queries, queries_host, static_cast<size_t>(s) * idx->d * 2,
                        cudaMemcpyHostToDevice, st) != cudaSuccess)
        return RALM_ERR_CUDA;
    ralm_status_t rs = search_device(idx, idx->h_queries, s, k, idx->h_ids, idx->h_scores, st);
    if (rs != RALM_OK) return rs;
    if (cudaMemcpyAsync(ids_host, idx->h_ids, sk * sizeof(int64_t), cudaMemcpyDeviceToHost, st) !=
            cudaSuccess ||
        cudaMemcpyAsync(scores_host, idx->h_scores, sk * sizeof(float), cudaMemcpyDeviceToHost, st) !=
            cudaSuccess)
        return RALM_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_cache_search(ralm_index_t *idx, const int64_t *cache_ids, int32_t R, int32_t C,
                                const void *queries, int32_t q, int32_t k, int64_t *ids,
                                float *scores, void *stream) {
    if (!idx || R < 0 || C < 1 || C > RALM_MAX_CACHE || q < 1 || k < 1 || k > idx->max_k)
        return RALM_ERR_INVALID_ARG;
    if (R == 0) return RALM_OK;
    if (!cache_ids || !queries || !ids || !scores || !aligned16(queries)) return RALM_ERR_INVALID_ARG;
    const int Cp = next_pow2(C);
    if (static_cast<long long>(R) * q * Cp > RALM_MAX_CACHE_KEYS) return RALM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid(R, (Cp + kCacheSlotsPerCta - 1) / kCacheSlotsPerCta);
    cache_score_kernel<<<grid, kCacheThreads, 0, st>>>(idx->corpus, idx->N, idx->d,
                                                       idx->metric == RALM_L2, cache_ids, C, Cp,
                                                       static_cast<const __half *>(queries), q,
                                                       idx->cache_keys, idx->status);
    if (cudaGetLastError() != cudaSuccess) return RALM_ERR_CUDA;
    cache_rank_kernel<<<R * q, kMergeThreads, 0, st>>>(idx->cache_keys, Cp, k, idx->metric == RALM_L2,
                                                       ids, scores);
    if (cudaGetLastError() != cudaSuccess) return RALM_ERR_CUDA;
    idx->launches += 2;
    return RALM_OK;
}

ralm_status_t ralm_verify(const int64_t *speculated_ids, const int64_t *retrieved_ids, int32_t R,
                          int32_t stride, int32_t ld, int32_t cmp_k, int32_t *first_mismatch,
                          void *stream) {
    if (R < 0 || stride < 0 || cmp_k < 1 || ld < cmp_k) return RALM_ERR_INVALID_ARG;
    if (R == 0) return RALM_OK;
    if (!first_mismatch) return RALM_ERR_INVALID_ARG;
    if (stride > 0 && (!speculated_ids || !retrieved_ids)) return RALM_ERR_INVALID_ARG;
    verify_kernel<<<(R + 3) / 4, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        speculated_ids, retrieved_ids, R, stride, ld, cmp_k, first_mismatch);
    return cudaGetLastError() == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_cache_update(int64_t *cache_ids, int32_t *cursor, int32_t R, int32_t C,
                                const int64_t *retrieved_ids, int32_t stride, int32_t ld, int32_t top,
                                const int32_t *steps, int32_t next_n, int64_t N, void *stream) {
    if (R < 0 || C < 1 || C > RALM_MAX_CACHE || stride < 0 || top < 1 || ld < top || next_n < 0 || N < 0)
        return RALM_ERR_INVALID_ARG;
    if (R == 0 || stride == 0) return RALM_OK;
    if (!cache_ids || !cursor || !retrieved_ids) return RALM_ERR_INVALID_ARG;
    cache_update_kernel<<<R, kCacheUpdateThreads, static_cast<size_t>(C) * sizeof(int64_t),
                          static_cast<cudaStream_t>(stream)>>>(cache_ids, cursor, C, retrieved_ids, stride, ld,
                                                               top, steps, next_n, N);
    return cudaGetLastError() == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_merge_lists(const int64_t *ids, const float *scores, const int64_t *row_offset, int32_t G,
                               int32_t s, int32_t k, ralm_metric_t metric, int64_t *out_ids, float *out_scores,
                               void *stream) {
    if (G < 1 || s < 0 || k < 1 || k > RALM_MAX_K || (metric != RALM_IP && metric != RALM_L2))
        return RALM_ERR_INVALID_ARG;
    if (s == 0) return RALM_OK;
    if (!ids || !scores || !row_offset || !out_ids || !out_scores) return RALM_ERR_INVALID_ARG;
    merge_lists_kernel<<<s, kMergeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        ids, scores, row_offset, G, s, k, metric == RALM_L2, out_ids, out_scores);
    return cudaGetLastError() == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_debug_fail_allocation(int32_t nth) {
    if (nth < 0) return RALM_ERR_INVALID_ARG;
    g_fail_allocation_in.store(nth);
    return RALM_OK;
}

ralm_status_t ralm_selftest_wait_timeout(int64_t limit_cycles, int32_t *device_status, void *stream) {
    if (!device_status || limit_cycles < 1 || limit_cycles > 2000000000LL) return RALM_ERR_INVALID_ARG;
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles, device_status);
    return cudaGetLastError() == cudaSuccess ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_device_status(ralm_index_t *idx, void *stream) {
    if (!idx) return RALM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, idx->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(idx->status, 0, sizeof(int), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return RALM_ERR_CUDA;
    if (word == kStatusTimeout) return RALM_ERR_TIMEOUT;
    if (word == kStatusBadCacheId) return RALM_ERR_BAD_CACHE_ID;
    if (word == kStatusInternal) return RALM_ERR_INTERNAL;
    return word == 0 ? RALM_OK : RALM_ERR_CUDA;
}

ralm_status_t ralm_index_set_variant(ralm_index_t *idx, int32_t variant) {
    if (!idx || variant < 0 || variant > 4) return RALM_ERR_INVALID_ARG;
    if (variant == 1 && idx->d > kFmaMaxD) return RALM_ERR_UNSUPPORTED;
    if (variant == 3 || variant == 4) {
        if ((idx->metric != RALM_IP && !idx->norms) || idx->d < kTcChunkK || !tensor_map_encoder())
            return RALM_ERR_UNSUPPORTED;
        if (!alloc_tc_workspace(idx, std::min(kTcMaxQueries, align_up(idx->max_s, 16)))) return RALM_ERR_OOM;
    }
    idx->variant = variant;
    return RALM_OK;
}

ralm_status_t ralm_index_enable_q8(ralm_index_t *idx, int32_t force) {
    if (!idx) return RALM_ERR_INVALID_ARG;
    if (idx->d % 16 != 0 || (idx->metric == RALM_L2 && idx->N > 0 && !idx->norms)) return RALM_ERR_UNSUPPORTED;
    idx->x8_force = force != 0;
    if (idx->x8 || idx->N == 0) return RALM_OK;
    ScanPlan probe;
    if (!plan_scan_q8(idx, 1, 1, &probe)) return RALM_ERR_UNSUPPORTED;
    uint8_t *x8 = nullptr;
    float *bound = nullptr;
    if (device_alloc(&x8, static_cast<size_t>(idx->N) * idx->d) != cudaSuccess ||
        device_alloc(&bound, sizeof(float) * idx->N) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(x8);
        return RALM_ERR_OOM;
    }
    if (!idx->spill && idx->max_k > kQ8MaxKWide) {
        // candidate lists of more than 256 slots live in global memory for this scan
        const int cap = std::max(512, 2 * next_pow2(idx->max_k));
        if (device_alloc(&idx->spill, sizeof(uint64_t) * idx->num_sms * kScanMaxPassQueries * static_cast<size_t>(cap)) !=
            cudaSuccess) {
            cudaGetLastError();
            idx->spill = nullptr;
            cudaFree(x8);
            cudaFree(bound);
            return RALM_ERR_OOM;
        }
        idx->spill_cap = cap;
    }
    const int blocks = static_cast<int>(std::min<long long>((idx->N + 7) / 8, 32LL * idx->num_sms));
    quantize_rows_kernel<<<blocks, 256>>>(idx->corpus, idx->N, idx->d, x8, bound);
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        cudaFree(x8);
        cudaFree(bound);
        return RALM_ERR_CUDA;
    }
    idx->x8 = x8;
    idx->x8_bound = bound;
    return RALM_OK;
}

ralm_status_t ralm_search_static(const void *corpus, int64_t N, int32_t d, ralm_metric_t metric,
                                 const void *queries, int32_t s, int32_t k, int64_t *ids,
                                 float *scores, int32_t *device_status, void *stream) {
    if (N < 0 || N >= (int64_t{1} << 31) || (!corpus && N > 0) || !aligned16(corpus))
        return RALM_ERR_INVALID_ARG;
    if (d < 8 || d > RALM_MAX_D || d % 8 != 0) return RALM_ERR_INVALID_ARG;
    if (metric != RALM_IP && metric != RALM_L2) return RALM_ERR_INVALID_ARG;
    if (s < 0 || k < 1) return RALM_ERR_INVALID_ARG;
    if (s > RALM_STATIC_MAX_S || k > RALM_STATIC_MAX_K) return RALM_ERR_STATIC_LIMIT;
    if (s > 0 && (!queries || !ids || !scores || !aligned16(queries))) return RALM_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (s == 0) {  // nothing to search; the caller's status word is still zeroed, as promised
        if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int), st) != cudaSuccess) return RALM_ERR_CUDA;
        return RALM_OK;
    }
    StaticDeviceState *dev = nullptr;
    ralm_status_t rs = static_state_for_current_device(&dev);
    if (rs != RALM_OK) return rs;
    if (dev->cc_major != 10) return RALM_ERR_UNSUPPORTED;
    int *status = device_status ? device_status : dev->status;
    // the scratch keeps whatever the previous call left; the partial lists are fully
    // rewritten by the scan, the status word is the one thing that must start at zero
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return RALM_ERR_CUDA;
    // a handle on the stack that points the ordinary search path at the static scratch
    ralm_index view;
    view.corpus = static_cast<const __half *>(corpus);
    view.N = N;
    view.d = d;
    view.metric = metric;
    view.max_s = RALM_STATIC_MAX_S;
    view.max_k = RALM_STATIC_MAX_K;
    view.device = 0;
    view.num_sms = std::min(dev->num_sms, RALM_STATIC_MAX_BLOCKS);
    view.smem_optin = dev->smem_optin;
    view.variant = 0;
    view.tune_warps = view.tune_depth = view.tune_rows = 0;
    view.partial = dev->partial;
    view.partial_keys = static_cast<long long>(RALM_STATIC_MAX_BLOCKS) * RALM_STATIC_MAX_S * RALM_STATIC_MAX_K;
    view.cache_keys = nullptr;
    view.merge_tmp = nullptr;
    view.tc_cand = nullptr;
    view.tc_cand_q = 0;
    view.tc_cand_cap = 0;
    view.tc_clusters = -1;
    view.tc_thr = nullptr;
    view.tc_gmax = nullptr;
    view.tc_tile_counter = nullptr;
    view.tc_two_phase = false;
    view.spill = nullptr;
    view.spill_cap = 0;
    view.pub = nullptr;
    view.scan_gmax = nullptr;
    view.norms = nullptr;  // no index, no stored norms: the scan derives them on the tensor cores
    view.x8 = nullptr;
    view.x8_bound = nullptr;
    view.x8_force = false;
    view.status = status;
    view.h_queries = nullptr;
    view.h_ids = nullptr;
    view.h_scores = nullptr;
    view.launches = 0;
    view.last_kernel = view.last_passes = view.last_phases = 0;
    view.last_sample_rows = 0;
    view.timing = false;
    return search_device(&view, static_cast<const __half *>(queries), s, k, ids, scores, st);
}

ralm_status_t ralm_index_set_tuning(ralm_index_t *idx, int32_t consumer_warps, int32_t ring_depth,
                                    int32_t tile_rows) {
    if (!idx || consumer_warps < 0 || consumer_warps > kMaxConsumerWarps || ring_depth < 0 ||
        ring_depth > kMaxStages || tile_rows < 0 || tile_rows > 64)
        return RALM_ERR_INVALID_ARG;
    idx->tune_warps = consumer_warps;
    idx->tune_depth = ring_depth;
    idx->tune_rows = tile_rows;
    return RALM_OK;
}

int64_t ralm_index_launch_count(const ralm_index_t *idx) { return idx ? idx->launches : 0; }

ralm_status_t ralm_index_set_timing(ralm_index_t *idx, int32_t enabled) {
    if (!idx) return RALM_ERR_INVALID_ARG;
    idx->timing = enabled != 0;
    return RALM_OK;
}

ralm_status_t ralm_index_read_timing(ralm_index_t *idx, double *total_ms, int64_t *launches) {
    if (!idx || !total_ms || !launches) return RALM_ERR_INVALID_ARG;
    double sum = 0.0;
    int64_t n = 0;
    ralm_status_t rs = RALM_OK;
    for (auto &ev : idx->timed) {
        float ms = 0.f;
        if (cudaEventSynchronize(ev.second) != cudaSuccess ||
            cudaEventElapsedTime(&ms, ev.first, ev.second) != cudaSuccess) {
            rs = RALM_ERR_CUDA;
        } else {
            sum += ms;
            ++n;
        }
        idx->spare.push_back(ev);
    }
    idx->timed.clear();
    *total_ms = sum;
    *launches = n;
    return rs;
}

ralm_status_t ralm_index_read_timing_list(ralm_index_t *idx, double *ms, int64_t capacity, int64_t *count) {
    if (!idx || !count || capacity < 0 || (capacity > 0 && !ms)) return RALM_ERR_INVALID_ARG;
    int64_t n = 0;
    ralm_status_t rs = RALM_OK;
    for (auto &ev : idx->timed) {
        float t = 0.f;
        if (cudaEventSynchronize(ev.second) != cudaSuccess || cudaEventElapsedTime(&t, ev.first, ev.second) != cudaSuccess)
            rs = RALM_ERR_CUDA;
        else if (n < capacity)
            ms[n++] = t;
        idx->spare.push_back(ev);
    }
    idx->timed.clear();
    *count = n;
    return rs;
}

ralm_status_t ralm_index_last_dispatch(const ralm_index_t *idx, int32_t *kernel, int32_t *passes, int32_t *phases,
                                       int64_t *sample_rows) {
    if (!idx || !kernel || !passes || !phases || !sample_rows) return RALM_ERR_INVALID_ARG;
    *kernel = idx->last_kernel;
    *passes = idx->last_passes;
    *phases = idx->last_phases;
    *sample_rows = idx->last_sample_rows;
    return RALM_OK;
}

const char *ralm_status_string(ralm_status_t status) {
    switch (status) {
        case RALM_OK: return "ok";
        case RALM_ERR_INVALID_ARG: return "invalid argument";
        case RALM_ERR_OOM: return "out of device memory";
        case RALM_ERR_CUDA: return "CUDA runtime error";
        case RALM_ERR_TIMEOUT: return "a device-side wait ran out";
        case RALM_ERR_UNSUPPORTED: return "unsupported device, shape or variant";
        case RALM_ERR_BAD_CACHE_ID: return "a cache id was outside [-1, N)";
        case RALM_ERR_INTERNAL: return "a candidate list overflowed (library defect; results not valid)";
        case RALM_ERR_STATIC_LIMIT:
            return "s or k exceeds what the built-in scratch of ralm_search_static can hold";
    }
    return "unknown status";
}

}  // extern "C"
