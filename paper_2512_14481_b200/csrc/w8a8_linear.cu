// Static W8A8 linear for sm_100a (Eq. 1 with the fixed learned factor, Eq. 2):
//   X_int = int8(clamp(rint(x * fl32(1/s_x)), -Qn, Qp))
//   acc   = X_int * W_int^T                      int8 x int8 -> int32 on tcgen05 tensor cores, accumulators in TMEM
//   y     = narrow(fl32(acc) * fl32(s_x * s_w[n]) (+ bias[n]))
//
// Persistent, warp-specialised kernels, one CTA per SM:
//   warp 0      TMA producer: W tiles and int8 A tiles -> 128-byte-swizzled shared memory
//   warp 1      MMA issuer: tcgen05.mma.kind::i8, 32 bytes of K per instruction, TMEM double-buffered
//   warps 2..5  epilogue: tcgen05.ld -> dequant -> 16-bit stores, overlapped with the next tile's mainloop
//   warps 6..13 (CTA-pair kernel) activation quantizer: Eq. 1 with the fixed factor on rows of x -> int8 A in the
//               workspace, published per 256-row block; the producers wait for the block they are about to load,
//               so the quantization of later rows runs under the MMAs of earlier ones and costs no launch
// Every wait on an mbarrier is bounded; a wait that gives up raises SASQ_ERR_TIMEOUT
// in the sticky status word and all roles fall through to the teardown.
//
// This file holds the host side (tensor maps, counters, launch planning, the C entry points); the kernels are in
//   linear_common.cuh     tile constants, LinearParams, bounded waits
//   gemm_pair.cuh         CTA-pair kernel, T > 128 (and groups of problems of any T)
//   gemm_small_t.cuh      small-T kernel, T <= 128
//   gemm_single.cuh       single-CTA kernel (fallback; also the 16-bit "FP weights" form)
//   gemm_grouped.cuh      grouped form of Eq. 3
//   quantize_kernels.cuh  activation quantizers as launches of their own
#include <algorithm>
#include <atomic>
#include <mutex>

#include "common.cuh"
#include "tcgen05.cuh"

namespace sasq {

SASQ_DEFINE_STATUS_WORD(g_linear_status)
void linear_reset_counters(cudaStream_t st);
int linear_status_read_and_clear(cudaStream_t st) {
    const int status = g_linear_status_read_and_clear(st);
    // a launch that gave up after a bounded wait may have left its readiness counters half counted: start clean
    if (status == SASQ_ERR_TIMEOUT) linear_reset_counters(st);
    return status;
}

}  // namespace sasq

#include "linear_common.cuh"
#include "gemm_single.cuh"
#include "gemm_grouped.cuh"
#include "gemm_pair.cuh"
#include "gemm_small_t.cuh"
#include "quantize_kernels.cuh"

namespace sasq {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// int8 [rows, K] row-major -> tiles of box_rows x 128 bytes, 128-byte swizzle, zero fill outside.
// Encoding a map costs a few microseconds on the host, which matters for decode-sized calls; weights are
// frozen and workspaces are reused, so the last few maps are kept (keyed by everything that defines them).
struct TmapKey {
    const void* base;
    long long rows, cols;
    int box_rows, box_cols, elem_bytes;
};
struct TmapEntry {
    TmapKey key;
    CUtensorMap map;
    bool valid;
};
constexpr int kTmapCache = 64;
std::mutex g_tmap_mutex;
TmapEntry g_tmap_cache[kTmapCache];
int g_tmap_next = 0;

// [rows, cols] row-major tensor of 1- or 2-byte elements, box of box_rows x box_cols whose inner extent is
// 32, 64 or 128 bytes and selects the matching swizzle
bool make_tmap_generic(CUtensorMap* m, const void* base, long long rows, long long cols, int box_rows, int box_cols,
                       int elem_bytes) {
    {
        std::lock_guard<std::mutex> lock(g_tmap_mutex);
        for (int i = 0; i < kTmapCache; ++i) {
            const TmapEntry& e = g_tmap_cache[i];
            if (e.valid && e.key.base == base && e.key.rows == rows && e.key.cols == cols &&
                e.key.box_rows == box_rows && e.key.box_cols == box_cols && e.key.elem_bytes == elem_bytes) {
                *m = e.map;
                return true;
            }
        }
    }
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const int inner = box_cols * elem_bytes;
    const CUtensorMapSwizzle sw = inner == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : inner == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                              : CU_TENSOR_MAP_SWIZZLE_32B;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)(cols * elem_bytes)};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    if (fn(m, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 2,
           const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    TmapEntry& e = g_tmap_cache[g_tmap_next];
    g_tmap_next = (g_tmap_next + 1) % kTmapCache;
    e.key = TmapKey{base, rows, cols, box_rows, box_cols, elem_bytes};
    e.map = *m;
    e.valid = true;
    return true;
}

// int8 operand [rows, K]: boxes of box_rows x 128 bytes
bool make_tmap(CUtensorMap* m, const void* base, long long rows, long long K, int box_rows) {
    return make_tmap_generic(m, base, rows, K, box_rows, BK, 1);
}
// 16-bit output [T, N]: boxes of 32 rows x box_cols columns (one epilogue warp's rows)
bool make_tmap_out(CUtensorMap* m, const void* base, long long T, long long N, int box_cols) {
    return make_tmap_generic(m, base, T, N, 32, box_cols, 2);
}

// Counters of the in-kernel activation quantizer.  They are zero when the library is loaded and every launch leaves
// the set it used at zero again.  Launches made directly draw the sets round-robin, so two of them share one only if
// more than kReadySlots launches of this kernel were running at the same time.  A launch that is being captured into
// a CUDA graph is different: its counters' address is frozen into the graph and used again by every replay, at
// times the library does not see.  Such a launch gets counters of its own from a second pool that is never handed
// out twice (a bump allocator; kCaptureCounters counters per process), so a replay can overlap launches made
// directly, or other graphs, on other streams without sharing a counter with them.
static __device__ unsigned g_a_ready[kReadySlots][kMaxRowBlocks];
static __device__ unsigned g_a_done[kReadySlots];
constexpr unsigned kCaptureCounters = 1u << 16;
static __device__ unsigned g_a_capture[kCaptureCounters];

}  // namespace

void linear_reset_counters(cudaStream_t st) {
    void *r = nullptr, *d = nullptr, *c = nullptr;
    if (cudaGetSymbolAddress(&r, g_a_ready) == cudaSuccess && cudaGetSymbolAddress(&d, g_a_done) == cudaSuccess &&
        cudaGetSymbolAddress(&c, g_a_capture) == cudaSuccess) {
        cudaMemsetAsync(r, 0, sizeof(unsigned) * kReadySlots * kMaxRowBlocks, st);
        cudaMemsetAsync(d, 0, sizeof(unsigned) * kReadySlots, st);
        cudaMemsetAsync(c, 0, sizeof(unsigned) * kCaptureCounters, st);
        cudaStreamSynchronize(st);
    }
}

namespace {

// `count` readiness counters and one completion counter for a launch on `st`.  SASQ_ERR_UNSUPPORTED when a captured
// launch finds the capture pool used up.
int next_ready_slot(cudaStream_t st, int count, unsigned** ready, unsigned** done) {
    static unsigned* ready_base[64] = {nullptr};
    static unsigned* done_base[64] = {nullptr};
    static unsigned* capture_base[64] = {nullptr};
    static std::atomic<unsigned> next{0};
    static std::atomic<unsigned> capture_next{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SASQ_ERR_CUDA;
    if (ready_base[dev] == nullptr) {
        unsigned *r = nullptr, *d = nullptr, *c = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&r), g_a_ready) != cudaSuccess) return SASQ_ERR_CUDA;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&d), g_a_done) != cudaSuccess) return SASQ_ERR_CUDA;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&c), g_a_capture) != cudaSuccess) return SASQ_ERR_CUDA;
        done_base[dev] = d;
        capture_base[dev] = c;
        ready_base[dev] = r;
    }
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &capturing) != cudaSuccess) return SASQ_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) {
        if (count < 0 || count > kMaxRowBlocks) return SASQ_ERR_UNSUPPORTED;
        const unsigned want = (unsigned)count + 1u;
        const unsigned at = capture_next.fetch_add(want, std::memory_order_relaxed);
        if (at > kCaptureCounters || at + want > kCaptureCounters) return SASQ_ERR_UNSUPPORTED;
        *ready = capture_base[dev] + at;
        *done = capture_base[dev] + at + count;
        return SASQ_OK;
    }
    const unsigned slot = next.fetch_add(1u, std::memory_order_relaxed) % kReadySlots;
    *ready = ready_base[dev] + (size_t)slot * kMaxRowBlocks;
    *done = done_base[dev] + slot;
    return SASQ_OK;
}

// Number of CTA pairs that can be resident at once (one pair per TPC); also opts the kernel in to its shared memory.
int pair_capacity(bool bf, int sm_count) {
    static int cache[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cache[dev][bf] != 0) return cache[dev][bf];
    const void* fn = bf ? reinterpret_cast<const void*>(w8a8_gemm_pair_kernel<true, false>)
                        : reinterpret_cast<const void*>(w8a8_gemm_pair_kernel<false, false>);
    const void* fn_small = bf ? reinterpret_cast<const void*>(w8a8_gemm_pair_kernel<true, true>)
                              : reinterpret_cast<const void*>(w8a8_gemm_pair_kernel<false, true>);
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(fn_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmemBytes) != cudaSuccess)
        return -1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)sm_count, 1, 1);
    cfg.blockDim = dim3(P_NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, fn, &cfg) != cudaSuccess || clusters <= 0) clusters = sm_count / 2;
    if (clusters > sm_count / 2) clusters = sm_count / 2;
    cache[dev][bf] = clusters;
    return clusters;
}

// Shared memory of a small-T launch with T rows: the smaller footprint (two CTAs per SM) up to D_LITE_MAX_TP rows.
int decode_ring_bytes(int64_t T) {
    const int64_t tp = (T + 15) / 16 * 16;
    return tp <= D_LITE_MAX_TP ? D_RING_BYTES_LITE : D_RING_BYTES;
}

// Largest K split (CTAs per cluster) of the small-T kernel with which all n_tiles clusters are resident at once (the
// in-kernel activation quantizer needs every CTA of the grid running) on at most one CTA per SM (with the smaller
// footprint the other half of each SM is left to the launch that follows); 0 if even one CTA per tile does not fit.
int decode_split(bool bf, int n_tiles, int k_blocks, int sm_count, int ring_bytes) {
    static int ready[64][2] = {};
    static int cap[64][2][2][4] = {};            // resident clusters for S = 1, 2, 4, 8; 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const void* fn = bf ? reinterpret_cast<const void*>(w8a8_decode_kernel<true>)
                        : reinterpret_cast<const void*>(w8a8_decode_kernel<false>);
    if (!ready[dev][bf]) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(D_RING_BYTES + sizeof(DecodeTail))) != cudaSuccess)
            return 0;
        ready[dev][bf] = 1;
    }
    const int lite = ring_bytes == D_RING_BYTES_LITE ? 1 : 0;
    for (int si = 3; si >= 0; --si) {
        const int S = 1 << si;
        if (S > k_blocks || (long long)n_tiles * S > sm_count) continue;
        if (cap[dev][bf][lite][si] == 0) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(sm_count / S * S), 1, 1);
            cfg.blockDim = dim3(D_THREADS, 1, 1);
            cfg.dynamicSmemBytes = (size_t)ring_bytes + sizeof(DecodeTail);
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)S;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, fn, &cfg) != cudaSuccess || clusters <= 0) clusters = -1;
            cap[dev][bf][lite][si] = clusters;
        }
        if (cap[dev][bf][lite][si] >= n_tiles) return S;
    }
    return 0;
}

// Column tiling of a 256-row block for `pairs` resident CTA pairs.  One MMA of N columns keeps the tensor pipe
// busy for about max(N, 208) / 2 cycles (below 208 columns the instruction is bound by reading its A operand), and a
// launch takes as long as its fullest pair: waves x that cost of the widest tile.  Tiles are at least 16 x 8 = 128
// columns wide unless N itself is narrower.  Fewer, wider tiles win ties (less fixed work per tile).
void plan_pair_tiles(PairParams* pp, int m_blocks, long long N, int pairs) {
    // the search below runs over up to N / 16 candidates; decode-sized calls are bound by the host, and a model has
    // a handful of distinct shapes: the last few plans are kept per thread
    struct Plan { int m_blocks, pairs; long long N; int n_tiles, base_units, rem_units, w_box_rows; };
    constexpr int kPlans = 16;
    thread_local Plan plans[kPlans] = {};
    thread_local int next_plan = 0;
    for (int i = 0; i < kPlans; ++i) {
        const Plan& c = plans[i];
        if (c.N == N && c.m_blocks == m_blocks && c.pairs == pairs && c.n_tiles != 0) {
            pp->pair_m_blocks = m_blocks;
            pp->n_tiles = c.n_tiles;
            pp->base_units = c.base_units;
            pp->rem_units = c.rem_units;
            pp->w_box_rows = c.w_box_rows;
            return;
        }
    }
    const int units = (int)((N + 15) / 16);
    int best_nt = (units + 15) / 16;
    double best_cost = -1.0;
    for (int nt = (units + 15) / 16; nt <= units; ++nt) {
        const int base = units / nt, rem = units % nt;
        const int max_w = 16 * (base + (rem ? 1 : 0));
        if (max_w > 256) continue;
        if (max_w < 128 && nt > (units + 15) / 16) break;
        const long long waves = ((long long)m_blocks * nt + pairs - 1) / pairs;
        const double cost = (double)waves * (max_w > 208 ? max_w : 208);
        if (best_cost < 0.0 || cost < 0.99 * best_cost) { best_cost = cost; best_nt = nt; }
    }
    pp->pair_m_blocks = m_blocks;
    pp->n_tiles = best_nt;
    pp->base_units = units / best_nt;
    pp->rem_units = units % best_nt;
    pp->w_box_rows = 8 * (pp->base_units + (pp->rem_units ? 1 : 0));
    plans[next_plan] = Plan{m_blocks, pairs, N, pp->n_tiles, pp->base_units, pp->rem_units, pp->w_box_rows};
    next_plan = (next_plan + 1) % kPlans;
}

int* status_word_ptr() {
    static int* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (cache[dev] == nullptr) {
        int* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_linear_status) != cudaSuccess) return nullptr;
        cache[dev] = p;
    }
    return cache[dev];
}

// opts the single-CTA kernel in to its shared memory once per device
bool single_kernel_ready(bool bf) {
    static bool done[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (done[dev][bf]) return true;
    const void* fn = bf ? reinterpret_cast<const void*>(w8a8_gemm_kernel<true, false>)
                        : reinterpret_cast<const void*>(w8a8_gemm_kernel<false, false>);
    const void* fn_fpw = bf ? reinterpret_cast<const void*>(w8a8_gemm_kernel<true, true>)
                            : reinterpret_cast<const void*>(w8a8_gemm_kernel<false, true>);
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(fn_fpw, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess)
        return false;
    done[dev][bf] = true;
    return true;
}

}  // namespace
}  // namespace sasq

extern "C" {

int sasq_set_gang_launch(int on) {
    return sasq::g_gang_launch.exchange(on ? 1 : 0, std::memory_order_relaxed);
}

long long sasq_debug_set_wait_limit(long long cycles) {
    const long long want = cycles < 0 ? sasq::kWaitLimit : cycles;
    return sasq::g_wait_limit.exchange(want, std::memory_order_relaxed);
}

int sasq_static_w8a8_linear_tiles(int64_t T, int64_t N, int num_pairs, int pair_id, int32_t* tiles_host, int cap) {
    using namespace sasq;
    if (T <= 0 || N <= 0 || T > (1 << 24) || N > (1 << 24) || num_pairs <= 0 || pair_id < 0 || pair_id >= num_pairs ||
        cap < 0 || (cap > 0 && tiles_host == nullptr))
        return -1;
    PairParams pp{};
    plan_pair_tiles(&pp, (int)((T + PBM - 1) / PBM), N, num_pairs);
    const int num_tiles = pp.pair_m_blocks * pp.n_tiles;
    int n = 0;
    for (int tile = pair_id; tile < num_tiles; tile += num_pairs, ++n) {
        if (n >= cap) continue;
        int n0, width;
        pair_tile_cols(pp, tile % pp.n_tiles, &n0, &width);
        tiles_host[3 * n + 0] = (tile / pp.n_tiles) * PBM;
        tiles_host[3 * n + 1] = n0;
        tiles_host[3 * n + 2] = width;
    }
    return n;
}

size_t sasq_static_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K) {
    (void)N;
    if (T <= 0 || K <= 0) return 0;
    // int8 copy of the activations, padded to whole 16-element groups
    return (size_t)(((T * K + 15) / 16) * 16 + 256);
}

}  // extern "C"

namespace sasq {
namespace {

// what every entry point of the linear checks before it launches anything
int check_linear_args(const void* x, const int8_t* w, const float* w_scale, const float* x_scale_dev,
                      const float* x_scales_vec, bool dynamic, const float* row_scale_out, const void* bias,
                      const void* y, const int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt, int bits) {
    if (T < 0 || N <= 0 || K <= 0) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (w == nullptr || w_scale == nullptr || (!dynamic && x_scale_dev == nullptr && x_scales_vec == nullptr))
        return SASQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_scales_vec) & 3u) return SASQ_ERR_INVALID_ARG;
    if (T > 0 && (x == nullptr || y == nullptr)) return SASQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(row_scale_out) & 3u) return SASQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(acc_out) ||
        (reinterpret_cast<uintptr_t>(w_scale) & 3u) || (reinterpret_cast<uintptr_t>(x_scale_dev) & 3u) ||
        (reinterpret_cast<uintptr_t>(bias) & 1u))
        return SASQ_ERR_INVALID_ARG;
    if (K % 16 != 0 || N % 8 != 0 || K > 131072 || T > (1 << 24) || N > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
    return SASQ_OK;
}

// When every problem of the launch has a single row block (nothing shared between tiles) and the lists fit the
// parameter block, deal the tiles out by cost: longest first, each to the pair with the least work so far.  The cost
// of a tile is its k-blocks (plus a few for the switch) times the MMA time of its width (one MMA of N columns keeps
// the tensor pipe busy for about max(N, 208) / 2 cycles).  Leaves gp->use_list = 0 otherwise.
void deal_tiles_by_cost(GroupParams* gp, int pairs) {
    gp->use_list = 0;
    const int np = gp->num_tiles < pairs ? gp->num_tiles : pairs;
    if (gp->count < 2 || gp->num_tiles > kMaxListTiles || np > kMaxListPairs) return;
    for (int q = 0; q < gp->count; ++q)
        if (gp->prob[q].pair_m_blocks != 1) return;
    struct Item { long long cost; int tile; };
    Item items[kMaxListTiles];
    int n = 0;
    for (int q = 0; q < gp->count; ++q) {
        const PairParams& pp = gp->prob[q];
        for (int j = 0; j < pp.n_tiles; ++j) {
            int n0, width;
            pair_tile_cols(pp, j, &n0, &width);
            items[n].cost = (long long)(pp.lp.k_blocks + 4) * (width > 208 ? width : 208);
            items[n].tile = pp.tile_begin + j;
            ++n;
        }
    }
    std::stable_sort(items, items + n, [](const Item& a, const Item& b) { return a.cost > b.cost; });
    // a binary min-heap of (load, pair): ties go to the lower pair index
    struct Slot { long long load; int pair; };
    Slot heap[kMaxListPairs];
    for (int pr = 0; pr < np; ++pr) heap[pr] = Slot{0, pr};            // sorted, hence a heap
    auto less = [](const Slot& a, const Slot& b) { return a.load < b.load || (a.load == b.load && a.pair < b.pair); };
    int owner[kMaxListTiles];
    int per_pair[kMaxListPairs] = {};
    for (int i = 0; i < n; ++i) {
        owner[i] = heap[0].pair;
        ++per_pair[heap[0].pair];
        heap[0].load += items[i].cost;
        int at = 0;                                                    // sift the grown root down
        for (;;) {
            int least = at;
            const int l = 2 * at + 1, r = l + 1;
            if (l < np && less(heap[l], heap[least])) least = l;
            if (r < np && less(heap[r], heap[least])) least = r;
            if (least == at) break;
            std::swap(heap[at], heap[least]);
            at = least;
        }
    }
    int at = 0;
    for (int pr = 0; pr < np; ++pr) {
        gp->list_begin[pr] = (uint16_t)at;
        at += per_pair[pr];
    }
    gp->list_begin[np] = (uint16_t)at;
    int fill[kMaxListPairs];
    for (int pr = 0; pr < np; ++pr) fill[pr] = gp->list_begin[pr];
    for (int i = 0; i < n; ++i) gp->tile_list[fill[owner[i]]++] = (uint16_t)items[i].tile;      // longest first
    gp->use_list = 1;
}

// One launch of the CTA-pair kernel over all problems of `gp`, on as many resident pairs as there are tiles.
int launch_pair_group(const GroupMaps& maps, const GroupParams& gp, int pairs, bool bf, cudaStream_t st,
                      bool small_layout = false) {
    const int grid = 2 * (gp.num_tiles < pairs ? gp.num_tiles : pairs);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(P_NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[3];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1] = pdl_attribute();
    attr[2].id = cudaLaunchAttributeCooperative;
    attr[2].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (gp.num_chunks != 0 && g_gang_launch.load(std::memory_order_relaxed)) ? 3 : 2;
    cudaError_t e;
    if (small_layout) {
        if (bf) e = cudaLaunchKernelEx(&cfg, w8a8_gemm_pair_kernel<true, true>, maps, gp);
        else e = cudaLaunchKernelEx(&cfg, w8a8_gemm_pair_kernel<false, true>, maps, gp);
    } else {
        if (bf) e = cudaLaunchKernelEx(&cfg, w8a8_gemm_pair_kernel<true, false>, maps, gp);
        else e = cudaLaunchKernelEx(&cfg, w8a8_gemm_pair_kernel<false, false>, maps, gp);
    }
    return e == cudaSuccess ? SASQ_OK : SASQ_ERR_CUDA;
}

// One launch of the small-T kernel over the problems of `dp` (all with T rows; prob[].lp, x, a_int8, tile_begin,
// n_tiles, quantize, qn, qp, row_scale_out and maps.w filled in by the caller): sets the shared geometry, draws the
// counters, encodes the activation maps and launches n_tiles clusters of `split` CTAs.
int launch_decode_group(DecodeMaps& maps, DecodeParams& dp, int T, int split, bool bf, cudaStream_t st) {
    dp.ring_bytes = decode_ring_bytes(T);
    const size_t smem_bytes = (size_t)dp.ring_bytes + sizeof(DecodeTail);
    dp.tp = (T + 15) / 16 * 16;
    const int stage_bytes = D_W_BYTES + dp.tp * BK;
    const int slot_bytes = (128 * (dp.tp + 4) * 4 + 1023) & ~1023;          // S x (128 / S) rows of tp + 4 words
    const int ring_bytes = dp.ring_bytes - slot_bytes;
    dp.slots_offset = ring_bytes;
    dp.stages = ring_bytes / stage_bytes < D_MAX_STAGES ? ring_bytes / stage_bytes : D_MAX_STAGES;
    dp.split = split;
    dp.tmem_cols = 32;
    while ((int)dp.tmem_cols < dp.tp) dp.tmem_cols <<= 1;
    // static factors and at most 16 rows: the CTAs quantize their own activation tiles in shared memory
    dp.local_x = dp.quantize && dp.row_scale_out == nullptr && dp.tp <= D_LITE_MAX_TP;
    if (dp.quantize && !dp.local_x) {
        const int rc = next_ready_slot(st, dp.count, &dp.ready, &dp.done);
        if (rc != SASQ_OK) return rc;
    }
    if (!dp.local_x)
        for (int q = 0; q < dp.count; ++q)
            if (!make_tmap(&maps.x[q], dp.prob[q].a_int8, T, dp.prob[q].lp.K, dp.tp)) return SASQ_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(dp.n_tiles * split), 1, 1);
    cfg.blockDim = dim3(D_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[3];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1] = pdl_attribute();
    attr[2].id = cudaLaunchAttributeCooperative;
    attr[2].val.cooperative = 1;
    cfg.attrs = attr;
    // with local activation tiles no CTA waits for another launch-mate outside its own cluster
    cfg.numAttrs = (dp.quantize && !dp.local_x && g_gang_launch.load(std::memory_order_relaxed)) ? 3 : 2;
    cudaError_t e;
    if (bf) e = cudaLaunchKernelEx(&cfg, w8a8_decode_kernel<true>, maps, dp);
    else e = cudaLaunchKernelEx(&cfg, w8a8_decode_kernel<false>, maps, dp);
    return e == cudaSuccess ? SASQ_OK : SASQ_ERR_CUDA;
}

// Cuts a list of problems into runs that fit one launch of the CTA-pair kernel (up to kMaxGroup problems,
// kMaxRowBlocks row blocks, kGroupCodeBytes of int8 codes) and tells `visit(first, last, grouped)` for each run
// whether it goes to that kernel in one launch: yes if all its problems have T > 128, or if it has small-T problems
// but at least two problems whose tiles fill every resident pair (the weights then stream through one launch
// instead of one latency chain per linear); otherwise its problems are launched one by one, in order.
template <typename Visit>
int for_each_run(int count, const sasq_linear_desc_t* descs, int pairs, Visit visit) {
    int first = 0;
    while (first < count) {
        int last = first, live = 0, blocks = 0, tiles = 0;
        long long codes = 0;
        bool small_t = false;
        while (last < count) {
            const sasq_linear_desc_t& d = descs[last];
            if (d.T > 0) {
                const long long m_blocks = (d.T + PBM - 1) / PBM;
                if (m_blocks > kMaxRowBlocks) break;                 // on its own, below
                if (live == kMaxGroup || blocks + m_blocks > kMaxRowBlocks ||
                    (live > 0 && codes + d.T * d.K > kGroupCodeBytes))
                    break;
                PairParams plan{};
                plan_pair_tiles(&plan, (int)m_blocks, d.N, pairs);
                tiles += plan.pair_m_blocks * plan.n_tiles;
                blocks += (int)m_blocks;
                codes += d.T * d.K;
                small_t = small_t || d.T <= BM;
                ++live;
            }
            ++last;
        }
        int rc;
        if (last == first) {                                          // a problem no launch can share
            rc = visit(first, first + 1, false);
            last = first + 1;
        } else {
            rc = visit(first, last, !small_t || (live >= 2 && tiles >= pairs));
        }
        if (rc != SASQ_OK) return rc;
        first = last;
    }
    return SASQ_OK;
}

// Within a run that does not go to the CTA-pair kernel: consecutive problems with the same T <= 128 whose
// 128-channel tiles all fit the device at once (one CTA each) share a launch of the small-T kernel, two to
// kMaxDecodeGroup of them; `visit(first, last, together)` is told for each segment.  Everything else goes alone.
template <typename Visit>
int for_each_small_segment(int first, int last, const sasq_linear_desc_t* descs, int sm_count, Visit visit) {
    int i = first;
    while (i < last) {
        const sasq_linear_desc_t& d = descs[i];
        if (d.T == 0) { ++i; continue; }
        int j = i + 1;
        if (d.T <= BM) {
            long long tiles = (d.N + 127) / 128;
            int live = 1;
            while (j < last && live < kMaxDecodeGroup) {
                const sasq_linear_desc_t& e = descs[j];
                if (e.T != 0) {
                    if (e.T != d.T || tiles + (e.N + 127) / 128 > sm_count) break;
                    tiles += (e.N + 127) / 128;
                    ++live;
                }
                ++j;
            }
            if (live >= 2 && tiles <= sm_count) {
                const int rc = visit(i, j, true);
                if (rc != SASQ_OK) return rc;
                i = j;
                continue;
            }
            j = i + 1;
        }
        const int rc = visit(i, j, false);
        if (rc != SASQ_OK) return rc;
        i = j;
    }
    return SASQ_OK;
}

// dynamic == false: static factor x_scale_dev (the hot path).  dynamic == true: every row gets its own max-based
// factor, written to row_scale_out (or to the workspace when that is NULL) by a launch that also quantizes the rows.
int linear_impl(const void* x, const int8_t* w, const float* w_scale, const float* x_scale_dev,
                const float* x_scales_vec, bool dynamic, float* row_scale_out, const void* bias, void* y, int32_t* acc_out, int64_t T, int64_t N, int64_t K,
                int dt, int bits, void* workspace, size_t ws_bytes, void* stream) {
    const int arg_rc = check_linear_args(x, w, w_scale, x_scale_dev, x_scales_vec, dynamic, row_scale_out, bias, y, acc_out,
                                         T, N, K, dt, bits);
    if (arg_rc != SASQ_OK) return arg_rc;
    if (T == 0) return SASQ_OK;
    const size_t ws_need = dynamic ? sasq_dynamic_w8a8_linear_workspace(T, N, K)
                           : x_scales_vec != nullptr ? sasq_static_w8a8_linear_per_channel_workspace(T, N, K)
                                                     : sasq_static_w8a8_linear_workspace(T, N, K);
    if (workspace == nullptr || !aligned16(workspace) || ws_bytes < ws_need) return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // 1. Eq. 1 with the fixed factor -> int8 activations in the workspace: inside the CTA-pair kernel when it is
    //    used and the row blocks fit its counters, otherwise by a launch of its own
    uint8_t* a_int8 = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(workspace) + 127) & ~uintptr_t(127));
    const float qn = (float)(1 << (bits - 1)), qp = (float)((1 << (bits - 1)) - 1);
    const int k_blocks = (int)((K + BK - 1) / BK);
    const int n_tiles128 = (int)((N + 127) / 128);
    const int split = (T <= BM && n_tiles128 <= sm_count)
                          ? decode_split(dt == SASQ_BF16, n_tiles128, k_blocks, sm_count, decode_ring_bytes(T)) : 0;
    const bool in_kernel_quantizer = !dynamic && (split > 0 || (T > BM && (T + PBM - 1) / PBM <= kMaxRowBlocks));
    const float* row_scale = nullptr;
    const float* chan_inv = nullptr;
    if (x_scales_vec != nullptr) {
        // one static factor per channel: their reciprocals go to the workspace (behind the codes) once per call
        float* inv = reinterpret_cast<float*>(reinterpret_cast<uintptr_t>(a_int8) + (uintptr_t)((T * K + 255) / 256 * 256));
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)((K + 255) / 256), 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1] = {pdl_attribute()};
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, reciprocal_factors_kernel, x_scales_vec, inv, (int)K, 1, status) != cudaSuccess)
            return SASQ_ERR_CUDA;
        chan_inv = inv;
    }
    // dynamic factors at small T: the small-T kernel computes them itself (a CTA's quantizer warps per row), so the
    // generation phase is one launch per linear
    const bool dynamic_inside = dynamic && split > 0;
    float* dyn_scales = nullptr;
    if (dynamic) {
        dyn_scales = row_scale_out;
        if (dyn_scales == nullptr) {
            const uintptr_t after = reinterpret_cast<uintptr_t>(a_int8) + (uintptr_t)((T * K + 255) / 256 * 256);
            dyn_scales = reinterpret_cast<float*>(after);
        }
        row_scale = dyn_scales;
    }
    if (dynamic && !dynamic_inside) {
        // per-token factors and codes by a launch of their own (the factor of a row needs the whole row first)
        float* rs = dyn_scales;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)T, 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1] = {pdl_attribute()};
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t qe;
        if (dt == SASQ_BF16)
            qe = cudaLaunchKernelEx(&cfg, quantize_rows_dynamic_kernel<true>, static_cast<const uint4*>(x),
                                    reinterpret_cast<uint2*>(a_int8), rs, (int)K, qn, qp);
        else
            qe = cudaLaunchKernelEx(&cfg, quantize_rows_dynamic_kernel<false>, static_cast<const uint4*>(x),
                                    reinterpret_cast<uint2*>(a_int8), rs, (int)K, qn, qp);
        if (qe != cudaSuccess) return SASQ_ERR_CUDA;
    } else if (!dynamic && !in_kernel_quantizer) {
        const long long n8 = (T * K) / 8;     // K % 16 == 0
        long long blocks = (n8 + 255) / 256;
        if (blocks > (long long)sm_count * 8) blocks = (long long)sm_count * 8;
        if (dt == SASQ_BF16)
            quantize_act_kernel<true><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                                   reinterpret_cast<uint2*>(a_int8), n8,
                                                                   x_scale_dev, chan_inv, (unsigned)(K / 8), qn, qp);
        else
            quantize_act_kernel<false><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                                    reinterpret_cast<uint2*>(a_int8), n8,
                                                                    x_scale_dev, chan_inv, (unsigned)(K / 8), qn, qp);
        if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    }

    // 2. TMA-fed tcgen05 GEMM with the dequant epilogue
    LinearParams p{};
    p.w_scale = w_scale;
    p.x_scale = x_scale_dev;
    p.row_scale = row_scale;
    p.chan_inv = chan_inv;
    p.bias = bias;
    p.y = y;
    p.acc_out = acc_out;
    p.T = (int)T; p.N = (int)N; p.K = (int)K;
    p.k_blocks = k_blocks;
    p.status = status;
    p.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    CUtensorMap tmap_a, tmap_w;
    if (split > 0) {
        // small T: 128-channel tiles, K split over a cluster, activations quantized inside the kernel
        DecodeParams dp{};
        DecodeMaps dmaps{};
        p.m_blocks = 1;
        p.n_blocks = n_tiles128;
        dp.count = 1;
        dp.prob[0].lp = p;
        dp.prob[0].a_int8 = a_int8;
        dp.prob[0].tile_begin = 0;
        dp.n_tiles = n_tiles128;
        dp.qn = qn;
        dp.qp = qp;
        if (in_kernel_quantizer || dynamic_inside) {
            dp.prob[0].x = static_cast<const uint16_t*>(x);
            dp.quantize = true;
            if (dynamic_inside) dp.row_scale_out = dyn_scales;
        }
        if (!make_tmap(&dmaps.w[0], w, N, K, 128)) return SASQ_ERR_CUDA;
        const int rc = launch_decode_group(dmaps, dp, (int)T, split, dt == SASQ_BF16, st);
        if (rc != SASQ_OK) return rc;
    } else if (T > BM) {
        // CTA pairs, 256-row blocks cut into evenly wide column tiles that fill whole waves of the resident pairs
        const int pairs = pair_capacity(dt == SASQ_BF16, sm_count);
        if (pairs <= 0) return SASQ_ERR_CUDA;
        GroupParams gp{};
        GroupMaps maps{};
        PairParams& pp = gp.prob[0];
        plan_pair_tiles(&pp, (int)((T + PBM - 1) / PBM), N, pairs);
        p.m_blocks = pp.pair_m_blocks;
        p.n_blocks = pp.n_tiles;
        pp.lp = p;
        pp.qn = qn;
        pp.qp = qp;
        gp.count = 1;
        gp.num_tiles = pp.pair_m_blocks * pp.n_tiles;
        if (in_kernel_quantizer) {
            pp.x = static_cast<const uint16_t*>(x);
            pp.a_int8 = a_int8;
            gp.ready_count = pp.pair_m_blocks;
            const int slot_rc = next_ready_slot(st, gp.ready_count, &gp.ready, &gp.done);
            if (slot_rc != SASQ_OK) return slot_rc;
            pp.ready = gp.ready;
            gp.num_chunks = (T * (K >> 3) + CONV_CHUNK - 1) / CONV_CHUNK;
        }
        if (!make_tmap(&maps.a[0], a_int8, T, K, 128) || !make_tmap(&maps.w[0], w, N, K, pp.w_box_rows) ||
            !make_tmap_out(&maps.y64[0], y, T, N, 64) || !make_tmap_out(&maps.y16[0], y, T, N, 16))
            return SASQ_ERR_CUDA;
        const int rc = launch_pair_group(maps, gp, pairs, dt == SASQ_BF16, st);
        if (rc != SASQ_OK) return rc;
    } else {
        p.m_blocks = (int)((T + BM - 1) / BM);
        p.n_blocks = (int)((N + BN - 1) / BN);
        if (!make_tmap(&tmap_a, a_int8, T, K, BM) || !make_tmap(&tmap_w, w, N, K, BN)) return SASQ_ERR_CUDA;
        const long long tiles = (long long)p.m_blocks * p.n_blocks;
        const int grid = (int)(tiles < sm_count ? tiles : sm_count);
        if (!single_kernel_ready(dt == SASQ_BF16)) return SASQ_ERR_CUDA;
        if (dt == SASQ_BF16) w8a8_gemm_kernel<true, false><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
        else w8a8_gemm_kernel<false, false><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
    }
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

}  // namespace
}  // namespace sasq

extern "C" {

int sasq_static_w8a8_linear(const void* x, const int8_t* w, const float* w_scale, const float* x_scale_dev,
                            const void* bias, void* y, int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt,
                            int bits, void* workspace, size_t ws_bytes, void* stream) {
    return sasq::linear_impl(x, w, w_scale, x_scale_dev, nullptr, false, nullptr, bias, y, acc_out, T, N, K, dt, bits,
                             workspace, ws_bytes, stream);
}

size_t sasq_static_w8a8_linear_multi_workspace(int count, const sasq_linear_desc_t* descs_host) {
    if (count <= 0 || descs_host == nullptr) return 0;
    size_t total = 0;
    for (int i = 0; i < count; ++i) {
        const size_t one = sasq_static_w8a8_linear_workspace(descs_host[i].T, descs_host[i].N, descs_host[i].K);
        total += (one + 255) / 256 * 256;
    }
    return total + 256;
}

int sasq_static_w8a8_linear_multi(int count, const sasq_linear_desc_t* descs_host, int dt, int bits, void* workspace,
                                  size_t ws_bytes, void* stream) {
    using namespace sasq;
    if (count < 0 || (count > 0 && descs_host == nullptr)) return SASQ_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        const sasq_linear_desc_t& d = descs_host[i];
        const int rc = check_linear_args(d.x, d.w, d.w_scale, d.x_scale, nullptr, false, nullptr, d.bias, d.y, nullptr,
                                         d.T, d.N, d.K, dt, bits);
        if (rc != SASQ_OK) return rc;
    }
    if (count == 0) return SASQ_OK;
    if (workspace == nullptr || !aligned16(workspace) ||
        ws_bytes < sasq_static_w8a8_linear_multi_workspace(count, descs_host))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf = dt == SASQ_BF16;
    const int pairs = pair_capacity(bf, sm_count);
    if (pairs <= 0) return SASQ_ERR_CUDA;
    const float qn = (float)(1 << (bits - 1)), qp = (float)((1 << (bits - 1)) - 1);
    const long long wait_limit = g_wait_limit.load(std::memory_order_relaxed);

    // workspace slice of problem i: the slices follow one another, each a multiple of 256 bytes
    const uintptr_t ws0 = (reinterpret_cast<uintptr_t>(workspace) + 255) & ~uintptr_t(255);
    auto slice_bytes = [&](int i) -> size_t {
        const sasq_linear_desc_t& d = descs_host[i];
        return (sasq_static_w8a8_linear_workspace(d.T, d.N, d.K) + 255) / 256 * 256;
    };
    auto slice = [&](int i) -> void* {
        uintptr_t at = ws0;
        for (int j = 0; j < i; ++j) at += slice_bytes(j);
        return reinterpret_cast<void*>(at);
    };

    auto run_alone = [&](int i) -> int {
        const sasq_linear_desc_t& d = descs_host[i];
        return linear_impl(d.x, d.w, d.w_scale, d.x_scale, nullptr, false, nullptr, d.bias, d.y, nullptr, d.T, d.N, d.K,
                           dt, bits, slice(i), slice_bytes(i), stream);
    };
    // one launch of the CTA-pair kernel for problems [first, last)
    auto run_group = [&](int first, int last) -> int {
        GroupParams gp{};
        GroupMaps maps{};
        bool small_layout = true;               // every problem has at most 32 rows: the 8-stage layout
        for (int i = first; i < last; ++i) small_layout = small_layout && descs_host[i].T <= P_SMALL_ROWS;
        for (int i = first; i < last; ++i) {
            if (descs_host[i].T == 0) continue;
            const sasq_linear_desc_t& d = descs_host[i];
            const int q = gp.count;
            PairParams& pp = gp.prob[q];
            plan_pair_tiles(&pp, (int)((d.T + PBM - 1) / PBM), d.N, pairs);
            LinearParams& p = pp.lp;
            p.w_scale = d.w_scale;
            p.x_scale = d.x_scale;
            p.bias = d.bias;
            p.y = d.y;
            p.T = (int)d.T; p.N = (int)d.N; p.K = (int)d.K;
            p.k_blocks = (int)((d.K + BK - 1) / BK);
            p.m_blocks = pp.pair_m_blocks;
            p.n_blocks = pp.n_tiles;
            p.status = status;
            p.wait_limit = wait_limit;
            pp.qn = qn;
            pp.qp = qp;
            pp.x = static_cast<const uint16_t*>(d.x);
            pp.a_int8 = reinterpret_cast<uint8_t*>(slice(i));
            pp.tile_begin = gp.num_tiles;
            pp.chunk_begin = gp.num_chunks;
            if (!make_tmap(&maps.a[q], pp.a_int8, d.T, d.K, small_layout ? P_SMALL_ROWS : 128) ||
                !make_tmap(&maps.w[q], d.w, d.N, d.K, pp.w_box_rows) ||
                !make_tmap_out(&maps.y64[q], d.y, d.T, d.N, 64) || !make_tmap_out(&maps.y16[q], d.y, d.T, d.N, 16))
                return SASQ_ERR_CUDA;
            gp.num_tiles += pp.pair_m_blocks * pp.n_tiles;
            gp.num_chunks += (d.T * (d.K >> 3) + CONV_CHUNK - 1) / CONV_CHUNK;
            gp.count = q + 1;
        }
        if (gp.count == 0) return SASQ_OK;
        int off = 0;
        for (int q = 0; q < gp.count; ++q) off += gp.prob[q].pair_m_blocks;
        gp.ready_count = off;
        const int slot_rc = next_ready_slot(st, gp.ready_count, &gp.ready, &gp.done);
        if (slot_rc != SASQ_OK) return slot_rc;
        off = 0;
        for (int q = 0; q < gp.count; ++q) {
            gp.prob[q].ready = gp.ready + off;
            off += gp.prob[q].pair_m_blocks;
        }
        deal_tiles_by_cost(&gp, pairs);
        return launch_pair_group(maps, gp, pairs, bf, st, small_layout);
    };

    // one launch of the small-T kernel for problems [first, last), all with the same T <= 128
    auto run_small_group = [&](int first, int last) -> int {
        DecodeParams dp{};
        DecodeMaps dmaps{};
        int T = 0, min_kblocks = 1 << 30;
        for (int i = first; i < last; ++i) {
            const sasq_linear_desc_t& d = descs_host[i];
            if (d.T == 0) continue;
            const int q = dp.count;
            DecodeProblem& pr = dp.prob[q];
            LinearParams& p = pr.lp;
            p.w_scale = d.w_scale;
            p.x_scale = d.x_scale;
            p.bias = d.bias;
            p.y = d.y;
            p.T = (int)d.T; p.N = (int)d.N; p.K = (int)d.K;
            p.k_blocks = (int)((d.K + BK - 1) / BK);
            p.m_blocks = 1;
            p.n_blocks = (int)((d.N + 127) / 128);
            p.status = status;
            p.wait_limit = wait_limit;
            pr.x = static_cast<const uint16_t*>(d.x);
            pr.a_int8 = reinterpret_cast<uint8_t*>(slice(i));
            pr.tile_begin = dp.n_tiles;
            if (!make_tmap(&dmaps.w[q], d.w, d.N, d.K, 128)) return SASQ_ERR_CUDA;
            dp.n_tiles += p.n_blocks;
            if (p.k_blocks < min_kblocks) min_kblocks = p.k_blocks;
            T = (int)d.T;
            dp.count = q + 1;
        }
        dp.quantize = true;
        dp.qn = qn;
        dp.qp = qp;
        const int split = decode_split(bf, dp.n_tiles, min_kblocks, sm_count, decode_ring_bytes(T));
        if (split <= 0) {                        // cannot all be resident after all: one by one
            int rc = SASQ_OK;
            for (int i = first; i < last && rc == SASQ_OK; ++i)
                if (descs_host[i].T > 0) rc = run_alone(i);
            return rc;
        }
        return launch_decode_group(dmaps, dp, T, split, bf, st);
    };

    return for_each_run(count, descs_host, pairs, [&](int first, int last, bool grouped) -> int {
        if (grouped) return run_group(first, last);
        return for_each_small_segment(first, last, descs_host, sm_count, [&](int a, int b, bool together) -> int {
            if (together) return run_small_group(a, b);
            int rc = SASQ_OK;
            for (int i = a; i < b && rc == SASQ_OK; ++i)
                if (descs_host[i].T > 0) rc = run_alone(i);
            return rc;
        });
    });
}

int sasq_static_w8a8_linear_multi_launches(int count, const sasq_linear_desc_t* descs_host, int num_pairs) {
    using namespace sasq;
    if (count < 0 || (count > 0 && descs_host == nullptr) || num_pairs <= 0) return -1;
    for (int i = 0; i < count; ++i)
        if (descs_host[i].T < 0 || descs_host[i].N <= 0 || descs_host[i].K <= 0) return -1;
    int launches = 0;
    for_each_run(count, descs_host, num_pairs, [&](int first, int last, bool grouped) -> int {
        if (grouped) {
            for (int i = first; i < last; ++i)
                if (descs_host[i].T > 0) { ++launches; break; }
            return SASQ_OK;
        }
        return for_each_small_segment(first, last, descs_host, 2 * num_pairs, [&](int a, int b, bool together) -> int {
            if (together) {
                ++launches;
                return SASQ_OK;
            }
            for (int i = a; i < b; ++i) {
                const sasq_linear_desc_t& d = descs_host[i];
                if (d.T == 0) continue;
                // the activation quantizer runs inside the GEMM launch unless the row blocks (T > 128) or the
                // 128-channel tiles (T <= 128) outnumber what its counters / the resident CTAs can hold
                const bool inside =
                    d.T > BM ? (d.T + PBM - 1) / PBM <= kMaxRowBlocks : (d.N + 127) / 128 <= 2 * num_pairs;
                launches += inside ? 1 : 2;
            }
            return SASQ_OK;
        });
    });
    return launches;
}

size_t sasq_fakequant_linear_fp_weights_workspace(int64_t T, int64_t N, int64_t K) {
    (void)N;
    if (T <= 0 || K <= 0) return 0;
    return (size_t)(T * K) * 2 + 256;           // the fake-quantized activations X', 16-bit
}

int sasq_fakequant_linear_fp_weights(const void* x, const void* w, const float* x_scale_dev, const void* bias, void* y,
                                     int64_t T, int64_t N, int64_t K, int dt, int bits, void* workspace,
                                     size_t ws_bytes, void* stream) {
    using namespace sasq;
    if (T < 0 || N <= 0 || K <= 0) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (w == nullptr || x_scale_dev == nullptr || (T > 0 && (x == nullptr || y == nullptr))) return SASQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || (reinterpret_cast<uintptr_t>(x_scale_dev) & 3u) ||
        (reinterpret_cast<uintptr_t>(bias) & 1u))
        return SASQ_ERR_INVALID_ARG;
    if (K % 8 != 0 || N % 8 != 0 || T > (1 << 24) || N > (1 << 24) || K > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
    if (T == 0) return SASQ_OK;
    if (workspace == nullptr || !aligned16(workspace) || ws_bytes < sasq_fakequant_linear_fp_weights_workspace(T, N, K))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf = dt == SASQ_BF16;
    if (!single_kernel_ready(bf)) return SASQ_ERR_CUDA;

    // 1. X' = g(X): the fake-quant forward (Eq. 1, Sec. 4.2) into the workspace; 2. Y = X' W^T on the tensor cores
    void* xq = reinterpret_cast<void*>((reinterpret_cast<uintptr_t>(workspace) + 127) & ~uintptr_t(127));
    const int rc = sasq_fakequant_fwd(x, xq, T * K, dt, x_scale_dev, bits, stream);
    if (rc != SASQ_OK) return rc;
    LinearParams p{};
    p.bias = bias;
    p.y = y;
    p.T = (int)T; p.N = (int)N; p.K = (int)K;
    p.k_blocks = (int)((K * 2 + BK - 1) / BK);
    p.m_blocks = (int)((T + BM - 1) / BM);
    p.n_blocks = (int)((N + BN - 1) / BN);
    p.status = status;
    p.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    CUtensorMap tmap_a, tmap_w;
    if (!make_tmap_generic(&tmap_a, xq, T, K, BM, BK / 2, 2) || !make_tmap_generic(&tmap_w, w, N, K, BN, BK / 2, 2))
        return SASQ_ERR_CUDA;
    const long long tiles = (long long)p.m_blocks * p.n_blocks;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    if (bf) w8a8_gemm_kernel<true, true><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
    else w8a8_gemm_kernel<false, true><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

size_t sasq_static_w8a8_linear_grouped_workspace(int64_t T, int64_t N, int64_t K) {
    (void)N;
    if (T <= 0 || K <= 0) return 0;
    // int8 codes, then one fp32 reciprocal per channel (the group's, repeated)
    return sasq_static_w8a8_linear_workspace(T, N, K) + 256 + (size_t)K * sizeof(float) + 256;
}

int sasq_static_w8a8_linear_grouped(const void* x, const int8_t* w, const float* w_scale, const float* s_group_dev,
                                    int64_t group, const void* bias, void* y, int64_t T, int64_t N, int64_t K, int dt,
                                    int bits, void* workspace, size_t ws_bytes, void* stream) {
    using namespace sasq;
    if (s_group_dev == nullptr || group <= 0) return SASQ_ERR_INVALID_ARG;
    const int rc = check_linear_args(x, w, w_scale, nullptr, s_group_dev, false, nullptr, bias, y, nullptr, T, N, K, dt,
                                     bits);
    if (rc != SASQ_OK) return rc;
    if (group % BK != 0 || K % group != 0) return SASQ_ERR_UNSUPPORTED;      // groups are whole 128-column k-blocks
    if (T == 0) return SASQ_OK;
    if (workspace == nullptr || !aligned16(workspace) || ws_bytes < sasq_static_w8a8_linear_grouped_workspace(T, N, K))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf = dt == SASQ_BF16;
    {
        static bool ready[64][2] = {};
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SASQ_ERR_CUDA;
        if (!ready[dev][bf]) {
            const void* fn = bf ? reinterpret_cast<const void*>(w8a8_grouped_kernel<true>)
                                : reinterpret_cast<const void*>(w8a8_grouped_kernel<false>);
            if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGroupedSmemBytes) !=
                cudaSuccess)
                return SASQ_ERR_CUDA;
            ready[dev][bf] = true;
        }
    }
    uint8_t* a_int8 = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(workspace) + 127) & ~uintptr_t(127));
    float* inv = reinterpret_cast<float*>(reinterpret_cast<uintptr_t>(a_int8) + (uintptr_t)((T * K + 255) / 256 * 256));
    const float qn = (float)(1 << (bits - 1)), qp = (float)((1 << (bits - 1)) - 1);

    // 1. fl32(1 / s_g) for every channel of its group, 2. Eq. 1 with those -> int8 codes, 3. the grouped GEMM
    reciprocal_factors_kernel<<<(unsigned)((K + 255) / 256), 256, 0, st>>>(s_group_dev, inv, (int)K, (int)group, status);
    const long long n8 = (T * K) / 8;
    long long blocks = (n8 + 255) / 256;
    if (blocks > (long long)sm_count * 8) blocks = (long long)sm_count * 8;
    if (bf)
        quantize_act_kernel<true><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                               reinterpret_cast<uint2*>(a_int8), n8, nullptr, inv,
                                                               (unsigned)(K / 8), qn, qp);
    else
        quantize_act_kernel<false><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                                reinterpret_cast<uint2*>(a_int8), n8, nullptr, inv,
                                                                (unsigned)(K / 8), qn, qp);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;

    GroupedParams gp{};
    LinearParams& p = gp.lp;
    p.w_scale = w_scale;
    p.bias = bias;
    p.y = y;
    p.T = (int)T; p.N = (int)N; p.K = (int)K;
    p.k_blocks = (int)(K / BK);
    p.m_blocks = (int)((T + BM - 1) / BM);
    p.n_blocks = (int)((N + GBN - 1) / GBN);
    p.status = status;
    p.wait_limit = g_wait_limit.load(std::memory_order_relaxed);
    gp.s_group = s_group_dev;
    gp.group_kblocks = (int)(group / BK);
    gp.groups = (int)(K / group);
    CUtensorMap tmap_a, tmap_w;
    if (!make_tmap(&tmap_a, a_int8, T, K, BM) || !make_tmap(&tmap_w, w, N, K, GBN)) return SASQ_ERR_CUDA;
    const long long tiles = (long long)p.m_blocks * p.n_blocks;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    if (bf) w8a8_grouped_kernel<true><<<grid, G_THREADS, kGroupedSmemBytes, st>>>(tmap_a, tmap_w, gp);
    else w8a8_grouped_kernel<false><<<grid, G_THREADS, kGroupedSmemBytes, st>>>(tmap_a, tmap_w, gp);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

size_t sasq_static_w8a8_linear_per_channel_workspace(int64_t T, int64_t N, int64_t K) {
    if (T <= 0 || K <= 0) return 0;
    // int8 codes, then one fp32 reciprocal per channel
    return sasq_static_w8a8_linear_workspace(T, N, K) + 256 + (size_t)K * sizeof(float) + 256;
}

int sasq_static_w8a8_linear_per_channel(const void* x, const int8_t* w, const float* w_scale,
                                        const float* x_scales_dev, const void* bias, void* y, int32_t* acc_out,
                                        int64_t T, int64_t N, int64_t K, int dt, int bits, void* workspace,
                                        size_t ws_bytes, void* stream) {
    if (x_scales_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    return sasq::linear_impl(x, w, w_scale, nullptr, x_scales_dev, false, nullptr, bias, y, acc_out, T, N, K, dt, bits,
                             workspace, ws_bytes, stream);
}

size_t sasq_dynamic_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K) {
    if (T <= 0 || K <= 0) return 0;
    // int8 codes, then one fp32 factor per row
    return sasq_static_w8a8_linear_workspace(T, N, K) + 256 + (size_t)T * sizeof(float) + 256;
}

int sasq_dynamic_w8a8_linear(const void* x, const int8_t* w, const float* w_scale, const void* bias, void* y,
                             float* row_scale_out, int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt, int bits,
                             void* workspace, size_t ws_bytes, void* stream) {
    return sasq::linear_impl(x, w, w_scale, nullptr, nullptr, true, row_scale_out, bias, y, acc_out, T, N, K, dt, bits,
                             workspace, ws_bytes, stream);
}

}  // extern "C"
