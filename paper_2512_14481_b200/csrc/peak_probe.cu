// Measurement aid: the rate at which the tensor cores of this device retire the instruction the W8A8 GEMM is built
// from (tcgen05.mma.cta_group::2.kind::i8, 256 x N x 32, both operands in shared memory) when nothing else is in the
// way: no loads, no epilogue, one CTA pair per TPC issuing back to back.  It is the ceiling the GEMM's roofline
// fraction can be quoted against on the same box, under the same power cap.  No arithmetic of the method is here; the
// operands are pseudo-random bytes (zeros would toggle no wires and draw less power than real codes do).
#include <atomic>

#include "common.cuh"
#include "tcgen05.cuh"

namespace sasq {
namespace {

constexpr int PR_THREADS = 128;
constexpr int PR_TILE_BYTES = 128 * 128;        // 128 rows x 128 bytes of K, 128-byte swizzle (random bytes: layout is moot)
constexpr int PR_BATCH = 32;                    // MMAs between two commits
constexpr int kProbeMaxPairs = 128;

struct ProbeTail {
    uint64_t done[2];
    uint32_t tmem_base;
};

static __device__ unsigned long long g_probe_cycles[kProbeMaxPairs];
static __device__ int g_probe_status;

__global__ void __launch_bounds__(PR_THREADS, 1)
int8_issue_probe_kernel(int batches, int n_cols, long long wait_limit) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* a_tile = smem_raw;                          // this CTA's 128 rows of A
    uint8_t* b_tile = smem_raw + PR_TILE_BYTES;          // this CTA's half (n_cols / 2 <= 128 rows) of B
    ProbeTail* tail = reinterpret_cast<ProbeTail*>(smem_raw + 2 * PR_TILE_BYTES);
    if ((ptx::smem_u32(smem_raw) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicMax(&g_probe_status, (int)SASQ_ERR_CUDA);
        return;
    }
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = ptx::cluster_ctarank();
    for (int i = threadIdx.x; i < 2 * PR_TILE_BYTES / 4; i += PR_THREADS) {
        uint32_t h = (uint32_t)i * 2654435761u + (uint32_t)blockIdx.x * 40503u + 12345u;      // a multiplicative hash
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        reinterpret_cast<uint32_t*>(smem_raw)[i] = h;
    }
    ptx::fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        ptx::mbar_init(&tail->done[0], 1);
        ptx::mbar_init(&tail->done[1], 1);
        ptx::mbar_init_fence();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&tail->tmem_base, 512);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;

    if (warp == 1 && rank == 0 && ptx::elect_one()) {
        const uint64_t a_desc = ptx::smem_desc_k_major_sw128(ptx::smem_u32(a_tile));
        const uint64_t b_desc = ptx::smem_desc_k_major_sw128(ptx::smem_u32(b_tile));
        const uint32_t idesc = ptx::idesc_i8(256, n_cols);
        bool ok = true;
        const long long t0 = clock64();
        for (int b = 0; b < batches && ok; ++b) {
            if (b >= 2) {
                // at most two batches in the queue: wait for the commit of batch b - 2 (bounded)
                const uint32_t parity = (uint32_t)(((b >> 1) - 1) & 1);
                const long long w0 = clock64();
                while (!ptx::mbar_try_wait(&tail->done[b & 1], parity)) {
                    if (clock64() - w0 > wait_limit) { ok = false; break; }
                }
                if (!ok) break;
            }
            const uint32_t d_tmem = tmem_base + (uint32_t)((b & 1) * 256);
#pragma unroll 1
            for (int i = 0; i < PR_BATCH / 4; ++i) {
                ptx::mma_i8_ss_pair(d_tmem, a_desc, b_desc, idesc, i == 0 ? 0u : 1u);
                ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 2, b_desc + 2, idesc);
                ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 4, b_desc + 4, idesc);
                ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 6, b_desc + 6, idesc);
            }
            ptx::mma_commit_pair(&tail->done[b & 1], 0x1);
        }
        // drain: the last commit on each barrier (bounded); after a give-up the MMAs still retire within microseconds
        for (int k = 0; k < 2 && ok; ++k) {
            const int last = batches - 1 - ((batches - 1 - k) & 1);      // last batch index with parity k
            if (last < 0) continue;
            const uint32_t parity = (uint32_t)((last >> 1) & 1);
            const long long w0 = clock64();
            while (!ptx::mbar_try_wait(&tail->done[k], parity)) {
                if (clock64() - w0 > wait_limit) { ok = false; break; }
            }
        }
        const long long t1 = clock64();
        if (!ok) {
            atomicMax(&g_probe_status, (int)SASQ_ERR_TIMEOUT);
            const long long w0 = clock64();
            while (clock64() - w0 < (1LL << 22)) __nanosleep(1000);
        }
        const unsigned pair = blockIdx.x >> 1;
        if (pair < (unsigned)kProbeMaxPairs) g_probe_cycles[pair] = (unsigned long long)(t1 - t0);
    }
    __syncwarp();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, 512);
    }
}

}  // namespace
}  // namespace sasq

extern "C" {

int sasq_debug_int8_issue_rate(int mma_per_pair, int n_cols, double* ops_per_second_host, double* mac_per_clk_sm_host,
                               void* stream) {
    using namespace sasq;
    if (mma_per_pair < PR_BATCH || n_cols < 32 || n_cols > 256 || n_cols % 32 != 0 ||
        ops_per_second_host == nullptr || mac_per_clk_sm_host == nullptr)
        return SASQ_ERR_INVALID_ARG;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = 2 * PR_TILE_BYTES + sizeof(ProbeTail);
    if (cudaFuncSetAttribute(int8_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return SASQ_ERR_CUDA;
    int pairs = sm_count / 2;
    if (pairs > kProbeMaxPairs) pairs = kProbeMaxPairs;
    const int batches = mma_per_pair / PR_BATCH;
    const int zero = 0;
    if (cudaMemcpyToSymbolAsync(g_probe_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return SASQ_ERR_CUDA;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SASQ_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(PR_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int rc = SASQ_OK;
    cudaEventRecord(e0, st);
    if (cudaLaunchKernelEx(&cfg, int8_issue_probe_kernel, batches, n_cols, (long long)1 << 31) != cudaSuccess)
        rc = SASQ_ERR_CUDA;
    cudaEventRecord(e1, st);
    if (cudaStreamSynchronize(st) != cudaSuccess) rc = SASQ_ERR_CUDA;
    float ms = 0.0f;
    if (rc == SASQ_OK && cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = SASQ_ERR_CUDA;
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != SASQ_OK) return rc;
    int status = 0;
    unsigned long long cycles[kProbeMaxPairs];
    if (cudaMemcpyFromSymbol(&status, g_probe_status, sizeof(int)) != cudaSuccess ||
        cudaMemcpyFromSymbol(cycles, g_probe_cycles, sizeof(unsigned long long) * pairs) != cudaSuccess)
        return SASQ_ERR_CUDA;
    if (status != 0) return status;
    unsigned long long worst = 1;
    for (int i = 0; i < pairs; ++i) worst = cycles[i] > worst ? cycles[i] : worst;
    const double mma = (double)batches * PR_BATCH;
    const double mac_per_mma = 256.0 * n_cols * 32.0;
    *ops_per_second_host = 2.0 * mac_per_mma * mma * pairs / ((double)ms * 1e-3);
    *mac_per_clk_sm_host = mac_per_mma * mma / (double)worst / 2.0;
    return SASQ_OK;
}

}  // extern "C"
