// Shared by the kernels of the W8A8 linear: tile constants, the launch parameters of one linear, bounded
// waits, the epilogue's factor rule.
#pragma once
#include <atomic>

#include "common.cuh"
#include "tcgen05.cuh"

namespace sasq {
namespace {

constexpr int BM = 128;            // rows of x per tile (UMMA M)
constexpr int BN = 256;            // output channels per tile (UMMA N)
constexpr int BK = 128;            // int8 elements (= bytes) of K per pipeline stage: one 128-byte swizzle row
constexpr int UMMA_K = 32;         // K per tcgen05.mma.kind::i8
static_assert(BK / UMMA_K == 4, "the issue loops are written for four MMAs per stage");
constexpr int STAGES = 4;
constexpr int ACC_BUFS = 2;        // TMEM accumulator buffers (2 x 256 columns = all 512)
constexpr int A_STAGE_BYTES = BM * BK;
constexpr int B_STAGE_BYTES = BN * BK;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int NUM_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr uint32_t TMEM_COLS = 512;
constexpr long long kWaitLimit = 1LL << 31;   // clock cycles a single wait may take (about a second)
std::atomic<long long> g_wait_limit{kWaitLimit};   // what launches use; tests shorten it to see the give-up path
// launch the kernels whose CTAs wait on one another as co-operative grids (the safe default: such a launch starts only
// when all of its CTAs can be resident; a caller that keeps every linear on one stream may switch it off)
std::atomic<int> g_gang_launch{1};

struct SharedTail {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[ACC_BUFS];
    uint64_t tmem_empty[ACC_BUFS];
    float scale[BN];               // s_x * s_w[n] of the tile being stored
    float bias[BN];
    uint32_t tmem_base;
    volatile int abort_flag;
};

constexpr size_t kSmemBytes = 1024 /* alignment slack */ + (size_t)STAGES * STAGE_BYTES + sizeof(SharedTail);

struct LinearParams {
    const float* w_scale;
    const float* x_scale;      // one static factor for the whole tensor, or
    const float* row_scale;    // [T] one factor per row (dynamic per-token quantization); then x_scale is unused
    const float* chan_inv;     // [K] fl32(1 / s_x[k]) for one static factor per channel; the output factor is then
                               // w_scale[n] alone (the caller folded s_x[k] into the weights); x_scale is unused
    const void* bias;
    void* y;
    int32_t* acc_out;
    int T, N, K;
    int m_blocks, n_blocks, k_blocks;
    int* status;
    long long wait_limit;
};

// factor of output (t, n): the staged per-channel value already holds s_x * s_w[n] for a static factor; with
// per-row factors it holds s_w[n] and the row's factor is multiplied in here, fl32(s_row * s_w[n])
__device__ __forceinline__ float out_scale(bool per_row, float s_row, float staged) {
    return per_row ? __fmul_rn(s_row, staged) : staged;
}

// Bounded wait: false (and the abort flag raised) if the phase did not complete in time
// or another role already gave up.
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, SharedTail* tail, const LinearParams& p) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int polls = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (p.wait_limit <= 0 || (++polls & 63) == 0) {      // a zero limit gives up at the first unsuccessful poll
            if (tail->abort_flag) return false;
            if (clock64() - t0 > p.wait_limit) {
                tail->abort_flag = 1;
                atomicMax(p.status, (int)SASQ_ERR_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

// Barrier over the 128 epilogue threads (named barrier 2) that also ANDs a predicate.
__device__ __forceinline__ bool epilogue_all_ok(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 2, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}

}  // namespace
}  // namespace sasq
