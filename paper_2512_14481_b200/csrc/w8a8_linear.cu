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
std::atomic<int> g_gang_launch{0};                 // launch the kernels whose CTAs wait on one another as co-operative grids

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

// FPW = true: the "FP weights" form (Table 3, Eq. 5): both operands are 16-bit floating point (A = the fake-quantized
// activations X' = g(X), B = the weights left as they are), kind::f16 MMAs with fp32 accumulators, no factors in the
// epilogue.  A stage row is still 128 bytes: 64 elements, four MMAs of K = 16.
template <bool BF, bool FPW>
__global__ void __launch_bounds__(NUM_THREADS, 1)
w8a8_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ LinearParams p) {
    constexpr int KB_ELEMS = FPW ? BK / 2 : BK;          // elements of K per stage (the maps count in elements)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    SharedTail* tail = reinterpret_cast<SharedTail*>(tiles + (size_t)STAGES * STAGE_BYTES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&tail->full[s], 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(&tail->tmem_full[b], 1);
            ptx::mbar_init(&tail->tmem_empty[b], EPI_THREADS);
        }
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tail->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;

    const int num_tiles = p.m_blocks * p.n_blocks;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_blk = tile % p.m_blocks, n_blk = tile / p.m_blocks;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = wait_bounded(&tail->empty[stage], phase ^ 1u, tail, p);
                    if (!ok) break;
                    uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
                    uint8_t* b_dst = a_dst + A_STAGE_BYTES;
                    ptx::mbar_arrive_expect_tx(&tail->full[stage], STAGE_BYTES);
                    ptx::tma_load_2d(a_dst, &tmap_a, &tail->full[stage], kb * KB_ELEMS, m_blk * BM);
                    ptx::tma_load_2d(b_dst, &tmap_w, &tail->full[stage], kb * KB_ELEMS, n_blk * BN);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // teardown: copies still in flight must land before the CTA's shared memory goes away.
            // Every armed full barrier either was consumed already (wait returns at once) or completes here.
            if (!ok) {
                for (int s = 0; s < STAGES; ++s) {
                    const long long t0 = clock64();
                    // the phase armed last for stage s: stages before `stage` are in `phase`, the others in phase^1
                    const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
                    while (!ptx::mbar_try_wait(&tail->full[s], par)) {
                        if (clock64() - t0 > (1LL << 24)) break;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            constexpr uint32_t idesc = FPW ? ptx::idesc_f16(BM, BN, BF) : ptx::idesc_i8(BM, BN);
            const uint64_t a_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles));
            const uint64_t b_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles) + A_STAGE_BYTES);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                ok = wait_bounded(&tail->tmem_empty[buf], acc_phase ^ 1u, tail, p);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                uint32_t accumulate = 0;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = wait_bounded(&tail->full[stage], phase, tail, p);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    // either kind advances 32 bytes of K per MMA: +2 in the descriptor's address field
                    if constexpr (FPW) {
                        ptx::mma_f16_ss(d_tmem, a_desc, b_desc, idesc, accumulate);
                        ptx::mma_f16_ss(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
                        ptx::mma_f16_ss(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
                        ptx::mma_f16_ss(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
                    } else {
                        ptx::mma_i8_ss(d_tmem, a_desc, b_desc, idesc, accumulate);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 2, b_desc + 2, idesc);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 4, b_desc + 4, idesc);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 6, b_desc + 6, idesc);
                    }
                    accumulate = 1u;
                    ptx::mma_commit(&tail->empty[stage]);          // stage reusable once these MMAs are done
                    if (kb == p.k_blocks - 1) ptx::mma_commit(&tail->tmem_full[buf]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue (warps 2..5) ----------------
        const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
        const int et = threadIdx.x - 64;                // 0..127
        const bool per_row = p.row_scale != nullptr;
        const bool one_factor = !FPW && !per_row && p.chan_inv == nullptr;   // one static factor for the whole tensor
        const float sx = one_factor ? __ldg(p.x_scale) : 1.0f;
        if (one_factor && blockIdx.x == 0 && et == 0 && scale_is_bad(sx)) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
            const int m_blk = tile % p.m_blocks, n_blk = tile / p.m_blocks;
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int n0 = n_blk * BN;
            // stage the per-channel factors (and bias) of this tile
            asm volatile("bar.sync 1, 128;" ::: "memory");
            for (int j = et; j < BN; j += EPI_THREADS) {
                const int n = n0 + j;
                if constexpr (!FPW) tail->scale[j] = (n < p.N) ? __fmul_rn(sx, __ldg(p.w_scale + n)) : 0.0f;
                if (p.bias != nullptr)
                    tail->bias[j] = (n < p.N) ? widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n)) : 0.0f;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");

            ok = wait_bounded(&tail->tmem_full[buf], acc_phase, tail, p);
            ok = epilogue_all_ok(ok);      // all 128 epilogue threads leave the loop together or not at all
            if (!ok) break;
            ptx::tc_fence_after_sync();

            const int row = m_blk * BM + quad * 32 + lane;
            const bool row_ok = row < p.T;
            const float s_row = (per_row && row_ok) ? __ldg(p.row_scale + row) : 1.0f;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
            uint16_t* yrow = reinterpret_cast<uint16_t*>(p.y) + (size_t)row * p.N + n0;
            int32_t* arow = p.acc_out ? p.acc_out + (size_t)row * p.N + n0 : nullptr;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(taddr + (uint32_t)c, v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    if (row_ok && (n0 + c + j) < p.N) {
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float f0, f1;
                            if constexpr (FPW) {
                                f0 = __uint_as_float(v[j + 2 * q]);
                                f1 = __uint_as_float(v[j + 2 * q + 1]);
                            } else {
                                f0 = __fmul_rn(__int2float_rn((int)v[j + 2 * q]),
                                               out_scale(per_row, s_row, tail->scale[c + j + 2 * q]));
                                f1 = __fmul_rn(__int2float_rn((int)v[j + 2 * q + 1]),
                                               out_scale(per_row, s_row, tail->scale[c + j + 2 * q + 1]));
                            }
                            if (p.bias != nullptr) {
                                f0 = __fadd_rn(f0, tail->bias[c + j + 2 * q]);
                                f1 = __fadd_rn(f1, tail->bias[c + j + 2 * q + 1]);
                            }
                            o[q] = narrow2<BF>(f0, f1);
                        }
                        *reinterpret_cast<uint4*>(yrow + c + j) = make_uint4(o[0], o[1], o[2], o[3]);
                        if (arow != nullptr) {
                            *reinterpret_cast<uint4*>(arow + c + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            *reinterpret_cast<uint4*>(arow + c + j + 4) =
                                make_uint4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                        }
                    }
                }
            }
            // this thread is done reading the accumulator buffer
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&tail->tmem_empty[buf]);
        }
    }

    // ---------------- teardown ----------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}


// ---------------------------------------------------------------------------
// Grouped form (Eq. 3): K is cut into groups of `group` columns, each with its own activation factor s_g.  The
// integer partial product of a group cannot be carried into the next one, so every group gets a fresh int32
// accumulator in TMEM (two of them, alternating), and while the MMAs of the next group run the folding warps add it
// to fp32 running sums that they keep in registers (v + fl32(acc) * fl32(s_g * s_w[n])):
//   y[t,n] = narrow( sum_g fl32(acc_g[t,n]) * fl32(s_g * s_w[n]) (+ bias[n]) ),   groups in order, fp32, no FMA.
// One CTA per 128 x 128 tile; TMEM columns [0,128) and [128,256) hold the two int32 accumulators.  With small groups
// the folding, not the MMAs, sets the pace (a 128-column group is four MMAs), so eight warps do it: two per TMEM
// lane quadrant, 64 columns (64 sums per thread) each.
// ---------------------------------------------------------------------------
constexpr int GBN = 128;
constexpr int G_STAGE_BYTES = BM * BK + GBN * BK;            // 32 KB
constexpr int G_STAGES = (STAGES * STAGE_BYTES) / G_STAGE_BYTES;   // the same ring: 6 stages
static_assert(G_STAGES <= 8, "GroupedTail holds the barriers of up to 8 stages");
constexpr int G_EPI_THREADS = 256;
constexpr int G_THREADS = 64 + G_EPI_THREADS;

struct GroupedTail {
    uint64_t full[8];
    uint64_t empty[8];
    uint64_t tmem_full[ACC_BUFS];
    uint64_t tmem_empty[ACC_BUFS];
    float scale[GBN];              // s_w[n] of the tile's columns
    float bias[GBN];
    uint32_t tmem_base;
    volatile int abort_flag;
};

constexpr size_t kGroupedSmemBytes = 1024 /* alignment slack */ + (size_t)G_STAGES * G_STAGE_BYTES + sizeof(GroupedTail);

struct GroupedParams {
    LinearParams lp;               // x_scale, row_scale, chan_inv unused here
    const float* s_group;          // [groups] activation factor of each K group
    int group_kblocks;             // k-blocks (of 128 columns) per group
    int groups;
};

__device__ __forceinline__ bool wait_bounded_g(uint64_t* bar, uint32_t parity, GroupedTail* tail, const LinearParams& p) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int polls = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (p.wait_limit <= 0 || (++polls & 63) == 0) {
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

// Barrier over the 256 folding threads (named barrier 2) that also ANDs a predicate.
__device__ __forceinline__ bool grouped_all_ok(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 2, 256, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(r)
        : "r"((uint32_t)ok)
        : "memory");
    return r != 0;
}

template <bool BF>
__global__ void __launch_bounds__(G_THREADS, 1)
w8a8_grouped_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                    const __grid_constant__ GroupedParams gp) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GroupedTail* tail = reinterpret_cast<GroupedTail*>(tiles + (size_t)G_STAGES * G_STAGE_BYTES);
    const LinearParams& p = gp.lp;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G_STAGES; ++s) {
            ptx::mbar_init(&tail->full[s], 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(&tail->tmem_full[b], 1);
            ptx::mbar_init(&tail->tmem_empty[b], G_EPI_THREADS / 32);       // one arrival per folding warp
        }
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tail->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;

    const int num_tiles = p.m_blocks * p.n_blocks;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_blk = tile % p.m_blocks, n_blk = tile / p.m_blocks;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = wait_bounded_g(&tail->empty[stage], phase ^ 1u, tail, p);
                    if (!ok) break;
                    uint8_t* a_dst = tiles + (size_t)stage * G_STAGE_BYTES;
                    uint8_t* b_dst = a_dst + BM * BK;
                    ptx::mbar_arrive_expect_tx(&tail->full[stage], G_STAGE_BYTES);
                    ptx::tma_load_2d(a_dst, &tmap_a, &tail->full[stage], kb * BK, m_blk * BM);
                    ptx::tma_load_2d(b_dst, &tmap_w, &tail->full[stage], kb * BK, n_blk * GBN);
                    if (++stage == G_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // after an abort, copies still in flight must land before the CTA's shared memory goes away
            if (!ok) {
                for (int s = 0; s < G_STAGES; ++s) {
                    const long long t0 = clock64();
                    const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
                    while (!ptx::mbar_try_wait(&tail->full[s], par)) {
                        if (clock64() - t0 > (1LL << 24)) break;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: a fresh accumulator for every group ----------------
        if (ptx::elect_one()) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, GBN);
            const uint64_t a_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles));
            const uint64_t b_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles) + BM * BK);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;                 // groups issued so far by this CTA
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int g = 0; g < gp.groups && ok; ++g, ++it) {
                    const int buf = it & 1;
                    const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                    ok = wait_bounded_g(&tail->tmem_empty[buf], acc_phase ^ 1u, tail, p);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(buf * GBN);
                    uint32_t accumulate = 0;
                    for (int kb = 0; kb < gp.group_kblocks; ++kb) {
                        ok = wait_bounded_g(&tail->full[stage], phase, tail, p);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
                        const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (G_STAGE_BYTES >> 4));
                        const uint64_t b_desc = b_desc0 + (uint64_t)(stage * (G_STAGE_BYTES >> 4));
                        ptx::mma_i8_ss(d_tmem, a_desc, b_desc, idesc, accumulate);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 2, b_desc + 2, idesc);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 4, b_desc + 4, idesc);
                        ptx::mma_i8_ss_acc(d_tmem, a_desc + 6, b_desc + 6, idesc);
                        accumulate = 1u;
                        ptx::mma_commit(&tail->empty[stage]);
                        if (kb == gp.group_kblocks - 1) ptx::mma_commit(&tail->tmem_full[buf]);
                        if (++stage == G_STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
        __syncwarp();
    } else {
        // ---------------- warps 2..9: fold each group into the fp32 sums ----------------
        const int quad = warp & 3;                      // TMEM lane quadrant this warp may access
        const int c_begin = warp < 6 ? 0 : GBN / 2;     // its half of the tile's columns
        const int et = threadIdx.x - 64;
        const bool has_bias = p.bias != nullptr;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int m_blk = tile % p.m_blocks, n_blk = tile / p.m_blocks;
            const int n0 = n_blk * GBN;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            for (int j = et; j < GBN; j += G_EPI_THREADS) {
                const int n = n0 + j;
                tail->scale[j] = (n < p.N) ? __ldg(p.w_scale + n) : 0.0f;
                if (has_bias)
                    tail->bias[j] = (n < p.N) ? widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n)) : 0.0f;
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const int row = m_blk * BM + quad * 32 + lane;
            const bool row_ok = row < p.T;
            uint16_t* yrow = reinterpret_cast<uint16_t*>(p.y) + (size_t)row * p.N + n0;
            const uint32_t lanes = tmem_base + ((uint32_t)(quad * 32) << 16);
            float run[GBN / 2];                         // the sums of this thread's row; +0 to start with
#pragma unroll
            for (int j = 0; j < GBN / 2; ++j) run[j] = 0.0f;
            for (int g = 0; g < gp.groups && ok; ++g, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                const float sg = __ldg(gp.s_group + g);
                if (tile == 0 && et == 0 && scale_is_bad(sg)) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
                // every warp waits on its own: whoever gives up raises the abort flag, which ends the others' waits
                ok = wait_bounded_g(&tail->tmem_full[buf], acc_phase, tail, p);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                uint32_t a0[32], a1[32];
                ptx::tmem_ld_32x32(lanes + (uint32_t)(buf * GBN + c_begin), a0);
                ptx::tmem_ld_32x32(lanes + (uint32_t)(buf * GBN + c_begin + 32), a1);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    run[j] = __fadd_rn(run[j], __fmul_rn(__int2float_rn((int)a0[j]),
                                                         __fmul_rn(sg, tail->scale[c_begin + j])));
                    run[32 + j] = __fadd_rn(run[32 + j], __fmul_rn(__int2float_rn((int)a1[j]),
                                                                   __fmul_rn(sg, tail->scale[c_begin + 32 + j])));
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&tail->tmem_empty[buf]);
            }
            if (ok && row_ok) {
#pragma unroll
                for (int j = 0; j < GBN / 2; j += 8) {
                    if (n0 + c_begin + j < p.N) {               // N % 8 == 0: eight columns are in or out together
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float f0 = run[j + 2 * q], f1 = run[j + 2 * q + 1];
                            if (has_bias) {
                                f0 = __fadd_rn(f0, tail->bias[c_begin + j + 2 * q]);
                                f1 = __fadd_rn(f1, tail->bias[c_begin + j + 2 * q + 1]);
                            }
                            o[q] = narrow2<BF>(f0, f1);
                        }
                        *reinterpret_cast<uint4*>(yrow + c_begin + j) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
            // the 256 threads go on to the next tile's barrier together or leave together
            ok = grouped_all_ok(ok);
        }
    }

    // ---------------- teardown ----------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------
// CTA-pair kernel (cta_group::2): two CTAs on neighbouring SMs share one 256 x BN
// output tile.  CTA r of the pair keeps rows [128 r, 128 r + 128) of A and rows
// [BN/2 r, BN/2 (r+1)) of W in its own shared memory, so each byte of W is read
// from shared memory by one SM only while feeding both tensor cores; at the int8
// rate a single CTA's 128 x 256 tile needs more shared-memory bandwidth (TMA
// writes + operand reads) than one SM has.  The leader CTA (rank 0) issues the
// MMAs; completion is multicast to the barriers of both CTAs.
//
// Tiling: every 256-row block of the output is cut into the same number of
// column tiles whose widths are multiples of 16 and differ by at most 16, so
// no tile is ragged; that number is chosen per problem so that the tiles fill
// whole waves of the resident pairs (plan_pair_tiles).
//
// The tensor pipe takes the next MMA only when the one before it is nearly
// done, so whatever the issuing lane does between two MMAs is time the pipe
// idles: the issue loop runs in one elected lane with nothing in it but the
// barrier poll, two descriptor adds, the MMAs and the commit.
// ---------------------------------------------------------------------------
constexpr int PBM = 256;                 // rows per pair tile
#ifndef SASQ_PAIR_STAGES
#define SASQ_PAIR_STAGES 5
#endif
constexpr int P_STAGES = SASQ_PAIR_STAGES;
constexpr int P_A_BYTES = 128 * BK;      // per CTA: 128 rows of A
constexpr int P_B_BYTES_MAX = 128 * BK;  // per CTA: up to 128 rows of W
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES_MAX;
// A stage holds the CTA's half of the W tile first, then its rows of A.  The kernel exists in two layouts of the
// same ring: 5 stages with all 128 rows of A, and, for launches whose problems all have T <= 32, 8 stages with 32
// rows of A (only the leader CTA has rows below T and loads them; the MMA still reads 128 rows from each CTA's
// shared memory, the rest being whatever lies behind, and the accumulator rows they produce are never stored).
// Such launches stream the weights once and are bound by the weight bytes in flight: 8 x 15 KB instead of 5 x 15 KB
// per CTA.
constexpr int P_SMALL_ROWS = 32;
constexpr int P_SMALL_STAGES = (P_STAGES * P_STAGE_BYTES) / (P_B_BYTES_MAX + P_SMALL_ROWS * BK);
constexpr int P_MAX_STAGES = P_SMALL_STAGES > P_STAGES ? P_SMALL_STAGES : P_STAGES;

constexpr int P_NUM_THREADS = 448;       // 14 warps: producer, MMA issuer, 4 epilogue, 8 activation quantizer
constexpr int CONV_THREADS = 256;
constexpr int CONV_WARPS = CONV_THREADS / 32;
constexpr int CONV_ITEMS = 16;           // 8-element items per lane and chunk: 16 128-bit loads in flight per lane
constexpr int CONV_CHUNK = 32 * CONV_ITEMS;   // items per chunk: one warp, 4096 elements
constexpr int kMaxRowBlocks = 1024;      // 256-row blocks the in-kernel quantizer can publish (T <= 262144)
constexpr int kReadySlots = 32;          // concurrently running launches that can each own a set of counters

constexpr int P_OUT_BUF_BYTES = 32 * 128;        // one epilogue warp's staging tile: 32 rows x 64 columns x 2 B
constexpr int P_OUT_BYTES = 4 * 2 * P_OUT_BUF_BYTES;   // 4 warps, double buffered

struct PairTail {
    uint64_t full[P_MAX_STAGES];   // used in the leader: its producer arms it with the bytes of both CTAs' loads
    uint64_t empty[P_MAX_STAGES];  // local: MMA of the pair has consumed the stage
    uint64_t tmem_full[ACC_BUFS];  // local: accumulators of the tile are complete
    uint64_t tmem_empty[ACC_BUFS]; // used in the leader: 8 epilogue warps (4 per CTA) have drained the buffer
    float scale[256];
    float bias[256];
    uint32_t tmem_base;
    volatile int abort_flag;
    int is_last_cta;
};

// the dynamic shared memory window of a CTA without static shared memory starts 1024-byte aligned; the kernel
// checks this and reports SASQ_ERR_CUDA through the status word instead of running if it ever does not hold
constexpr size_t kPairSmemBytes = (size_t)P_STAGES * P_STAGE_BYTES + P_OUT_BYTES + sizeof(PairTail);

struct PairParams {
    LinearParams lp;
    int pair_m_blocks;  // ceil(T / 256)
    int n_tiles;        // column tiles per 256-row block
    int base_units;     // tile j is (base_units + (j < rem_units)) * 16 columns wide
    int rem_units;
    int w_box_rows;     // rows of W each CTA loads per stage: half of the widest tile
    // in-kernel activation quantizer (x == nullptr: A was quantized by an earlier launch)
    const uint16_t* x;  // [T, K] 16-bit activations
    uint8_t* a_int8;    // [T, K] int8 codes (workspace), what tmap_a reads
    unsigned* ready;    // [pair_m_blocks] 8-element items of each 256-row block that are quantized and visible; zero at launch
    unsigned* done;     // CTAs that have finished; the last one zeroes `ready` and this counter again
    float qn, qp;
    // place of this problem in a launch that runs several problems back to back
    int tile_begin;         // tiles of the problems before it
    long long chunk_begin;  // quantizer chunks of the problems before it
};

// One launch runs up to kMaxGroup independent linears back to back: every CTA pair walks one list of tiles that
// covers all of them, and the quantizer warps walk one list of chunks, so the activation quantization of a problem
// (the head of a launch) and the drain of its last tiles overlap with the MMAs of its neighbours.
constexpr int kMaxGroup = 8;
// The quantizer warps run ahead of the MMAs through the whole chunk list, so the int8 activations of every problem of
// a launch are written early and read back later: a launch takes problems only while those codes (with the weights
// streaming past them) stay in the 126 MB L2.
constexpr long long kGroupCodeBytes = 80ll << 20;
// Which tiles a pair computes.  By default pair p takes tiles p, p + pairs, ... of the launch's tile list (column
// tiles fastest, so the pairs of a wave share the rows of A and walk through W together).  When every problem has a
// single 256-row block nothing is shared between tiles, and tiles of different problems cost very different amounts
// (their K differs): the host then deals the tiles out by cost (longest first, always to the least loaded pair) and
// passes each pair's list.
constexpr int kMaxListTiles = 512;
constexpr int kMaxListPairs = 96;
struct GroupParams {
    int count;
    int num_tiles;          // over all problems
    long long num_chunks;   // quantizer chunks over all problems (0: every A was quantized by an earlier launch)
    int ready_count;        // counters the last CTA zeroes again
    unsigned* ready;
    unsigned* done;
    PairParams prob[kMaxGroup];
    int use_list;                                // 0: round-robin over the tile list; 1: the lists below
    uint16_t list_begin[kMaxListPairs + 1];      // pair p computes tile_list[list_begin[p] .. list_begin[p + 1])
    uint16_t tile_list[kMaxListTiles];
};

// the tiles of one pair, in the order it computes them
struct TileWalk {
    int at, end, step;
    bool list;
    __device__ __forceinline__ TileWalk(const GroupParams& gp, int pair_id, int num_pairs) {
        list = gp.use_list != 0;
        at = list ? (int)gp.list_begin[pair_id] : pair_id;
        end = list ? (int)gp.list_begin[pair_id + 1] : gp.num_tiles;
        step = list ? 1 : num_pairs;
    }
    __device__ __forceinline__ bool more() const { return at < end; }
    __device__ __forceinline__ void next() { at += step; }
    __device__ __forceinline__ int tile(const GroupParams& gp) const { return list ? (int)gp.tile_list[at] : at; }
};
// the problem tile g belongs to
__device__ __forceinline__ int problem_of(const GroupParams& gp, int g) {
    int q = 0;
    while (q + 1 < gp.count && g >= gp.prob[q + 1].tile_begin) ++q;
    return q;
}
struct GroupMaps {
    CUtensorMap a[kMaxGroup], w[kMaxGroup], y64[kMaxGroup], y16[kMaxGroup];
};

// first column and width of column tile j
__host__ __device__ __forceinline__ void pair_tile_cols(const PairParams& pp, int j, int* n0, int* width) {
    const int extra = j < pp.rem_units ? j : pp.rem_units;
    *n0 = 16 * (j * pp.base_units + extra);
    *width = 16 * (pp.base_units + (j < pp.rem_units ? 1 : 0));
}

// Eq. 1 with the fixed factor on 8 consecutive elements: one 128-bit word of 16-bit values -> 8 int8 codes.
//   t = x * fl32(1/s) (one fp32 multiply);  code = clamp(rint(t), -Qn, Qp).
// fmax first: it maps NaN to -Qn (the documented behaviour) and applies the lower clamp.  With 8 bits the upper
// clamp and the rounding are what the saturating round-to-nearest-even conversion to s32 followed by the
// saturating pack to s8 does anyway (Qn = 128, Qp = 127); narrower codes take an fmin as well.
template <bool BF, bool EIGHT_BITS>
__device__ __forceinline__ uint2 quantize8(const uint4& v, float inv, float qn, float qp) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int c[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = widen2<BF>(w[q]);
        float t0 = fmaxf(__fmul_rn(f.x, inv), -qn);
        float t1 = fmaxf(__fmul_rn(f.y, inv), -qn);
        if constexpr (!EIGHT_BITS) {
            t0 = fminf(t0, qp);
            t1 = fminf(t1, qp);
        }
        c[2 * q] = __float2int_rn(t0);          // saturates at the int32 range
        c[2 * q + 1] = __float2int_rn(t1);
    }
    uint32_t lo, hi, t;
    // cvt.pack.sat.s8.s32.b32 d, a, b, c:  d = (sat8(a) << 8 | sat8(b)) | (c << 16)
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[3]), "r"(c[2]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(c[1]), "r"(c[0]), "r"(t));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[7]), "r"(c[6]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(c[5]), "r"(c[4]), "r"(t));
    return make_uint2(lo, hi);
}

// the same with one factor per channel: inv8 points at the reciprocals of the 8 channels of this word
template <bool BF>
__device__ __forceinline__ uint2 quantize8_channels(const uint4& v, const float* inv8, float qn, float qp) {
    const float4 ia = __ldg(reinterpret_cast<const float4*>(inv8));
    const float4 ib = __ldg(reinterpret_cast<const float4*>(inv8) + 1);
    const float inv[8] = {ia.x, ia.y, ia.z, ia.w, ib.x, ib.y, ib.z, ib.w};
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    int c[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = widen2<BF>(w[q]);
        c[2 * q] = __float2int_rn(fminf(fmaxf(__fmul_rn(f.x, inv[2 * q]), -qn), qp));
        c[2 * q + 1] = __float2int_rn(fminf(fmaxf(__fmul_rn(f.y, inv[2 * q + 1]), -qn), qp));
    }
    uint32_t lo, hi, t;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[3]), "r"(c[2]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(lo) : "r"(c[1]), "r"(c[0]), "r"(t));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(c[7]), "r"(c[6]), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(c[5]), "r"(c[4]), "r"(t));
    return make_uint2(lo, hi);
}

__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// ---- in-kernel activation quantizer: one chunk = 32 lanes x CONV_ITEMS items of 8 elements, contiguous in x ----
struct ConvJob {
    const uint4* src;            // x as 128-bit words (8 elements each)
    uint2* dst;                  // int8 codes as 64-bit words
    unsigned* ready;             // per 256-row block: items quantized and visible
    long long total;             // items in x
    long long items_per_block;   // items per 256-row block
    float inv, qn, qp;
    bool eight;
    const float* chan_inv;       // per-channel reciprocals, or NULL
    unsigned vec_per_row;        // K / 8
};

__device__ __forceinline__ void conv_load(const ConvJob& j, long long c, int lane, uint4 (&v)[CONV_ITEMS]) {
#pragma unroll
    for (int u = 0; u < CONV_ITEMS; ++u) {
        const long long i = c * CONV_CHUNK + u * 32 + lane;
        if (i < j.total) v[u] = ld_stream16(j.src + i);
    }
}

template <bool BF>
__device__ __forceinline__ void conv_store(const ConvJob& j, long long c, int lane, const uint4 (&v)[CONV_ITEMS]) {
    if (j.chan_inv != nullptr) {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total)
                j.dst[i] = quantize8_channels<BF>(v[u], j.chan_inv + 8 * (unsigned)(i % j.vec_per_row), j.qn, j.qp);
        }
    } else if (j.eight) {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total) j.dst[i] = quantize8<BF, true>(v[u], j.inv, j.qn, j.qp);
        }
    } else {
#pragma unroll
        for (int u = 0; u < CONV_ITEMS; ++u) {
            const long long i = c * CONV_CHUNK + u * 32 + lane;
            if (i < j.total) j.dst[i] = quantize8<BF, false>(v[u], j.inv, j.qn, j.qp);
        }
    }
}

// every lane's stores visible at GPU scope (and to the TMA unit), then one add per row block the chunk touches
__device__ __forceinline__ void conv_publish(const ConvJob& j, long long c, int lane) {
    asm volatile("fence.proxy.async.global;" ::: "memory");
    __threadfence();
    __syncwarp();
    if (lane == 0) {
        const long long first = c * CONV_CHUNK;
        const long long end = (first + CONV_CHUNK < j.total) ? first + CONV_CHUNK : j.total;
        long long i = first;
        while (i < end) {
            const long long blk = i / j.items_per_block;
            const long long blk_end = (blk + 1) * j.items_per_block;
            const long long upto = blk_end < end ? blk_end : end;
            atomicAdd(j.ready + blk, (unsigned)(upto - i));
            i = upto;
        }
    }
}

// Bounded wait until *counter (written by other CTAs with a fence before their atomic add) reaches `need`.
__device__ __forceinline__ bool wait_rows_ready(const unsigned* counter, unsigned need, PairTail* tail,
                                                const LinearParams& p) {
    const long long t0 = clock64();
    int polls = 0;
    for (;;) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (v >= need) return true;
        if (p.wait_limit <= 0 || (++polls & 15) == 0) {
            if (tail->abort_flag) return false;
            if (clock64() - t0 > p.wait_limit) {
                tail->abort_flag = 1;
                atomicMax(p.status, (int)SASQ_ERR_TIMEOUT);
                return false;
            }
        }
        __nanosleep(64);
    }
}

__device__ __forceinline__ bool wait_bounded_pair(uint64_t* bar, uint32_t parity, PairTail* tail,
                                                  const LinearParams& p) {
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

template <bool BF, bool SMALL>
__global__ void __launch_bounds__(P_NUM_THREADS, 1)
w8a8_gemm_pair_kernel(const __grid_constant__ GroupMaps maps, const __grid_constant__ GroupParams gp) {
    constexpr int STAGES = SMALL ? P_SMALL_STAGES : P_STAGES;
    constexpr int A_BYTES = SMALL ? P_SMALL_ROWS * BK : P_A_BYTES;
    constexpr int STAGE_BYTES = P_B_BYTES_MAX + A_BYTES;
    static_assert(STAGES * STAGE_BYTES <= P_STAGES * P_STAGE_BYTES, "both layouts use the same ring");
    static_assert(STAGE_BYTES % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    uint8_t* out_stage = tiles + (size_t)P_STAGES * P_STAGE_BYTES;          // 1024-byte aligned
    PairTail* tail = reinterpret_cast<PairTail*>(out_stage + P_OUT_BYTES);
    const LinearParams& p0 = gp.prob[0].lp;         // the status word and the wait limit are the same for all problems
    if ((ptx::smem_u32(tiles) & 1023u) != 0) {      // uniform over the grid: every CTA returns before any barrier
        if (threadIdx.x == 0) atomicMax(p0.status, (int)SASQ_ERR_CUDA);
        return;
    }

    pdl_launch_dependents();

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();        // 0 = leader

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&tail->full[s], 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        for (int b = 0; b < ACC_BUFS; ++b) {
            ptx::mbar_init(&tail->tmem_full[b], 1);
            ptx::mbar_init(&tail->tmem_empty[b], 8);
        }
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        for (int q = 0; q < gp.count; ++q) {
            ptx::prefetch_tensormap(&maps.a[q]);
            ptx::prefetch_tensormap(&maps.w[q]);
            ptx::prefetch_tensormap(&maps.y64[q]);
            ptx::prefetch_tensormap(&maps.y16[q]);
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(&tail->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();            // both CTAs' barriers exist before anyone signals across the pair
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;
    pdl_wait();                         // set-up done; from here on global memory of earlier kernels is used

    const int pair_id = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        if (ptx::elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int ready_blk = -1, ready_q = -1;
            for (TileWalk walk(gp, pair_id, num_pairs); walk.more() && ok; walk.next()) {
                const int g = walk.tile(gp);
                const int q = problem_of(gp, g);
                const PairParams& pp = gp.prob[q];
                const LinearParams& p = pp.lp;
                const CUtensorMap* tmap_a = &maps.a[q];
                const CUtensorMap* tmap_w = &maps.w[q];
                // bytes both CTAs' loads deliver per stage: two halves of the W tile, and A from both (or, in the
                // small layout, from the leader alone)
                const uint32_t stage_tx = (uint32_t)(2 * pp.w_box_rows * BK + (SMALL ? A_BYTES : 2 * A_BYTES));
                const bool load_a = !SMALL || rank == 0;
                const int tile = g - pp.tile_begin;
                const int m_blk = tile / pp.n_tiles;
                int n0, bn;
                pair_tile_cols(pp, tile - m_blk * pp.n_tiles, &n0, &bn);
                const int a_row = m_blk * PBM + (int)rank * 128;
                // this CTA's half of the tile's W rows; the box is as high as half the widest tile, so a narrower
                // tile fetches 8 rows it does not use (rows past N read as zero)
                const int w_row = n0 + (int)rank * (bn >> 1);
                int kb_a = 0;            // k-blocks of this tile whose W half is already on its way
                if (pp.x != nullptr && (m_blk != ready_blk || q != ready_q)) {
                    // The rows of this block must have been quantized, by whichever CTAs had them, and be visible
                    // to the TMA unit before the first A load of the tile.  W does not depend on that: while
                    // waiting, fill the free stages with the W halves of the first k-blocks.
                    const int rows = p.T - m_blk * PBM;
                    const unsigned need = (unsigned)((rows < PBM ? rows : PBM) * (p.K >> 3));
                    int st = stage;
                    uint32_t ph = phase;
                    while (kb_a < p.k_blocks && kb_a < STAGES && ptx::mbar_test_wait(&tail->empty[st], ph ^ 1u)) {
                        const uint32_t full_leader = ptx::mapa_u32(ptx::smem_u32(&tail->full[st]), 0);
                        if (rank == 0) ptx::mbar_arrive_expect_tx(&tail->full[st], stage_tx);
                        ptx::tma_load_2d_pair(tiles + (size_t)st * STAGE_BYTES, tmap_w, full_leader, kb_a * BK, w_row);
                        ++kb_a;
                        if (++st == STAGES) { st = 0; ph ^= 1u; }
                    }
                    ok = wait_rows_ready(pp.ready + m_blk, need, tail, p);
                    if (!ok) break;
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    ready_blk = m_blk;
                    ready_q = q;
                }
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    uint8_t* w_dst = tiles + (size_t)stage * STAGE_BYTES;
                    // Only the leader arms the barrier (with the bytes of both CTAs); the partner's copies
                    // may complete first, which merely drives the transaction count negative for a while:
                    // the phase cannot complete before the leader's arrival.
                    const uint32_t full_leader = ptx::mapa_u32(ptx::smem_u32(&tail->full[stage]), 0);
                    if (kb >= kb_a) {
                        ok = wait_bounded_pair(&tail->empty[stage], phase ^ 1u, tail, p);
                        if (!ok) break;
                        if (rank == 0) ptx::mbar_arrive_expect_tx(&tail->full[stage], stage_tx);
                        ptx::tma_load_2d_pair(w_dst, tmap_w, full_leader, kb * BK, w_row);
                    }
                    if (load_a) ptx::tma_load_2d_pair(w_dst + P_B_BYTES_MAX, tmap_a, full_leader, kb * BK, a_row);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // after an abort, copies may still be in flight into this CTA's shared memory: their barrier lives in
            // the leader, so give them a bounded grace period (a copy takes microseconds) before the CTA may exit
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < (1LL << 22)) __nanosleep(1000);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (rank == 0 && ptx::elect_one()) {
            const uint64_t a_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles) + P_B_BYTES_MAX);
            const uint64_t b_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(tiles));
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (TileWalk walk(gp, pair_id, num_pairs); walk.more() && ok; walk.next(), ++it) {
                const int g = walk.tile(gp);
                const int q = problem_of(gp, g);
                const PairParams& pp = gp.prob[q];
                const LinearParams& p = pp.lp;
                int n0, bn;
                pair_tile_cols(pp, (g - pp.tile_begin) % pp.n_tiles, &n0, &bn);
                const uint32_t idesc = ptx::idesc_i8(PBM, bn);
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                ok = wait_bounded_pair(&tail->tmem_empty[buf], acc_phase ^ 1u, tail, p);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                uint32_t accumulate = 0;            // the first MMA of a tile overwrites the accumulators
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = wait_bounded_pair(&tail->full[stage], phase, tail, p);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // 32 bytes of K per MMA inside the swizzled 128-byte row: +2 in the descriptor's address field
                    const uint64_t a_desc = a_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    ptx::mma_i8_ss_pair(d_tmem, a_desc, b_desc, idesc, accumulate);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 2, b_desc + 2, idesc);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 4, b_desc + 4, idesc);
                    ptx::mma_i8_ss_pair_acc(d_tmem, a_desc + 6, b_desc + 6, idesc);
                    accumulate = 1u;
                    ptx::mma_commit_pair(&tail->empty[stage], 0x3);          // stage reusable once these MMAs are done
                    if (kb == p.k_blocks - 1) ptx::mma_commit_pair(&tail->tmem_full[buf], 0x3);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ---------------- activation quantizer (warps 6..13 of both CTAs) ----------------
        // x is taken as a flat run of T * K / 8 items of 8 elements, cut into chunks of 4096 elements that are
        // dealt round-robin over all quantizer warps of the grid in address order, so the row blocks become ready
        // in the order the tiles need them.  Every warp runs its own load -> quantize -> store -> fence -> publish
        // pipeline with 16 128-bit loads in flight per lane; the warps drift apart, which keeps DRAM busy while
        // some of them wait for their stores to be acknowledged.
        // With several problems in the launch their chunks form one list, in problem order.
        {
            const int cw = warp - (P_NUM_THREADS - CONV_THREADS) / 32;          // 0..7
            const long long stride = (long long)gridDim.x * CONV_WARPS;
            ConvJob job{};
            int q = 0, job_q = -1;
            for (long long c = (long long)blockIdx.x * CONV_WARPS + cw; c < gp.num_chunks; c += stride) {
                while (q + 1 < gp.count && c >= gp.prob[q + 1].chunk_begin) ++q;
                if (q != job_q) {
                    const PairParams& pp = gp.prob[q];
                    const LinearParams& p = pp.lp;
                    job.src = reinterpret_cast<const uint4*>(pp.x);
                    job.dst = reinterpret_cast<uint2*>(pp.a_int8);
                    job.ready = pp.ready;
                    job.total = (long long)p.T * (p.K >> 3);
                    job.items_per_block = (long long)PBM * (p.K >> 3);
                    job.chan_inv = p.chan_inv;
                    job.vec_per_row = (unsigned)(p.K >> 3);
                    job.inv = p.chan_inv == nullptr ? __fdiv_rn(1.0f, __ldg(p.x_scale)) : 0.0f;
                    job.qn = pp.qn;
                    job.qp = pp.qp;
                    job.eight = pp.qp == 127.0f;
                    job_q = q;
                }
                const long long lc = c - gp.prob[q].chunk_begin;
                uint4 v[CONV_ITEMS];
                conv_load(job, lc, lane, v);
                conv_store<BF>(job, lc, lane, v);
                conv_publish(job, lc, lane);
            }
        }
    } else {
        // ---------------- epilogue (warps 2..5 of both CTAs) ----------------
        const int quad = warp & 3;
        const int et = threadIdx.x - 64;
        if (blockIdx.x == 0 && et < gp.count) {          // one thread per problem checks its static factor
            const LinearParams& pe = gp.prob[et].lp;
            if (pe.row_scale == nullptr && pe.chan_inv == nullptr && scale_is_bad(__ldg(pe.x_scale)))
                atomicMax(pe.status, (int)SASQ_ERR_BAD_SCALE);
        }
        // The outputs are not read again by this launch: their lines should leave L2 first, during the launch (whose
        // DRAM interface is mostly idle), instead of staying behind dirty and being written back under the next kernel.
        const uint64_t y_policy = ptx::l2_policy_evict_first();
        bool ok = true;
        int it = 0;
        unsigned out_flip = 0;
        for (TileWalk walk(gp, pair_id, num_pairs); walk.more() && ok; walk.next(), ++it) {
            const int g = walk.tile(gp);
            const int q = problem_of(gp, g);
            const PairParams& pp = gp.prob[q];
            const LinearParams& p = pp.lp;
            const CUtensorMap* tmap_y64 = &maps.y64[q];
            const CUtensorMap* tmap_y16 = &maps.y16[q];
            const bool per_row = p.row_scale != nullptr;
            const bool one_factor = !per_row && p.chan_inv == nullptr;       // one static factor for the whole tensor
            const float sx = one_factor ? __ldg(p.x_scale) : 1.0f;
            const bool has_bias = p.bias != nullptr;
            const int tile = g - pp.tile_begin;
            const int m_blk = tile / pp.n_tiles;
            int n0, bn;
            pair_tile_cols(pp, tile - m_blk * pp.n_tiles, &n0, &bn);
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            for (int j = et; j < bn; j += EPI_THREADS) {
                const int n = n0 + j;
                tail->scale[j] = (n < p.N) ? __fmul_rn(sx, __ldg(p.w_scale + n)) : 0.0f;
                if (has_bias)
                    tail->bias[j] = (n < p.N) ? widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n)) : 0.0f;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");

            ok = wait_bounded_pair(&tail->tmem_full[buf], acc_phase, tail, p);
            ok = epilogue_all_ok(ok);
            if (!ok) break;
            ptx::tc_fence_after_sync();

            // Each warp owns 32 rows.  64 columns at a time: TMEM -> registers -> dequantise -> this warp's
            // 128-byte-swizzled staging tile -> one TMA store (whole 128-byte lines; rows >= T and columns >= N
            // are clipped by the tensor map).  A tile width that is not a multiple of 64 ends in 16-column pieces.
            const int row0 = m_blk * PBM + (int)rank * 128 + quad * 32;
            const int row = row0 + lane;
            const bool row_ok = row < p.T;
            const float s_row = (per_row && row_ok) ? __ldg(p.row_scale + row) : 1.0f;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 256);
            int32_t* arow = p.acc_out ? p.acc_out + (size_t)row * p.N + n0 : nullptr;
            uint8_t* my_stage = out_stage + (size_t)quad * 2 * P_OUT_BUF_BYTES;
            int c = 0;
#pragma unroll 1
            for (; c + 64 <= bn; c += 64) {
                uint8_t* sbuf = my_stage + (size_t)(out_flip & 1) * P_OUT_BUF_BYTES;
                if (lane == 0) ptx::bulk_wait_group_read<1>();      // the store that used this buffer has read it
                __syncwarp();
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(taddr + (uint32_t)(c + 32 * h), v);
                    ptx::tmem_ld_wait();
                    const float* sc = tail->scale + c + 32 * h;
                    const float* bi = tail->bias + c + 32 * h;
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            float f0 = __fmul_rn(__int2float_rn((int)v[j + 2 * q]), out_scale(per_row, s_row, sc[j + 2 * q]));
                            float f1 = __fmul_rn(__int2float_rn((int)v[j + 2 * q + 1]),
                                                 out_scale(per_row, s_row, sc[j + 2 * q + 1]));
                            if (has_bias) {
                                f0 = __fadd_rn(f0, bi[j + 2 * q]);
                                f1 = __fadd_rn(f1, bi[j + 2 * q + 1]);
                            }
                            o[q] = narrow2<BF>(f0, f1);
                        }
                        const int piece = 4 * h + (j >> 3);           // 16-byte piece of the 128-byte row
                        *reinterpret_cast<uint4*>(sbuf + lane * 128 + ((piece ^ (lane & 7)) << 4)) =
                            make_uint4(o[0], o[1], o[2], o[3]);
                        if (arow != nullptr && row_ok && (n0 + c + 32 * h + j) < p.N) {
                            int32_t* a = arow + c + 32 * h + j;
                            *reinterpret_cast<uint4*>(a) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            *reinterpret_cast<uint4*>(a + 4) = make_uint4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                        }
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::tma_store_2d_hint(tmap_y64, sbuf, n0 + c, row0, y_policy);
                    ptx::bulk_commit_group();
                }
                ++out_flip;
            }
#pragma unroll 1
            for (; c < bn; c += 16) {       // 16-column pieces: 32-byte rows, 32-byte swizzle
                uint8_t* sbuf = my_stage + (size_t)(out_flip & 1) * P_OUT_BUF_BYTES;
                if (lane == 0) ptx::bulk_wait_group_read<1>();
                __syncwarp();
                uint32_t v[16];
                ptx::tmem_ld_32x16(taddr + (uint32_t)c, v);
                ptx::tmem_ld_wait();
                const float* sc = tail->scale + c;
                const float* bi = tail->bias + c;
#pragma unroll
                for (int j = 0; j < 16; j += 8) {
                    uint32_t o[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float f0 = __fmul_rn(__int2float_rn((int)v[j + 2 * q]), out_scale(per_row, s_row, sc[j + 2 * q]));
                        float f1 = __fmul_rn(__int2float_rn((int)v[j + 2 * q + 1]),
                                                 out_scale(per_row, s_row, sc[j + 2 * q + 1]));
                        if (has_bias) {
                            f0 = __fadd_rn(f0, bi[j + 2 * q]);
                            f1 = __fadd_rn(f1, bi[j + 2 * q + 1]);
                        }
                        o[q] = narrow2<BF>(f0, f1);
                    }
                    const int piece = j >> 3;
                    *reinterpret_cast<uint4*>(sbuf + lane * 32 + ((piece ^ ((lane >> 2) & 1)) << 4)) =
                        make_uint4(o[0], o[1], o[2], o[3]);
                    if (arow != nullptr && row_ok && (n0 + c + j) < p.N) {
                        int32_t* a = arow + c + j;
                        *reinterpret_cast<uint4*>(a) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        *reinterpret_cast<uint4*>(a + 4) = make_uint4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::tma_store_2d_hint(tmap_y16, sbuf, n0 + c, row0, y_policy);
                    ptx::bulk_commit_group();
                }
                ++out_flip;
            }
            // this warp has drained the accumulator buffer: tell the leader's MMA issuer
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa_u32(ptx::smem_u32(&tail->tmem_empty[buf]), 0));
        }
        // the output stores have read their shared-memory source; the writes themselves are complete by the end of
        // the grid, which is all that a later kernel or the host can observe
        if (lane == 0) ptx::bulk_wait_group_read<0>();
    }

    // ---------------- teardown ----------------
    // Neither CTA may leave while its partner can still read its shared memory, signal its barriers or
    // run MMAs into its TMEM.  The epilogues of both CTAs have seen the last tile's accumulators complete
    // (or every role has given up after a bounded wait), so a pair-wide barrier is enough.
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
    if (gp.done != nullptr) {
        // the CTA that finishes last leaves the counters at zero for the next launch that draws them
        if (threadIdx.x == 0) tail->is_last_cta = (atomicAdd(gp.done, 1u) == gridDim.x - 1) ? 1 : 0;
        __syncthreads();
        if (tail->is_last_cta) {
            for (int i = threadIdx.x; i < gp.ready_count; i += P_NUM_THREADS) gp.ready[i] = 0u;
            if (threadIdx.x == 0) *gp.done = 0u;
        }
    }
}

// Eq. 1 with the fixed factor, written once to int8 (operand A of the GEMM).
// 16 elements per thread: two 128-bit loads, one 128-bit store.
// ---------------------------------------------------------------------------
// Small-T kernel (T <= 128: decode and short prompts).  The work is streaming W once from HBM, so the roles of the
// operands are swapped: 128 rows of W are the M side of the MMA (every instruction consumes 4 KB of weights), the
// T activation rows, padded to a multiple of 16, are the N side, and the accumulator tile in TMEM is
// [128 output channels x T tokens].  To occupy the whole chip a cluster of S CTAs shares one 128-channel tile and
// splits K; each CTA sends its partial accumulators through distributed shared memory to the CTA that owns the
// channels (CTA r owns 128 / S of them), and after one cluster barrier every CTA adds the S partials of its channels
// (int32: exact in any order), dequantises and stores them.
//   warp 0      TMA producer: W tile (128 x 128 B) + int8 activation tile (TP x 128 B) per stage
//   warp 1      MMA issuer
//   warps 2..5  first the activation quantizer (Eq. 1 with the fixed factor, all CTAs share the T x K elements and
//               publish through one counter; the producers load activation tiles only after it is complete, the
//               weight tiles of the first stages are on their way by then), then the epilogue
// ---------------------------------------------------------------------------
constexpr int D_THREADS = 192;
constexpr int D_W_BYTES = 128 * BK;          // weight tile of a stage
constexpr int D_MAX_STAGES = 8;
constexpr int D_RING_BYTES = 192 * 1024;     // stages x (weight tile + activation tile) fit in here

struct DecodeTail {
    uint64_t full[D_MAX_STAGES];
    uint64_t empty[D_MAX_STAGES];
    uint64_t acc_full;
    uint32_t tmem_base;
    volatile int abort_flag;
    int is_last_cta;
    float row_max[4];    // dynamic per-token factors: the four quantizer warps' maxima of the row in hand
};

// One launch may carry several independent problems with the same T (the q/k/v projections of a decode step, say):
// the 128-channel tiles of all of them form one list of clusters, and every CTA helps to quantize every problem's x.
constexpr int kMaxDecodeGroup = 8;
struct DecodeProblem {
    LinearParams lp;
    const uint16_t* x;   // NULL: the codes in a_int8 were written by an earlier launch
    uint8_t* a_int8;
    int tile_begin;      // 128-channel tiles of the problems before this one
};
struct DecodeMaps {
    CUtensorMap w[kMaxDecodeGroup], x[kMaxDecodeGroup];
};
struct DecodeParams {
    int count;
    DecodeProblem prob[kMaxDecodeGroup];
    int tp;              // T rounded up to a multiple of 16: N of the MMA
    int stages;
    int split;           // CTAs per cluster = K slices
    int n_tiles;         // 128-channel tiles of all problems
    uint32_t tmem_cols;  // power of two >= max(32, tp)
    int slots_offset;    // byte offset of the reduction slots in the CTA's shared memory: behind the stages, never
                         // under them, because peers write there while this CTA may still be in its mainloop
    bool quantize;       // the activation quantizer runs inside this launch
    unsigned* ready;     // [count] per problem: 16-element items quantized and visible; zero at launch
    unsigned* done;
    float qn, qp;
    float* row_scale_out;   // non-NULL: dynamic per-token factors, computed here (a CTA's four quantizer warps per
                            // row) and written there; lp.row_scale points at the same array for the epilogue
};

constexpr int D_DYN_WORDS = 12;   // 128-bit words of a row a quantizer thread keeps in registers between the two passes

__device__ __forceinline__ bool wait_bounded_d(uint64_t* bar, uint32_t parity, DecodeTail* tail, const LinearParams& p) {
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

template <bool BF>
__global__ void __launch_bounds__(D_THREADS, 1)
w8a8_decode_kernel(const __grid_constant__ DecodeMaps maps, const __grid_constant__ DecodeParams dp) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* ring = smem_raw;
    DecodeTail* tail = reinterpret_cast<DecodeTail*>(ring + D_RING_BYTES);
    // the problem this cluster's tile belongs to
    const int tile_all = blockIdx.x / dp.split;
    int q_mine = 0;
    while (q_mine + 1 < dp.count && tile_all >= dp.prob[q_mine + 1].tile_begin) ++q_mine;
    const DecodeProblem& me = dp.prob[q_mine];
    const LinearParams& p = me.lp;
    const CUtensorMap* tmap_w = &maps.w[q_mine];
    const CUtensorMap* tmap_x = &maps.x[q_mine];
    if ((ptx::smem_u32(ring) & 1023u) != 0) {       // uniform over the grid: every CTA returns before any barrier
        if (threadIdx.x == 0) atomicMax(p.status, (int)SASQ_ERR_CUDA);
        return;
    }
    pdl_launch_dependents();

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int rank = (int)ptx::cluster_ctarank();
    const int n_tile = tile_all - me.tile_begin;
    const int n0 = n_tile * 128;
    const int stage_bytes = D_W_BYTES + dp.tp * BK;
    // this CTA's slice of the k-blocks
    const int kb_begin = (int)(((long long)rank * p.k_blocks) / dp.split);
    const int kb_end = (int)(((long long)(rank + 1) * p.k_blocks) / dp.split);

    if (threadIdx.x == 0) {
        for (int s = 0; s < dp.stages; ++s) {
            ptx::mbar_init(&tail->full[s], 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        ptx::mbar_init(&tail->acc_full, 1);
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        ptx::prefetch_tensormap(tmap_w);
        ptx::prefetch_tensormap(tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tail->tmem_base, dp.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;
    pdl_wait();                         // set-up done; from here on global memory of earlier kernels is used

    // 16-element items the in-kernel quantizer has to publish (none if the activations came quantized)
    const unsigned items_total = dp.quantize ? (unsigned)(((long long)p.T * p.K) >> 4) : 0u;   // of this CTA's problem

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            bool ok = true;
            int stage = 0;
            uint32_t phase = 0;
            // weight tiles of the first stages go out at once; the activation tiles follow when every CTA has
            // quantized its share of x
            int early = kb_end - kb_begin < dp.stages ? kb_end - kb_begin : dp.stages;
            for (int i = 0; i < early; ++i) {
                ptx::mbar_arrive_expect_tx(&tail->full[i], (uint32_t)stage_bytes);
                ptx::tma_load_2d(ring + (size_t)i * stage_bytes, tmap_w, &tail->full[i], (kb_begin + i) * BK, n0);
            }
            if (items_total != 0) {
                const long long t0 = clock64();
                int polls = 0;
                for (;;) {
                    unsigned v;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(dp.ready + q_mine) : "memory");
                    if (v >= items_total) break;
                    if (p.wait_limit <= 0 || (++polls & 15) == 0) {
                        if (tail->abort_flag) { ok = false; break; }
                        if (clock64() - t0 > p.wait_limit) {
                            tail->abort_flag = 1;
                            atomicMax(p.status, (int)SASQ_ERR_TIMEOUT);
                            ok = false;
                            break;
                        }
                    }
                    __nanosleep(32);
                }
                asm volatile("fence.proxy.async.global;" ::: "memory");
            }
            for (int kb = kb_begin; kb < kb_end && ok; ++kb) {
                uint8_t* w_dst = ring + (size_t)stage * stage_bytes;
                if (kb - kb_begin >= early) {
                    ok = wait_bounded_d(&tail->empty[stage], phase ^ 1u, tail, p);
                    if (!ok) break;
                    ptx::mbar_arrive_expect_tx(&tail->full[stage], (uint32_t)stage_bytes);
                    ptx::tma_load_2d(w_dst, tmap_w, &tail->full[stage], kb * BK, n0);
                }
                ptx::tma_load_2d(w_dst + D_W_BYTES, tmap_x, &tail->full[stage], kb * BK, 0);
                if (++stage == dp.stages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {      // copies in flight must land before the CTA's shared memory goes away
                const long long t0 = clock64();
                while (clock64() - t0 < (1LL << 22)) __nanosleep(1000);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (ptx::elect_one()) {
            const uint32_t idesc = ptx::idesc_i8(128, dp.tp);
            const uint64_t w_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(ring));
            const uint64_t x_desc0 = ptx::smem_desc_k_major_sw128(ptx::smem_u32(ring) + D_W_BYTES);
            const uint32_t stage_step = (uint32_t)(stage_bytes >> 4);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t accumulate = 0;
            bool ok = true;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                ok = wait_bounded_d(&tail->full[stage], phase, tail, p);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint64_t w_desc = w_desc0 + (uint64_t)(stage * stage_step);
                const uint64_t x_desc = x_desc0 + (uint64_t)(stage * stage_step);
                ptx::mma_i8_ss(tmem_base, w_desc, x_desc, idesc, accumulate);
                ptx::mma_i8_ss_acc(tmem_base, w_desc + 2, x_desc + 2, idesc);
                ptx::mma_i8_ss_acc(tmem_base, w_desc + 4, x_desc + 4, idesc);
                ptx::mma_i8_ss_acc(tmem_base, w_desc + 6, x_desc + 6, idesc);
                accumulate = 1u;
                ptx::mma_commit(&tail->empty[stage]);
                if (++stage == dp.stages) { stage = 0; phase ^= 1u; }
            }
            if (ok) ptx::mma_commit(&tail->acc_full);       // also right for an empty slice: arrives at once
        }
        __syncwarp();
    } else {
        // ---------------- activation quantizer, then epilogue (warps 2..5) ----------------
        const int et = threadIdx.x - 64;                       // 0..127
        if (dp.quantize && dp.row_scale_out != nullptr) {
            // Dynamic per-token quantization (Sec. 4.4, generation phase) inside the launch: the rows are dealt to
            // the CTAs, and the 128 quantizer threads of a CTA take a row together.  The row's factor is its own
            // max-based one, s_t = max_k |x[t,k]| / Qp (Eq. 1; an all-zero row takes s_t = 1).  Each thread keeps its
            // words of the row in registers between the maximum and the quantization (rows longer than
            // 128 x D_DYN_WORDS words read the rest a second time).
            const int vec = p.K >> 3;
            unsigned rows_done = 0;
            for (int r = blockIdx.x; r < p.T; r += gridDim.x) {
                const uint4* row = reinterpret_cast<const uint4*>(me.x) + (size_t)r * vec;
                uint4 keep[D_DYN_WORDS];
                float m = 0.0f;
#pragma unroll
                for (int u = 0; u < D_DYN_WORDS; ++u) {
                    const int i = et + 128 * u;
                    if (i < vec) {
                        keep[u] = row[i];
                        const uint32_t w4[4] = {keep[u].x, keep[u].y, keep[u].z, keep[u].w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float2 f = widen2<BF>(w4[q]);
                            m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
                        }
                    }
                }
                for (int i = et + 128 * D_DYN_WORDS; i < vec; i += 128) {
                    const uint4 v = row[i];
                    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float2 f = widen2<BF>(w4[q]);
                        m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
                    }
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
                if (lane == 0) tail->row_max[warp - 2] = m;
                asm volatile("bar.sync 3, 128;" ::: "memory");
                m = fmaxf(fmaxf(tail->row_max[0], tail->row_max[1]), fmaxf(tail->row_max[2], tail->row_max[3]));
                const float sc = m > 0.0f ? __fdiv_rn(m, dp.qp) : 1.0f;
                const float inv = __fdiv_rn(1.0f, sc);
                if (et == 0) dp.row_scale_out[r] = sc;
                uint2* orow = reinterpret_cast<uint2*>(me.a_int8) + (size_t)r * vec;
#pragma unroll
                for (int u = 0; u < D_DYN_WORDS; ++u) {
                    const int i = et + 128 * u;
                    if (i < vec) orow[i] = quantize8<BF, false>(keep[u], inv, dp.qn, dp.qp);
                }
                for (int i = et + 128 * D_DYN_WORDS; i < vec; i += 128)
                    orow[i] = quantize8<BF, false>(row[i], inv, dp.qn, dp.qp);
                ++rows_done;
                asm volatile("bar.sync 3, 128;" ::: "memory");      // row_max is free for the next row
            }
            asm volatile("fence.proxy.async.global;" ::: "memory");
            __threadfence();
            asm volatile("bar.sync 3, 128;" ::: "memory");          // every thread's codes are out and fenced
            if (et == 0 && rows_done != 0) atomicAdd(dp.ready + q_mine, rows_done * (unsigned)(p.K >> 4));
        } else if (dp.quantize) {
            // every CTA takes its share of every problem's x, in problem order
            for (int q = 0; q < dp.count; ++q) {
                const DecodeProblem& pr = dp.prob[q];
                const LinearParams& lp = pr.lp;
                const bool one = lp.chan_inv == nullptr;                 // one static factor for the whole tensor
                const float sxq = one ? __ldg(lp.x_scale) : 1.0f;
                if (one && blockIdx.x == 0 && et == 0 && scale_is_bad(sxq)) atomicMax(lp.status, (int)SASQ_ERR_BAD_SCALE);
                const float inv = __fdiv_rn(1.0f, sxq);
                const uint4* src = reinterpret_cast<const uint4*>(pr.x);
                uint4* dst = reinterpret_cast<uint4*>(pr.a_int8);
                const unsigned items = (unsigned)(((long long)lp.T * lp.K) >> 4);
                unsigned mine = 0;
                for (unsigned i = blockIdx.x * 128u + (unsigned)et; i < items; i += gridDim.x * 128u) {
                    const uint4 a = ld_stream16(src + 2 * (size_t)i), b = ld_stream16(src + 2 * (size_t)i + 1);
                    uint2 lo, hi;
                    if (lp.chan_inv != nullptr) {
                        const float* ci = lp.chan_inv + 16 * (i % (unsigned)(lp.K >> 4));
                        lo = quantize8_channels<BF>(a, ci, dp.qn, dp.qp);
                        hi = quantize8_channels<BF>(b, ci + 8, dp.qn, dp.qp);
                    } else {
                        lo = quantize8<BF, false>(a, inv, dp.qn, dp.qp);
                        hi = quantize8<BF, false>(b, inv, dp.qn, dp.qp);
                    }
                    dst[i] = make_uint4(lo.x, lo.y, hi.x, hi.y);
                    ++mine;
                }
                asm volatile("fence.proxy.async.global;" ::: "memory");
                __threadfence();
                // one add per warp
                for (int off = 16; off > 0; off >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, off);
                if (lane == 0 && mine != 0) atomicAdd(dp.ready + q, mine);
            }
        } else if (blockIdx.x == 0 && et == 0 && p.row_scale == nullptr && p.chan_inv == nullptr &&
                   scale_is_bad(__ldg(p.x_scale))) {
            atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);             // codes from an earlier launch: check the factor
        }

        // epilogue part 1: this CTA's partial accumulators go from TMEM straight into the shared memory of the CTA
        // that will reduce them (remote stores through distributed shared memory, into slots behind the pipeline stages).  CTA r
        // owns channels [r * 128 / S, (r + 1) * 128 / S) of the tile and holds one slot per K slice:
        // [S slots][128 / S channels][tp + 4 words]; rows tp + 4 words apart keep 128-bit accesses aligned and
        // let eight consecutive rows cover all banks.
        const int quad = warp & 3;                              // TMEM lane quadrant of this warp
        const int pstride = dp.tp + 4;
        const int rows = 128 / dp.split;
        bool ok = wait_bounded_d(&tail->acc_full, 0u, tail, p);
        ok = epilogue_all_ok(ok);
        if (ok) {
            ptx::tc_fence_after_sync();
            const int n_local = quad * 32 + lane;
            const int owner = n_local / rows;
            const uint32_t local = ptx::smem_u32(ring) + (uint32_t)dp.slots_offset +
                                   (uint32_t)((rank * rows + (n_local - owner * rows)) * pstride) * 4u;
            const uint32_t dst = ptx::mapa_u32(local, (uint32_t)owner);
            if (kb_end > kb_begin) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
                for (int c = 0; c < dp.tp; c += 16) {
                    uint32_t v[16];
                    ptx::tmem_ld_32x16(taddr + (uint32_t)c, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)(c + 4 * j) * 4u),
                                     "r"(v[4 * j]), "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3]) : "memory");
                }
            } else {
                for (int c = 0; c < dp.tp; c += 4)
                    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(dst + (uint32_t)c * 4u), "r"(0u)
                                 : "memory");
            }
        }
        ptx::tc_fence_before_sync();
    }

    // every CTA's partials are in their owner's shared memory after this barrier (or the launch has been abandoned:
    // a role gave up after a bounded wait and the status word says so; the sums below are then garbage but every
    // access stays in bounds).  Nobody touches another CTA's shared memory afterwards, so the CTAs may finish
    // independently.
    __syncthreads();
    ptx::cluster_sync_all();

    if (warp >= 2) {
        // epilogue part 2: add the S slots of this CTA's channels, dequantise, store.  One work item = one channel
        // x four consecutive tokens (one 128-bit read per slot); consecutive threads take consecutive channels so
        // that the 16-bit stores of one token coalesce.
        const int et = threadIdx.x - 64;
        const int rows = 128 / dp.split;
        const int pstride = dp.tp + 4;
        const bool has_bias = p.bias != nullptr;
        const bool per_row = p.row_scale != nullptr;
        const float sx = (per_row || p.chan_inv != nullptr) ? 1.0f : __ldg(p.x_scale);
        const int items = rows * (dp.tp >> 2);
        const int32_t* slots = reinterpret_cast<const int32_t*>(ring + dp.slots_offset);
        for (int it = et; it < items; it += 128) {
            const int r_local = it % rows;
            const int t0 = (it / rows) << 2;
            const int n = n0 + rank * rows + r_local;
            int32_t acc[4] = {0, 0, 0, 0};
            for (int r = 0; r < dp.split; ++r) {
                const int4 v = *reinterpret_cast<const int4*>(slots + (size_t)(r * rows + r_local) * pstride + t0);
                acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
            }
            if (n < p.N) {
                const float ws = __ldg(p.w_scale + n);
                const float sc = __fmul_rn(sx, ws);
                const float bv = has_bias ? widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n)) : 0.0f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int t = t0 + j;
                    if (t < p.T) {
                        // a plain load: in the dynamic mode other CTAs wrote the factors during this launch
                        const float sct = per_row ? __fmul_rn(p.row_scale[t], ws) : sc;
                        float f = __fmul_rn(__int2float_rn(acc[j]), sct);
                        if (has_bias) f = __fadd_rn(f, bv);
                        reinterpret_cast<uint16_t*>(p.y)[(size_t)t * p.N + n] = narrow1<BF>(f);
                        if (p.acc_out != nullptr) p.acc_out[(size_t)t * p.N + n] = acc[j];
                    }
                }
            }
        }
    }

    // ---------------- teardown ----------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, dp.tmem_cols);
    }
    // the CTA that finishes last leaves the counters at zero for the next launch that draws them
    if (dp.quantize && threadIdx.x == 0) {
        if (atomicAdd(dp.done, 1u) == gridDim.x - 1) {
            for (int q = 0; q < dp.count; ++q) dp.ready[q] = 0u;
            *dp.done = 0u;
        }
    }
}

// The same quantizer as a launch of its own (small T, or more row blocks than the in-kernel counters hold):
// 8 elements per thread and step, one 128-bit load, one 64-bit store.
template <bool BF>
__global__ void __launch_bounds__(256) quantize_act_kernel(const uint4* __restrict__ x, uint2* __restrict__ out,
                                                           long long n8, const float* __restrict__ x_scale,
                                                           const float* __restrict__ chan_inv, unsigned vec_per_row,
                                                           float qn, float qp) {
    pdl_wait();
    const float inv = chan_inv == nullptr ? __fdiv_rn(1.0f, __ldg(x_scale)) : 0.0f;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride)
        out[i] = chan_inv == nullptr ? quantize8<BF, false>(x[i], inv, qn, qp)
                                     : quantize8_channels<BF>(x[i], chan_inv + 8 * (unsigned)(i % vec_per_row), qn, qp);
}

// reciprocals of the per-channel factors, fl32(1 / s[k / group]) (group = 1: one factor per channel), once per
// call; a zero / non-finite factor is reported
__global__ void __launch_bounds__(256) reciprocal_factors_kernel(const float* __restrict__ s, float* __restrict__ inv,
                                                                 int K, int group, int* status) {
    pdl_launch_dependents();
    pdl_wait();
    const int k = blockIdx.x * 256 + threadIdx.x;
    if (k >= K) return;
    const float sk = s[k / group];
    if (scale_is_bad(sk)) atomicMax(status, (int)SASQ_ERR_BAD_SCALE);
    inv[k] = __fdiv_rn(1.0f, sk);
}

// Dynamic per-token quantization (Sec. 4.4, generation phase): one block per row of x.  The row's factor is its
// own max-based one, s_t = max_k |x[t,k]| / Qp (Eq. 1; an all-zero row takes s_t = 1), then the row is quantized with
// it exactly like the static path: code = clamp(rint(x * fl32(1 / s_t))).  The row is read twice; the second read
// comes from L2.
template <bool BF>
__global__ void __launch_bounds__(256) quantize_rows_dynamic_kernel(const uint4* __restrict__ x, uint2* __restrict__ out,
                                                                    float* __restrict__ row_scale, int K, float qn,
                                                                    float qp) {
    __shared__ float warp_max[8];
    __shared__ float s_inv;
    pdl_launch_dependents();
    pdl_wait();
    const int vec = K >> 3;
    const uint4* row = x + (size_t)blockIdx.x * vec;
    float m = 0.0f;
    for (int i = threadIdx.x; i < vec; i += 256) {
        const uint4 v = row[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 f = widen2<BF>(w[q]);
            m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        float mm = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) mm = fmaxf(mm, warp_max[w]);
        const float sc = mm > 0.0f ? __fdiv_rn(mm, qp) : 1.0f;
        row_scale[blockIdx.x] = sc;
        s_inv = __fdiv_rn(1.0f, sc);
    }
    __syncthreads();
    const float inv = s_inv;
    uint2* orow = out + (size_t)blockIdx.x * vec;
    for (int i = threadIdx.x; i < vec; i += 256) orow[i] = quantize8<BF, false>(row[i], inv, qn, qp);
}

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
// the set it used at zero again; launches draw the sets round-robin, so two launches share one only if more than
// kReadySlots launches of this kernel were running at the same time.
static __device__ unsigned g_a_ready[kReadySlots][kMaxRowBlocks];
static __device__ unsigned g_a_done[kReadySlots];

}  // namespace

void linear_reset_counters(cudaStream_t st) {
    void *r = nullptr, *d = nullptr;
    if (cudaGetSymbolAddress(&r, g_a_ready) == cudaSuccess && cudaGetSymbolAddress(&d, g_a_done) == cudaSuccess) {
        cudaMemsetAsync(r, 0, sizeof(unsigned) * kReadySlots * kMaxRowBlocks, st);
        cudaMemsetAsync(d, 0, sizeof(unsigned) * kReadySlots, st);
        cudaStreamSynchronize(st);
    }
}

namespace {

bool next_ready_slot(unsigned** ready, unsigned** done) {
    static unsigned* ready_base[64] = {nullptr};
    static unsigned* done_base[64] = {nullptr};
    static std::atomic<unsigned> next{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (ready_base[dev] == nullptr) {
        unsigned *r = nullptr, *d = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&r), g_a_ready) != cudaSuccess) return false;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&d), g_a_done) != cudaSuccess) return false;
        done_base[dev] = d;
        ready_base[dev] = r;
    }
    const unsigned slot = next.fetch_add(1u, std::memory_order_relaxed) % kReadySlots;
    *ready = ready_base[dev] + (size_t)slot * kMaxRowBlocks;
    *done = done_base[dev] + slot;
    return true;
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

// Largest K split (CTAs per cluster) of the small-T kernel with which all n_tiles clusters are resident at once (the
// in-kernel activation quantizer needs every CTA of the grid running); 0 if even one CTA per tile does not fit.
int decode_split(bool bf, int n_tiles, int k_blocks, int sm_count, size_t smem_bytes) {
    static int ready[64][2] = {};
    static int cap[64][2][4] = {};            // resident clusters for S = 1, 2, 4, 8; 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const void* fn = bf ? reinterpret_cast<const void*>(w8a8_decode_kernel<true>)
                        : reinterpret_cast<const void*>(w8a8_decode_kernel<false>);
    if (!ready[dev][bf]) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
            return 0;
        ready[dev][bf] = 1;
    }
    for (int si = 3; si >= 0; --si) {
        const int S = 1 << si;
        if (S > k_blocks || (long long)n_tiles * S > sm_count) continue;
        if (cap[dev][bf][si] == 0) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(sm_count / S * S), 1, 1);
            cfg.blockDim = dim3(D_THREADS, 1, 1);
            cfg.dynamicSmemBytes = smem_bytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)S;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, fn, &cfg) != cudaSuccess || clusters <= 0) clusters = -1;
            cap[dev][bf][si] = clusters;
        }
        if (cap[dev][bf][si] >= n_tiles) return S;
    }
    return 0;
}

// Column tiling of a 256-row block for `pairs` resident CTA pairs.  One MMA of N columns keeps the tensor pipe
// busy for about max(N, 208) / 2 cycles (below 208 columns the instruction is bound by reading its A operand), and a
// launch takes as long as its fullest pair: waves x that cost of the widest tile.  Tiles are at least 16 x 8 = 128
// columns wide unless N itself is narrower.  Fewer, wider tiles win ties (less fixed work per tile).
void plan_pair_tiles(PairParams* pp, int m_blocks, long long N, int pairs) {
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
    constexpr size_t kDecodeSmem = (size_t)D_RING_BYTES + sizeof(DecodeTail);
    dp.tp = (T + 15) / 16 * 16;
    const int stage_bytes = D_W_BYTES + dp.tp * BK;
    const int slot_bytes = (128 * (dp.tp + 4) * 4 + 1023) & ~1023;          // S x (128 / S) rows of tp + 4 words
    const int ring_bytes = D_RING_BYTES - slot_bytes;
    dp.slots_offset = ring_bytes;
    dp.stages = ring_bytes / stage_bytes < D_MAX_STAGES ? ring_bytes / stage_bytes : D_MAX_STAGES;
    dp.split = split;
    dp.tmem_cols = 32;
    while ((int)dp.tmem_cols < dp.tp) dp.tmem_cols <<= 1;
    if (dp.quantize && !next_ready_slot(&dp.ready, &dp.done)) return SASQ_ERR_CUDA;
    for (int q = 0; q < dp.count; ++q)
        if (!make_tmap(&maps.x[q], dp.prob[q].a_int8, T, dp.prob[q].lp.K, dp.tp)) return SASQ_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(dp.n_tiles * split), 1, 1);
    cfg.blockDim = dim3(D_THREADS, 1, 1);
    cfg.dynamicSmemBytes = kDecodeSmem;
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
    cfg.numAttrs = (dp.quantize && g_gang_launch.load(std::memory_order_relaxed)) ? 3 : 2;
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
    constexpr size_t kDecodeSmem = (size_t)D_RING_BYTES + sizeof(DecodeTail);
    const int n_tiles128 = (int)((N + 127) / 128);
    const int split = (T <= BM && n_tiles128 <= sm_count)
                          ? decode_split(dt == SASQ_BF16, n_tiles128, k_blocks, sm_count, kDecodeSmem) : 0;
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
    cudaError_t e;
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
            if (!next_ready_slot(&gp.ready, &gp.done)) return SASQ_ERR_CUDA;
            pp.ready = gp.ready;
            gp.ready_count = pp.pair_m_blocks;
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
        if (!next_ready_slot(&gp.ready, &gp.done)) return SASQ_ERR_CUDA;
        int off = 0;
        for (int q = 0; q < gp.count; ++q) {
            gp.prob[q].ready = gp.ready + off;
            off += gp.prob[q].pair_m_blocks;
        }
        gp.ready_count = off;
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
        constexpr size_t kDecodeSmem = (size_t)D_RING_BYTES + sizeof(DecodeTail);
        const int split = decode_split(bf, dp.n_tiles, min_kblocks, sm_count, kDecodeSmem);
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
