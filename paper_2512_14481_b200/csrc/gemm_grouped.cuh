// Grouped form of Eq. 3: per-group int32 accumulators folded into fp32 sums.
#pragma once

#include "linear_common.cuh"

namespace sasq {
namespace {

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

}  // namespace
}  // namespace sasq
