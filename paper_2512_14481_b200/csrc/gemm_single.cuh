// Single-CTA 128 x 256-tile GEMM kernel (int8, or 16-bit operands for the "FP weights" form): the fallback when
// neither the CTA-pair kernel nor the small-T kernel applies.
#pragma once

#include "linear_common.cuh"

namespace sasq {
namespace {

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

}  // namespace
}  // namespace sasq
