// Small-T kernel (T <= 128): swapped operands, K split over a cluster, for one or several same-T problems.
#pragma once

#include "gemm_pair.cuh"

namespace sasq {
namespace {

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
//   warps 2..5  first the activation quantizer (Eq. 1 with the fixed factor), then the epilogue.  Up to 16 rows every
//               CTA quantizes what its own K slice needs straight into the activation tiles of its stages: a row
//               block this small is cheaper to convert 32 times over than to pass through global memory, a counter
//               and a second set of loads (3 us of a 10 us launch, measured).  Above that all CTAs share the T x K
//               elements and publish through one counter; the producers load activation tiles only after it is
//               complete, the weight tiles of the first stages are on their way by then
// ---------------------------------------------------------------------------
constexpr int D_THREADS = 192;
constexpr int D_W_BYTES = 128 * BK;          // weight tile of a stage
constexpr int D_MAX_STAGES = 8;
constexpr int D_RING_BYTES = 192 * 1024;     // stages x (weight tile + activation tile) fit in here
// With T <= 16 a launch is one latency chain (set-up, weights, a few MMAs, reduction, stores) and nothing in it is
// long enough to hide the others.  Such launches take a little less than half of an SM's shared memory, so that
// the CTAs of the NEXT launch of the stream are resident beside them from the start and have their first weight
// tiles in shared memory by the time the kernel before them has finished (the weights are frozen: they are
// requested before the wait on the earlier kernel).
constexpr int D_RING_BYTES_LITE = 108 * 1024;
constexpr int D_LITE_MAX_TP = 16;        // (at 32 rows converting the rows in every CTA was measured slower: 134 against 113 us)

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
    int ring_bytes;      // D_RING_BYTES or D_RING_BYTES_LITE: stages and reduction slots; the barriers follow
    int slots_offset;    // byte offset of the reduction slots in the CTA's shared memory: behind the stages, never
                         // under them, because peers write there while this CTA may still be in its mainloop
    bool local_x;        // T <= 16 with static factors: every CTA quantizes the part of x its own K slice needs
                         // straight into the activation tiles of its pipeline stages (no codes in global memory, no
                         // counter, no activation loads); `quantize`, `ready` and `done` are then unused
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

// Eq. 1 with the fixed factor on the tp x 128 elements of every k-block of a CTA's K slice, written as int8 codes
// into the activation tile of the k-block's pipeline stage: rows of 128 bytes with the 128-byte swizzle the MMA's
// descriptor expects (16-byte piece c of row r sits at piece c ^ (r & 7)).  Run by the 128 threads of warps 2..5.
// One item = 8 adjacent elements of a row (one 128-bit load); a k-block has tp x 16 items, PER per thread; rows >= T
// and columns >= K are zeros.  The words of DEPTH k-blocks are in flight per thread: a slot is refilled as soon as
// it has been converted, so the loads' latency is paid once, not once per k-block.
template <bool BF, int PER, int DEPTH>
__device__ __forceinline__ void local_activation_tiles(const DecodeParams& dp, const DecodeProblem& me, DecodeTail* tail,
                                                       uint8_t* ring, int stage_bytes, int kb_begin, int kb_end, int et,
                                                       int lane) {
    const LinearParams& p = me.lp;
    const bool one = p.chan_inv == nullptr;                       // one static factor for the whole tensor
    const uint4* xsrc = reinterpret_cast<const uint4*>(me.x);
    const int vec_per_row = p.K >> 3;
    const int items_per_kb = dp.tp * 16;
    uint4 buf[DEPTH][PER];
    auto load_kb = [&](int kb, uint4 (&v)[PER]) {
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int item = et + 128 * u;
            const int r = item >> 4, c8 = kb * 16 + (item & 15);                  // row, 8-element column group
            v[u] = (item < items_per_kb && r < p.T && c8 < vec_per_row) ? ld_stream16(xsrc + (size_t)r * vec_per_row + c8)
                                                                         : make_uint4(0u, 0u, 0u, 0u);
        }
    };
#pragma unroll
    for (int d = 0; d < DEPTH; ++d)
        if (kb_begin + d < kb_end) load_kb(kb_begin + d, buf[d]);
    // the factor is fetched with the first loads already in flight
    const float sxq = one ? __ldg(p.x_scale) : 1.0f;
    if (one && blockIdx.x == 0 && et == 0 && scale_is_bad(sxq)) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
    const float inv = __fdiv_rn(1.0f, sxq);
    int stage = 0;
    uint32_t phase = 0;
    for (int base = kb_begin; base < kb_end; base += DEPTH) {
#pragma unroll
        for (int d = 0; d < DEPTH; ++d) {
            const int kb = base + d;
            if (kb < kb_end) {
                if (kb - kb_begin >= dp.stages) {           // the MMAs that read this tile before have completed
                    if (!wait_bounded_d(&tail->empty[stage], phase ^ 1u, tail, p)) return;
                }
                uint8_t* x_tile = ring + (size_t)stage * stage_bytes + D_W_BYTES;
#pragma unroll
                for (int u = 0; u < PER; ++u) {
                    const int item = et + 128 * u;
                    if (item < items_per_kb) {
                        const int r = item >> 4, j = item & 15;
                        const uint2 codes = one ? quantize8<BF, false>(buf[d][u], inv, dp.qn, dp.qp)
                                                : quantize8_channels<BF>(buf[d][u], p.chan_inv + 8 * (kb * 16 + j), dp.qn,
                                                                         dp.qp);
                        *reinterpret_cast<uint2*>(x_tile + r * 128 + (((j >> 1) ^ (r & 7)) << 4) + ((j & 1) << 3)) = codes;
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&tail->full[stage]);
                if (kb + DEPTH < kb_end) load_kb(kb + DEPTH, buf[d]);
                if (++stage == dp.stages) { stage = 0; phase ^= 1u; }
            }
        }
    }
}

// fl32(a) for a 32-bit integer, round to nearest even (what cvt.rn.f32.s32 returns), on the integer and FMA pipes:
// a = hi * 2^16 + lo with hi in [-2^15, 2^15) and lo in [0, 2^16); each half becomes a float exactly by adding it to
// the mantissa of a constant and subtracting the constant, and one fused multiply-add rounds hi * 65536 + lo, which
// is a itself, once.  The conversion pipe takes about 30 cycles per warp instruction here (measured: 135 cycles per
// output with two conversions each), and in this kernel's last phase a warp has nothing else to overlap them with.
__device__ __forceinline__ float int_to_float_exact(int a) {
    const float hi = __fsub_rn(__int_as_float(0x4B400000 + (a >> 16)), 12582912.0f);                     // 1.5 * 2^23 + hi
    const float lo = __fsub_rn(__uint_as_float(0x4B000000u | ((unsigned)a & 0xFFFFu)), 8388608.0f);      // 2^23 + lo
    return __fmaf_rn(hi, 65536.0f, lo);
}

template <bool BF>
__global__ void __launch_bounds__(D_THREADS, 1)
w8a8_decode_kernel(const __grid_constant__ DecodeMaps maps, const __grid_constant__ DecodeParams dp) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* ring = smem_raw;
    DecodeTail* tail = reinterpret_cast<DecodeTail*>(ring + dp.ring_bytes);
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
            // a stage is full when its weight tile has landed (the producer's arrival with the byte count) and, with
            // local activation tiles, when each of the four quantizer warps has written its share of the tile
            ptx::mbar_init(&tail->full[s], dp.local_x ? 5 : 1);
            ptx::mbar_init(&tail->empty[s], 1);
        }
        ptx::mbar_init(&tail->acc_full, 1);
        tail->abort_flag = 0;
        ptx::mbar_init_fence();
        ptx::prefetch_tensormap(tmap_w);
        if (!dp.local_x) ptx::prefetch_tensormap(tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tail->tmem_base, dp.tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = tail->tmem_base;
    // Set-up done.  From here on memory that earlier kernels of the stream may have written (x, the factors) or may
    // still be using (y, the workspace) is touched; the producer warp first requests its weight tiles, which depend on
    // no earlier kernel, and waits afterwards.
    if (warp != 0) pdl_wait();

    // 16-element items the in-kernel quantizer has to publish (none if the activations came quantized)
    const unsigned items_total =
        (dp.quantize && !dp.local_x) ? (unsigned)(((long long)p.T * p.K) >> 4) : 0u;             // of this CTA's problem

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (ptx::elect_one()) {
            bool ok = true;
            int stage = 0;
            uint32_t phase = 0;
            // weight tiles of the first stages go out at once; the activation tiles follow when every CTA has
            // quantized its share of x
            int early = kb_end - kb_begin < dp.stages ? kb_end - kb_begin : dp.stages;
            const uint32_t stage_tx = dp.local_x ? (uint32_t)D_W_BYTES : (uint32_t)stage_bytes;
            for (int i = 0; i < early; ++i) {
                ptx::mbar_arrive_expect_tx(&tail->full[i], stage_tx);
                ptx::tma_load_2d(ring + (size_t)i * stage_bytes, tmap_w, &tail->full[i], (kb_begin + i) * BK, n0);
            }
            pdl_wait();
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
                    ptx::mbar_arrive_expect_tx(&tail->full[stage], stage_tx);
                    ptx::tma_load_2d(w_dst, tmap_w, &tail->full[stage], kb * BK, n0);
                }
                if (!dp.local_x) ptx::tma_load_2d(w_dst + D_W_BYTES, tmap_x, &tail->full[stage], kb * BK, 0);
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
        if (dp.local_x) {
            local_activation_tiles<BF, (D_LITE_MAX_TP * 16) / 128, 8>(dp, me, tail, ring, stage_bytes, kb_begin, kb_end, et,
                                                                      lane);
        } else if (dp.quantize && dp.row_scale_out != nullptr) {
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
                // 32 columns per read where the width allows: a read takes a few hundred cycles to come back
                int c = 0;
                for (; c + 32 <= dp.tp; c += 32) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(taddr + (uint32_t)c, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)(c + 4 * j) * 4u),
                                     "r"(v[4 * j]), "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3]) : "memory");
                }
                for (; c < dp.tp; c += 16) {
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
    // what the stores below need from global memory is requested before the barrier, not after it
    float pre_sx = 1.0f, pre_ws = 0.0f, pre_bias = 0.0f;
    if (warp >= 2) {
        const int rows_own = 128 / dp.split;
        const int n_first = n0 + rank * rows_own + (threadIdx.x - 64) % rows_own;
        if (p.row_scale == nullptr && p.chan_inv == nullptr) pre_sx = __ldg(p.x_scale);
        if (n_first < p.N) {
            pre_ws = __ldg(p.w_scale + n_first);
            if (p.bias != nullptr) pre_bias = widen1<BF>(__ldg(reinterpret_cast<const uint16_t*>(p.bias) + n_first));
        }
    }
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
        const float sx = pre_sx;
        const int items = rows * (dp.tp >> 2);
        // rows divides 128, so a thread's items all belong to ONE channel: its factors were fetched before the
        // barrier and are not loaded again per item (a dependent global load per item made this loop, not the
        // weights, the longest part of a 128-row launch)
        const int r_local = et % rows;
        const int n = n0 + rank * rows + r_local;
        const float ws = pre_ws;
        const float sc = __fmul_rn(sx, ws);
        const float bv = pre_bias;
        if (dp.tp <= 80) {
            // Up to 80 rows the outputs are written directly, 2 bytes per lane: the gathered form below costs a
            // barrier and a second pass and only pays from 96 rows up (measured, same run: 16 rows 77 against 85 us
            // for a layer's four dependent calls, 48 rows 85 against 91, 96 rows and up 2 to 10 % the other way).
            const int32_t* slots = reinterpret_cast<const int32_t*>(ring + dp.slots_offset);
            for (int it = et; it < items; it += 128) {
                const int t0 = (it / rows) << 2;
                int32_t acc[4] = {0, 0, 0, 0};
                for (int r = 0; r < dp.split; ++r) {
                    const int4 v = *reinterpret_cast<const int4*>(slots + (size_t)(r * rows + r_local) * pstride + t0);
                    acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
                }
                if (n < p.N) {
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
        } else {
            // Four items at a time: first all their slot reads (explicit shared-memory loads: through generic pointers the
            // compiler would have to keep every read behind the global stores before it), then their outputs, so that
            // the latencies of the conversions and of the address arithmetic overlap instead of adding up (a thread has
            // up to 32 items and a warp has the SM sub-partition to itself).
            const int rows_log2 = 31 - __clz(rows);                 // rows is a power of two
            const uint32_t slots_s = ptx::smem_u32(ring) + (uint32_t)dp.slots_offset;
            // The outputs of the CTA (T tokens x rows channels) are gathered in shared memory, [token][channel], and then
            // written with 128-bit stores: 2-byte stores, one channel per lane and one token per instruction, were the
            // longest phase of a 128-row launch (13 us of 33 for 128 channels).  The pipeline stages are free by now:
            // the accumulators this warp read were complete, so every load had landed and every MMA had read it.
            uint16_t* y_stage = reinterpret_cast<uint16_t*>(ring);
            int32_t* acc_n = p.acc_out != nullptr ? p.acc_out + n : nullptr;
            const int T = p.T;
            const size_t N = (size_t)p.N;
            for (int it0 = et; it0 < items; it0 += 4 * 128) {
                int32_t acc[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int it = it0 + 128 * u;
                    acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0;
                    if (it < items) {
                        const int t0 = (it >> rows_log2) << 2;
                        for (int r = 0; r < dp.split; ++r) {
                            int4 v;
                            asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                         : "r"(slots_s + (uint32_t)(((r << rows_log2) + r_local) * pstride + t0) * 4u));
                            acc[u][0] += v.x; acc[u][1] += v.y; acc[u][2] += v.z; acc[u][3] += v.w;
                        }
                    }
                }
                if (n < p.N) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int it = it0 + 128 * u;
                        if (it < items) {
                            const int t0 = (it >> rows_log2) << 2;
                            float f[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int t = t0 + j;
                                // a plain load: in the dynamic mode other CTAs wrote the factors during this launch
                                const float sct = (per_row && t < T) ? __fmul_rn(p.row_scale[t], ws) : sc;
                                f[j] = __fmul_rn(int_to_float_exact(acc[u][j]), sct);
                                if (has_bias) f[j] = __fadd_rn(f[j], bv);
                                if (acc_n != nullptr && t < T) acc_n[(size_t)t * N] = acc[u][j];
                            }
                            // two values per narrowing instruction; rows t >= T of the staging tile are never copied out
                            const uint32_t lo = narrow2<BF>(f[0], f[1]), hi = narrow2<BF>(f[2], f[3]);
                            uint16_t* dst = y_stage + t0 * rows + r_local;
                            dst[0] = (uint16_t)(lo & 0xFFFFu);
                            dst[rows] = (uint16_t)(lo >> 16);
                            dst[2 * rows] = (uint16_t)(hi & 0xFFFFu);
                            dst[3 * rows] = (uint16_t)(hi >> 16);
                        }
                    }
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            {
                const int vec_per_token = rows >> 3;                          // rows >= 16: whole groups of 8 channels
                const int vecs = T * vec_per_token;
                const int n_first = n0 + rank * rows;
                uint16_t* y = reinterpret_cast<uint16_t*>(p.y);
                for (int v = et; v < vecs; v += 128) {
                    const int t = v / vec_per_token, c8 = v - t * vec_per_token;
                    const int nn = n_first + 8 * c8;
                    if (nn < p.N)                                             // N % 8 == 0: a group is inside or outside
                        *reinterpret_cast<uint4*>(y + (size_t)t * N + nn) =
                            *reinterpret_cast<const uint4*>(y_stage + t * rows + 8 * c8);
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
    if (dp.quantize && !dp.local_x && threadIdx.x == 0) {
        if (atomicAdd(dp.done, 1u) == gridDim.x - 1) {
            for (int q = 0; q < dp.count; ++q) dp.ready[q] = 0u;
            *dp.done = 0u;
        }
    }
}

}  // namespace
}  // namespace sasq
