// Fake-quant forward / STE backward / fused kernels (sm_100a).
//
// One streaming pass over the tensors: 128-bit coalesced loads of x (and the
// upstream gradient), fp32 arithmetic in the fixed order
//     t = x * fl32(1/s);  r = rint(t);  c = clamp(r, -Qn, Qp)          (Eq. 1)
//     y = narrow(c * s)                                                (Sec. 4.2)
//     m = (c == r);  dx = m ? g : 0                                    (Eq. 4)
//     ds += g * (m ? r - t : c)                                        (chain rule)
// 128-bit stores of y and dx, and a deterministic reduction of ds:
// fp32 tree over the 8 products of a vector -> double per thread -> warp
// shuffles -> shared memory -> one double per (tensor, block) in the workspace.
// The block that finishes last (a ticket counter) adds the block partials in a
// fixed order and writes the gradients: one launch, no second pass.
//
// The path is HBM-bound: 4 B / element forward, 6 B backward, 8 B fused.
#pragma once

#include "common.cuh"

namespace sasq {

constexpr int kMaxDescsPerLaunch = 32;   // descriptors that fit one launch's parameter block
constexpr int kMaxGrid = 2048;           // upper bound on blocks per launch (sizes the workspace)

struct QDesc {
    const uint4* x;
    const uint4* g;
    uint4* y;
    uint4* dx;
    long long numel;
    int scale_index;
    int pad;
};

struct QParams {
    QDesc d[kMaxDescsPerLaunch];
    const float* scales;
    double* partials;        // [n][gridDim.x]
    int n;
    float qn;                // 2^(b-1)
    float qp;                // 2^(b-1) - 1
    int* status;
    // second stage (backward only)
    float* grad_scales;
    unsigned* ticket;        // zero before the launch; the last block leaves it zero again
    unsigned accumulate_mask; // bit j: descriptor j's slot is added to, not overwritten
};

struct Quant2 {
    uint32_t y;      // two narrowed outputs
    uint32_t dx;     // two masked gradients
    float p0, p1;    // g * dy/ds
};

// The operator's two non-linear steps, with the ablations of Table 3: VARIANT 0 = full operator,
// 1 = "w/o round" (the rounding step is the identity), 2 = "w/o clamp" (the clamp is the identity and always
// passes the gradient).
template <int VARIANT>
__device__ __forceinline__ float step_round(float t) {
    if constexpr (VARIANT == 1) return t;
    else return rintf(t);
}
template <int VARIANT>
__device__ __forceinline__ float step_clamp(float r, float qn, float qp) {
    if constexpr (VARIANT == 2) return r;
    else return fminf(fmaxf(r, -qn), qp);
}
template <int VARIANT>
__device__ __forceinline__ bool clamp_passes(float c, float r) {
    if constexpr (VARIANT == 2) return true;
    else return c == r;                   // false for NaN as well
}

template <bool BF, bool FWD, bool BWD, int VARIANT>
__device__ __forceinline__ Quant2 quant_pair(uint32_t xw, uint32_t gw, float s, float inv, float qn, float qp) {
    Quant2 o;
    const float2 xf = widen2<BF>(xw);
    const float t0 = __fmul_rn(xf.x, inv);
    const float t1 = __fmul_rn(xf.y, inv);
    const float r0 = step_round<VARIANT>(t0);
    const float r1 = step_round<VARIANT>(t1);
    const float c0 = step_clamp<VARIANT>(r0, qn, qp);
    const float c1 = step_clamp<VARIANT>(r1, qn, qp);
    if constexpr (FWD) {
        o.y = narrow2<BF>(__fmul_rn(c0, s), __fmul_rn(c1, s));
    }
    if constexpr (BWD) {
        const float2 gf = widen2<BF>(gw);
        const bool in0 = clamp_passes<VARIANT>(c0, r0);
        const bool in1 = clamp_passes<VARIANT>(c1, r1);
        o.dx = (in0 ? (gw & 0x0000FFFFu) : 0u) | (in1 ? (gw & 0xFFFF0000u) : 0u);
        o.p0 = __fmul_rn(gf.x, in0 ? __fsub_rn(r0, t0) : c0);
        o.p1 = __fmul_rn(gf.y, in1 ? __fsub_rn(r1, t1) : c1);
    }
    return o;
}

template <int HINT>
__device__ __forceinline__ uint4 load16(const uint4* p) {
    uint4 v;
    if constexpr (HINT == 0) {
        v = *p;
    } else if constexpr (HINT == 1) {
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    } else if constexpr (HINT == 2) {
        asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    } else {
        // streaming, not kept in L1, through the coherent path: valid when the launch also stores to these addresses
        // (y may alias x and grad_x may alias grad_y)
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    }
    return v;
}

template <int HINT>
__device__ __forceinline__ void store16(uint4* p, const uint4& v) {
    if constexpr (HINT == 0) {
        *p = v;
    } else {
        asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                     : "memory");
    }
}

// Block-level sum of one double per thread in a fixed order: lanes by xor
// shuffles (16, 8, 4, 2, 1), then warp 0 adds the warp sums in warp order.
template <int THREADS>
__device__ __forceinline__ double block_sum_fixed(double v, double* smem /* [THREADS/32] */) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) tot += smem[w];
    }
    __syncthreads();
    return tot;   // valid in thread 0
}

template <bool BF, bool FWD, bool BWD, int THREADS, int UNROLL, int MIN_BLOCKS, int LHINT, int SHINT, int VARIANT = 0>
__global__ void __launch_bounds__(THREADS, MIN_BLOCKS) fakequant_kernel(const __grid_constant__ QParams p) {
    __shared__ double warp_sums[THREADS / 32];
    pdl_launch_dependents();
    pdl_wait();
    const float qn = p.qn, qp = p.qp;
    const long long gtid = (long long)blockIdx.x * THREADS + threadIdx.x;
    const long long gstride = (long long)gridDim.x * THREADS;

    for (int ti = 0; ti < p.n; ++ti) {
        const QDesc& d = p.d[ti];
        const float s = __ldg(p.scales + d.scale_index);
        const float inv = __fdiv_rn(1.0f, s);
        if (gtid == 0 && scale_is_bad(s)) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
        const long long nvec = d.numel >> 3;
        double acc = 0.0;

        // The loop bound is the block's, so that every thread makes the same number of trips and the block can meet
        // at a barrier on each: warps that run in step touch neighbouring DRAM pages together, and the whole grid
        // sweeps the tensors as one front.  Measured: 96.9 -> 95.0 us for the 583 MB of the 7B layer's seven tensors;
        // letting the warps drift further apart (no barrier between tensors either) costs 3 % instead.
        for (long long v0b = (long long)blockIdx.x * THREADS; v0b < nvec; v0b += gstride * UNROLL) {
            const long long v0 = v0b + threadIdx.x;
            __syncthreads();
            uint4 xv[UNROLL], gv[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const long long v = v0 + (long long)u * gstride;
                if (v < nvec) {
                    xv[u] = load16<LHINT>(d.x + v);
                    if constexpr (BWD) gv[u] = load16<LHINT>(d.g + v);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const long long v = v0 + (long long)u * gstride;
                if (v < nvec) {
                    const uint32_t xw[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
                    uint32_t gw[4] = {0u, 0u, 0u, 0u};
                    if constexpr (BWD) { gw[0] = gv[u].x; gw[1] = gv[u].y; gw[2] = gv[u].z; gw[3] = gv[u].w; }
                    Quant2 q[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) q[j] = quant_pair<BF, FWD, BWD, VARIANT>(xw[j], gw[j], s, inv, qn, qp);
                    if constexpr (FWD) store16<SHINT>(d.y + v, make_uint4(q[0].y, q[1].y, q[2].y, q[3].y));
                    if constexpr (BWD) {
                        store16<SHINT>(d.dx + v, make_uint4(q[0].dx, q[1].dx, q[2].dx, q[3].dx));
                        const float a = __fadd_rn(__fadd_rn(q[0].p0, q[0].p1), __fadd_rn(q[1].p0, q[1].p1));
                        const float b = __fadd_rn(__fadd_rn(q[2].p0, q[2].p1), __fadd_rn(q[3].p0, q[3].p1));
                        acc += (double)__fadd_rn(a, b);
                    }
                }
            }
        }

        // ragged tail (numel % 8 elements): one element per thread of the last block
        const int tail = (int)(d.numel & 7);
        if (tail != 0 && blockIdx.x == gridDim.x - 1 && threadIdx.x < tail) {
            const long long i = (nvec << 3) + threadIdx.x;
            const uint16_t xh = reinterpret_cast<const uint16_t*>(d.x)[i];
            const float xf = widen1<BF>(xh);
            const float t = __fmul_rn(xf, inv);
            const float r = step_round<VARIANT>(t);
            const float c = step_clamp<VARIANT>(r, qn, qp);
            if constexpr (FWD) reinterpret_cast<uint16_t*>(d.y)[i] = narrow1<BF>(__fmul_rn(c, s));
            if constexpr (BWD) {
                const uint16_t gh = reinterpret_cast<const uint16_t*>(d.g)[i];
                const bool in = clamp_passes<VARIANT>(c, r);
                reinterpret_cast<uint16_t*>(d.dx)[i] = in ? gh : (uint16_t)0;
                acc += (double)__fmul_rn(widen1<BF>(gh), in ? __fsub_rn(r, t) : c);
            }
        }

        if constexpr (BWD) {
            const double tot = block_sum_fixed<THREADS>(acc, warp_sums);
            if (threadIdx.x == 0) p.partials[(long long)ti * gridDim.x + blockIdx.x] = tot;
        }
    }

    if constexpr (BWD) {
        // Second stage, by whichever block finishes last.  Warp w totals the partials of descriptors w, w + W, ...:
        // per lane blocks lane, lane + 32, ... in that order (loads issued 16 at a time so that their latencies
        // overlap), then the xor-shuffle tree.  Then one lane per factor slot adds the totals of the descriptors
        // that share the slot, in descriptor order.  The order depends only on the launch shape, so the result
        // is bit-identical from run to run.
        __shared__ unsigned s_ticket;
        __shared__ double s_total[kMaxDescsPerLaunch];
        if (threadIdx.x == 0) {
            __threadfence();                                   // this block's partials before its ticket
            s_ticket = atomicAdd(p.ticket, 1u);
        }
        __syncthreads();
        if (s_ticket != gridDim.x - 1) return;
        __threadfence();                                       // every other block's partials after their tickets
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int nblk = (int)gridDim.x;
        for (int j = warp; j < p.n; j += THREADS / 32) {
            const double* part = p.partials + (long long)j * nblk;
            double acc = 0.0;
            for (int i0 = lane; i0 < nblk; i0 += 32 * 16) {
                double v[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const int i = i0 + 32 * u;
                    v[u] = (i < nblk) ? __ldcg(part + i) : 0.0;
                }
#pragma unroll
                for (int u = 0; u < 16; ++u) acc += v[u];
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
            if (lane == 0) s_total[j] = acc;
        }
        __syncthreads();
        if (threadIdx.x < p.n) {
            const int j = threadIdx.x;
            const int slot = p.d[j].scale_index;
            bool first = true;
            for (int k = 0; k < j; ++k) first = first && (p.d[k].scale_index != slot);
            if (first) {
                double tot = 0.0;
                for (int k = j; k < p.n; ++k)
                    if (p.d[k].scale_index == slot) tot += s_total[k];
                const float prev = ((p.accumulate_mask >> j) & 1u) ? p.grad_scales[slot] : 0.0f;
                p.grad_scales[slot] = prev + (float)tot;
            }
        }
        if (threadIdx.x == 0) *p.ticket = 0u;                  // ready for the next launch that draws this counter
    }
}

}  // namespace sasq
