// Activation quantizers that run as launches of their own, and the reciprocals of per-channel / per-group factors.
#pragma once

#include "gemm_pair.cuh"

namespace sasq {
namespace {

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

}  // namespace
}  // namespace sasq
