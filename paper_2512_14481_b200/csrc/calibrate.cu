// PTQ initialisation helpers (Sec. 4.1; Eq. 1): the max-based activation factor
// S = max|X| / Qp of one calibration batch, and the per-output-channel weight
// quantizer.  They run once at set-up, not on the hot path.
#include "common.cuh"

namespace sasq {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxBlocks = 1024;

__device__ __forceinline__ float block_max(float v, float* smem) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
    __syncthreads();
    float m = 0.0f;
    if (threadIdx.x < 32) {
        m = (threadIdx.x < kThreads / 32) ? smem[threadIdx.x] : 0.0f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    }
    __syncthreads();
    return m;   // valid in warp 0
}

template <bool BF>
__global__ void __launch_bounds__(kThreads) absmax_partial_kernel(const uint16_t* __restrict__ x, long long numel,
                                                                  float* __restrict__ partial) {
    __shared__ float smem[kThreads / 32];
    float m = 0.0f;
    const long long stride = (long long)gridDim.x * kThreads;
    const long long nvec = numel >> 3;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < nvec; i += stride) {
        const uint4 v = xv[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = widen2<BF>(w[j]);
            m = fmaxf(m, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (int)(numel & 7))
        m = fmaxf(m, fabsf(widen1<BF>(x[(nvec << 3) + threadIdx.x])));
    m = block_max(m, smem);
    if (threadIdx.x == 0) partial[blockIdx.x] = m;
}

__global__ void __launch_bounds__(kThreads) absmax_final_kernel(const float* __restrict__ partial, int n, float qp,
                                                                float* __restrict__ scale_out) {
    __shared__ float smem[kThreads / 32];
    float m = 0.0f;
    for (int i = threadIdx.x; i < n; i += kThreads) m = fmaxf(m, partial[i]);
    m = block_max(m, smem);
    if (threadIdx.x == 0) scale_out[0] = __fdiv_rn(m, qp);
}

// Max-based factor per channel (column of x[T, K]).  A thread owns 8 adjacent channels (one 128-bit word per row)
// and walks down the rows of its block's row group; the groups meet in an atomic max on the bit patterns of the
// (non-negative) maxima, whose integer order is their order as floats.
template <bool BF>
__global__ void __launch_bounds__(kThreads) absmax_channels_kernel(const uint4* __restrict__ x, int T, int vec_per_row,
                                                                   int rows_per_group, unsigned* __restrict__ max_bits) {
    const int cv = blockIdx.x * kThreads + threadIdx.x;          // which 8-channel word of a row
    if (cv >= vec_per_row) return;
    const int r0 = blockIdx.y * rows_per_group;
    const int r1 = r0 + rows_per_group < T ? r0 + rows_per_group : T;
    float m[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    for (int r = r0; r < r1; ++r) {
        const uint4 v = x[(size_t)r * vec_per_row + cv];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = widen2<BF>(w[j]);
            m[2 * j] = fmaxf(m[2 * j], fabsf(f.x));
            m[2 * j + 1] = fmaxf(m[2 * j + 1], fabsf(f.y));
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) atomicMax(max_bits + 8 * cv + j, __float_as_uint(m[j]));
}

// bit patterns of the maxima -> factors, in place: s[k] = max / Qp
__global__ void __launch_bounds__(kThreads) absmax_channels_final_kernel(unsigned* __restrict__ max_bits, int K, float qp) {
    const int k = blockIdx.x * kThreads + threadIdx.x;
    if (k < K) max_bits[k] = __float_as_uint(__fdiv_rn(__uint_as_float(max_bits[k]), qp));
}

// avg[i] <- avg[i] + (value[i] - avg[i]) / count: the mean of the first `count` values once each has been fed in turn
__global__ void __launch_bounds__(kThreads) running_mean_kernel(float* __restrict__ avg, const float* __restrict__ value,
                                                                int n, float count) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i < n) {
        const float a = avg[i];
        avg[i] = count <= 1.0f ? value[i] : __fadd_rn(a, __fdiv_rn(__fsub_rn(value[i], a), count));
    }
}

// one block per output channel (row of w[N, K])
__global__ void __launch_bounds__(kThreads) quantize_weight_kernel(const float* __restrict__ w, int8_t* __restrict__ w_int,
                                                                   float* __restrict__ w_scale, long long K, float qn,
                                                                   float qp) {
    __shared__ float smem[kThreads / 32];
    __shared__ float s_inv;
    const float* row = w + (long long)blockIdx.x * K;
    float m = 0.0f;
    for (long long k = threadIdx.x; k < K; k += kThreads) m = fmaxf(m, fabsf(row[k]));
    m = block_max(m, smem);
    if (threadIdx.x == 0) {
        const float sc = m > 0.0f ? __fdiv_rn(m, qp) : 1.0f;
        w_scale[blockIdx.x] = sc;
        s_inv = __fdiv_rn(1.0f, sc);
    }
    __syncthreads();
    const float inv = s_inv;
    int8_t* out = w_int + (long long)blockIdx.x * K;
    for (long long k = threadIdx.x; k < K; k += kThreads) {
        const float r = rintf(__fmul_rn(row[k], inv));
        out[k] = (int8_t)(int)fminf(fmaxf(r, -qn), qp);
    }
}

// One AdamW step on the factors (the only trainable parameters, Sec. 4.2 / 5.1), fp32, one thread per factor:
//   m = b1 m + (1 - b1) g;  v = b2 v + (1 - b2) g^2;  s -= lr * ( (m / c1) / (sqrt(v / c2) + eps) + wd * s )
// with the bias corrections c1 = 1 - b1^step, c2 = 1 - b2^step computed on the host.
__global__ void __launch_bounds__(kThreads) adamw_scales_kernel(float* __restrict__ s, const float* __restrict__ g,
                                                                float* __restrict__ m, float* __restrict__ v, int n,
                                                                float lr, float b1, float b2, float eps, float wd,
                                                                float c1, float c2) {
    const int i = blockIdx.x * kThreads + threadIdx.x;
    if (i >= n) return;
    const float gi = g[i];
    const float mi = __fadd_rn(__fmul_rn(b1, m[i]), __fmul_rn(1.0f - b1, gi));
    const float vi = __fadd_rn(__fmul_rn(b2, v[i]), __fmul_rn(1.0f - b2, __fmul_rn(gi, gi)));
    m[i] = mi;
    v[i] = vi;
    const float mhat = __fdiv_rn(mi, c1);
    const float vhat = __fdiv_rn(vi, c2);
    const float si = s[i];
    const float upd = __fadd_rn(__fdiv_rn(mhat, __fadd_rn(__fsqrt_rn(vhat), eps)), __fmul_rn(wd, si));
    s[i] = __fsub_rn(si, __fmul_rn(lr, upd));
}

}  // namespace
}  // namespace sasq

extern "C" {

int sasq_adamw_scales(float* scales_dev, const float* grad_scales_dev, float* exp_avg_dev, float* exp_avg_sq_dev,
                      int n, int step, float lr, float beta1, float beta2, float eps, float weight_decay,
                      void* stream) {
    using namespace sasq;
    if (n < 0 || step < 1) return SASQ_ERR_INVALID_ARG;
    if (n > 0 && (scales_dev == nullptr || grad_scales_dev == nullptr || exp_avg_dev == nullptr ||
                  exp_avg_sq_dev == nullptr))
        return SASQ_ERR_INVALID_ARG;
    if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps > 0.0f))
        return SASQ_ERR_INVALID_ARG;
    if (n == 0) return SASQ_OK;
    if (device_sm_count_if_sm100() <= 0) return SASQ_ERR_UNSUPPORTED;
    double p1 = 1.0, p2 = 1.0;
    for (int i = 0; i < step; ++i) { p1 *= (double)beta1; p2 *= (double)beta2; }
    adamw_scales_kernel<<<(n + kThreads - 1) / kThreads, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        scales_dev, grad_scales_dev, exp_avg_dev, exp_avg_sq_dev, n, lr, beta1, beta2, eps, weight_decay,
        (float)(1.0 - p1), (float)(1.0 - p2));
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

size_t sasq_absmax_scale_workspace(int64_t numel) {
    (void)numel;
    return (size_t)sasq::kMaxBlocks * sizeof(float);
}

int sasq_absmax_scale(const void* x, int64_t numel, int dt, int bits, float* scale_out_dev, void* workspace,
                      size_t ws_bytes, void* stream) {
    using namespace sasq;
    if (numel < 0 || scale_out_dev == nullptr || bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (numel > 0 && (x == nullptr || !aligned16(x))) return SASQ_ERR_INVALID_ARG;
    if (workspace == nullptr || !aligned16(workspace) || ws_bytes < sasq_absmax_scale_workspace(numel))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    long long blocks = ((numel >> 3) + kThreads - 1) / kThreads;
    if (blocks < 1) blocks = 1;
    if (blocks > kMaxBlocks) blocks = kMaxBlocks;
    if (blocks > (long long)sm_count * 4) blocks = (long long)sm_count * 4;
    float* partial = static_cast<float*>(workspace);
    if (dt == SASQ_BF16)
        absmax_partial_kernel<true><<<(int)blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), numel, partial);
    else
        absmax_partial_kernel<false><<<(int)blocks, kThreads, 0, st>>>(static_cast<const uint16_t*>(x), numel, partial);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    absmax_final_kernel<<<1, kThreads, 0, st>>>(partial, (int)blocks, (float)((1 << (bits - 1)) - 1), scale_out_dev);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

int sasq_absmax_scale_per_channel(const void* x, int64_t T, int64_t K, int dt, int bits, float* scales_out_dev,
                                  void* stream) {
    using namespace sasq;
    if (T < 0 || K <= 0 || scales_out_dev == nullptr || bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (T > 0 && (x == nullptr || !aligned16(x))) return SASQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(scales_out_dev) & 3u) return SASQ_ERR_INVALID_ARG;
    if (K % 8 != 0 || T > (1 << 24) || K > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* bits_out = reinterpret_cast<unsigned*>(scales_out_dev);
    if (cudaMemsetAsync(bits_out, 0, sizeof(unsigned) * (size_t)K, st) != cudaSuccess) return SASQ_ERR_CUDA;
    if (T > 0) {
        const int vec = (int)(K / 8);
        const int col_blocks = (vec + kThreads - 1) / kThreads;
        // enough row groups to fill the GPU a few times over, at least 16 rows each
        long long groups = ((long long)sm_count * 8 + col_blocks - 1) / col_blocks;
        if (groups > (T + 15) / 16) groups = (T + 15) / 16;
        if (groups < 1) groups = 1;
        if (groups > 65535) groups = 65535;
        const int rows_per_group = (int)((T + groups - 1) / groups);
        const dim3 grid((unsigned)col_blocks, (unsigned)((T + rows_per_group - 1) / rows_per_group), 1);
        if (dt == SASQ_BF16)
            absmax_channels_kernel<true><<<grid, kThreads, 0, st>>>(static_cast<const uint4*>(x), (int)T, vec,
                                                                   rows_per_group, bits_out);
        else
            absmax_channels_kernel<false><<<grid, kThreads, 0, st>>>(static_cast<const uint4*>(x), (int)T, vec,
                                                                    rows_per_group, bits_out);
        if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    }
    absmax_channels_final_kernel<<<(unsigned)((K + kThreads - 1) / kThreads), kThreads, 0, st>>>(
        bits_out, (int)K, (float)((1 << (bits - 1)) - 1));
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

int sasq_running_mean(float* mean_dev, const float* value_dev, int n, int count, void* stream) {
    using namespace sasq;
    if (n < 0 || count < 1 || (n > 0 && (mean_dev == nullptr || value_dev == nullptr))) return SASQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(mean_dev) & 3u) || (reinterpret_cast<uintptr_t>(value_dev) & 3u))
        return SASQ_ERR_INVALID_ARG;
    if (n == 0) return SASQ_OK;
    if (device_sm_count_if_sm100() <= 0) return SASQ_ERR_UNSUPPORTED;
    running_mean_kernel<<<(unsigned)((n + kThreads - 1) / kThreads), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        mean_dev, value_dev, n, (float)count);
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

int sasq_quantize_weight(const float* w, int8_t* w_int, float* w_scale, int64_t N, int64_t K, int bits,
                         void* stream) {
    using namespace sasq;
    if (N < 0 || K <= 0 || bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (N > 0 && (w == nullptr || w_int == nullptr || w_scale == nullptr)) return SASQ_ERR_INVALID_ARG;
    if (N > 0x7FFFFFFF) return SASQ_ERR_UNSUPPORTED;
    if (N == 0) return SASQ_OK;
    if (device_sm_count_if_sm100() <= 0) return SASQ_ERR_UNSUPPORTED;
    quantize_weight_kernel<<<(int)N, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        w, w_int, w_scale, K, (float)(1 << (bits - 1)), (float)((1 << (bits - 1)) - 1));
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

}  // extern "C"
