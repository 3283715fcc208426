// Fake-quant forward / STE backward with one factor per channel (column of x[T, K]): the granularity of the
// paper's experiments (Fig. 2b, Sec. 5.1).  Per element the arithmetic is that of the per-tensor kernel with
// s = s[k]:
//     t = x * fl32(1/s[k]);  r = rint(t);  c = clamp(r, -Qn, Qp);  y = narrow(c * s[k])          (Eq. 1, Sec. 4.2)
//     m = (c == r);  dx = m ? g : 0                                                               (Eq. 4)
//     ds[k] = sum over the T rows of  g * (m ? r - t : c)                                         (chain rule)
// A thread owns 8 adjacent channels (one 128-bit vector per row) and walks down the rows of its row group, so its
// factors, their reciprocals and its 8 partial sums (double) stay in registers; a block covers 2048 adjacent
// channels, i.e. 4 KB contiguous per row.  Each (row group, channel) partial goes to the workspace as fp32; a second
// small kernel adds the row groups of every channel in row-group order in double.  Both orders are fixed by the
// launch shape: the gradients are bit-identical from run to run.
// HBM-bound: 8 algorithmic bytes per element fused (4 forward only, 6 backward only); the partials add
// 2 * row_groups * 4 bytes per channel.
#include "common.cuh"

namespace sasq {

int* per_channel_status_ptr();      // the fake-quant status word (fakequant.cu)

namespace {

#ifndef SASQ_PC_UNROLL
#define SASQ_PC_UNROLL 4
#endif
#ifndef SASQ_PC_BLOCKS_PER_SM
#define SASQ_PC_BLOCKS_PER_SM 2
#endif
constexpr int kPcThreads = 256;
constexpr int kPcUnroll = SASQ_PC_UNROLL;                 // rows in flight per thread (twice as many without a backward part)
constexpr int kPcBlocksPerSM = SASQ_PC_BLOCKS_PER_SM;
constexpr int kPcMaxRowGroups = 148 * 4;                  // sizes the workspace

struct PcParams {
    const uint4* x;
    const uint4* g;
    uint4* y;
    uint4* dx;
    const float* scales;    // [K]
    float* partials;        // [row_groups][K]
    long long T;
    int K;
    int vec_per_row;        // K / 8
    float qn, qp;
    int* status;
};

__device__ __forceinline__ uint4 pc_load(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void pc_store(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <bool BF, bool FWD, bool BWD>
__global__ void __launch_bounds__(kPcThreads, kPcBlocksPerSM) fakequant_pc_kernel(const __grid_constant__ PcParams p) {
    pdl_launch_dependents();
    pdl_wait();
    const int cv = blockIdx.x * blockDim.x + threadIdx.x;        // which 8-channel vector of a row
    if (cv >= p.vec_per_row) return;
    const int rg = blockIdx.y, n_rg = gridDim.y;
    const float qn = p.qn, qp = p.qp;

    float s[8], inv[8];
    {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p.scales) + 2 * cv);
        const float4 b = __ldg(reinterpret_cast<const float4*>(p.scales) + 2 * cv + 1);
        s[0] = a.x; s[1] = a.y; s[2] = a.z; s[3] = a.w; s[4] = b.x; s[5] = b.y; s[6] = b.z; s[7] = b.w;
        bool bad = false;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            inv[j] = __fdiv_rn(1.0f, s[j]);
            bad = bad || scale_is_bad(s[j]);
        }
        if (rg == 0 && bad) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
    }
    double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
    constexpr int UNROLL = BWD ? kPcUnroll : 2 * kPcUnroll;

    for (long long r0 = rg; r0 < p.T; r0 += (long long)n_rg * UNROLL) {
        uint4 xv[UNROLL], gv[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long r = r0 + (long long)u * n_rg;
            if (r < p.T) {
                xv[u] = pc_load(p.x + r * p.vec_per_row + cv);
                if constexpr (BWD) gv[u] = pc_load(p.g + r * p.vec_per_row + cv);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long r = r0 + (long long)u * n_rg;
            if (r < p.T) {
                const uint32_t xw[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
                uint32_t gw[4] = {0u, 0u, 0u, 0u};
                if constexpr (BWD) { gw[0] = gv[u].x; gw[1] = gv[u].y; gw[2] = gv[u].z; gw[3] = gv[u].w; }
                uint32_t yo[4], dxo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 xf = widen2<BF>(xw[q]);
                    const float t0 = __fmul_rn(xf.x, inv[2 * q]);
                    const float t1 = __fmul_rn(xf.y, inv[2 * q + 1]);
                    const float r_0 = rintf(t0), r_1 = rintf(t1);
                    const float c0 = fminf(fmaxf(r_0, -qn), qp);
                    const float c1 = fminf(fmaxf(r_1, -qn), qp);
                    if constexpr (FWD) yo[q] = narrow2<BF>(__fmul_rn(c0, s[2 * q]), __fmul_rn(c1, s[2 * q + 1]));
                    if constexpr (BWD) {
                        const float2 gf = widen2<BF>(gw[q]);
                        const bool in0 = (c0 == r_0), in1 = (c1 == r_1);      // false for NaN as well
                        dxo[q] = (in0 ? (gw[q] & 0x0000FFFFu) : 0u) | (in1 ? (gw[q] & 0xFFFF0000u) : 0u);
                        acc[2 * q] += (double)__fmul_rn(gf.x, in0 ? __fsub_rn(r_0, t0) : c0);
                        acc[2 * q + 1] += (double)__fmul_rn(gf.y, in1 ? __fsub_rn(r_1, t1) : c1);
                    }
                }
                if constexpr (FWD) pc_store(p.y + r * p.vec_per_row + cv, make_uint4(yo[0], yo[1], yo[2], yo[3]));
                if constexpr (BWD) pc_store(p.dx + r * p.vec_per_row + cv, make_uint4(dxo[0], dxo[1], dxo[2], dxo[3]));
            }
        }
    }
    if constexpr (BWD) {
        float4* out = reinterpret_cast<float4*>(p.partials + (size_t)rg * p.K) + 2 * cv;
        out[0] = make_float4((float)acc[0], (float)acc[1], (float)acc[2], (float)acc[3]);
        out[1] = make_float4((float)acc[4], (float)acc[5], (float)acc[6], (float)acc[7]);
    }
}

// Second stage: 64 channels per block, four threads per channel.  Thread (part, channel) adds a contiguous quarter
// of the row groups in row-group order (16 loads in flight), then the four quarters are added in order: fixed by the
// launch shape, double accumulation throughout.
__global__ void __launch_bounds__(kPcThreads) fakequant_pc_combine_kernel(const float* __restrict__ partials,
                                                                          float* __restrict__ grad_scales, int K,
                                                                          int row_groups, int accumulate) {
    __shared__ double quarter[4][64];
    pdl_launch_dependents();
    pdl_wait();
    const int ch = threadIdx.x & 63, part = threadIdx.x >> 6;
    const int k = blockIdx.x * 64 + ch;
    const int rg_begin = (part * row_groups) / 4, rg_end = ((part + 1) * row_groups) / 4;
    double tot = 0.0;
    if (k < K) {
        for (int rg0 = rg_begin; rg0 < rg_end; rg0 += 16) {
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = (rg0 + u < rg_end) ? __ldcg(partials + (size_t)(rg0 + u) * K + k) : 0.0f;
#pragma unroll
            for (int u = 0; u < 16; ++u) tot += (double)v[u];
        }
    }
    quarter[part][ch] = tot;
    __syncthreads();
    if (part == 0 && k < K) {
        const double sum = ((quarter[0][ch] + quarter[1][ch]) + quarter[2][ch]) + quarter[3][ch];
        const float prev = accumulate ? grad_scales[k] : 0.0f;
        grad_scales[k] = prev + (float)sum;
    }
}

// threads per block such that the blocks of a row are equally full: a row of K / 8 vectors is cut into the fewest
// blocks of at most 256 threads, then those blocks are made equally wide (K = 11008: 6 blocks of 232, not 5 x 256 + 96)
int pc_block_threads(int K) {
    const int vec = K / 8;
    const int col_blocks = (vec + kPcThreads - 1) / kPcThreads;
    return ((vec + col_blocks - 1) / col_blocks + 7) & ~7;      // whole 128-byte lines per block and row
}

int pc_row_groups(long long T, int K, int sm_count) {
    const int col_blocks = (K / 8 + kPcThreads - 1) / kPcThreads;
    // as many row groups as keep the whole grid resident at once (a few blocks too many would run as a second wave)
    long long rg = ((long long)kPcBlocksPerSM * sm_count) / col_blocks;
    if (rg > kPcMaxRowGroups) rg = kPcMaxRowGroups;
    if (rg > T) rg = T;
    if (rg < 1) rg = 1;
    return (int)rg;
}

template <bool BF, bool FWD, bool BWD>
cudaError_t pc_launch(const PcParams& p, dim3 grid, cudaStream_t st) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3((unsigned)pc_block_threads(p.K), 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fakequant_pc_kernel<BF, FWD, BWD>, p);
}

template <bool BF>
cudaError_t pc_launch_mode(bool fwd, bool bwd, const PcParams& p, dim3 grid, cudaStream_t st) {
    if (fwd && bwd) return pc_launch<BF, true, true>(p, grid, st);
    if (fwd) return pc_launch<BF, true, false>(p, grid, st);
    return pc_launch<BF, false, true>(p, grid, st);
}

}  // namespace
}  // namespace sasq

extern "C" {

size_t sasq_fakequant_per_channel_workspace(int64_t T, int64_t K) {
    (void)T;
    if (K <= 0) return 0;
    return (size_t)sasq::kPcMaxRowGroups * (size_t)K * sizeof(float);
}

int sasq_fakequant_fwd_bwd_per_channel(const void* x, const void* grad_y, void* y, void* grad_x,
                                       float* grad_scales_dev, int accumulate, int64_t T, int64_t K, int dt,
                                       const float* scales_dev, int bits, void* workspace, size_t ws_bytes,
                                       void* stream) {
    using namespace sasq;
    if (T < 0 || K <= 0 || scales_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8 || (dt != SASQ_F16 && dt != SASQ_BF16)) return SASQ_ERR_INVALID_ARG;
    if (K % 8 != 0 || K > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0) {       // nothing to quantize: the gradients of an empty sum are zero
        if (grad_scales_dev != nullptr && !accumulate &&
            cudaMemsetAsync(grad_scales_dev, 0, sizeof(float) * (size_t)K, st) != cudaSuccess)
            return SASQ_ERR_CUDA;
        return SASQ_OK;
    }
    const bool fwd = y != nullptr, bwd = grad_y != nullptr;
    if (!fwd && !bwd) return SASQ_ERR_INVALID_ARG;
    if (bwd != (grad_x != nullptr)) return SASQ_ERR_INVALID_ARG;
    if (bwd && grad_scales_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (x == nullptr) return SASQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(grad_y) || !aligned16(y) || !aligned16(grad_x) || !aligned16(scales_dev))
        return SASQ_ERR_INVALID_ARG;
    if (bwd && (workspace == nullptr || !aligned16(workspace) ||
                ws_bytes < sasq_fakequant_per_channel_workspace(T, K)))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = per_channel_status_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;

    PcParams p{};
    p.x = static_cast<const uint4*>(x);
    p.g = static_cast<const uint4*>(grad_y);
    p.y = static_cast<uint4*>(y);
    p.dx = static_cast<uint4*>(grad_x);
    p.scales = scales_dev;
    p.partials = static_cast<float*>(workspace);
    p.T = T;
    p.K = (int)K;
    p.vec_per_row = (int)(K / 8);
    p.qn = (float)(1 << (bits - 1));
    p.qp = (float)((1 << (bits - 1)) - 1);
    p.status = status;
    const int row_groups = pc_row_groups(T, (int)K, sm_count);
    const dim3 grid((unsigned)((p.vec_per_row + kPcThreads - 1) / kPcThreads), (unsigned)row_groups, 1);
    const cudaError_t e = (dt == SASQ_BF16) ? pc_launch_mode<true>(fwd, bwd, p, grid, st)
                                            : pc_launch_mode<false>(fwd, bwd, p, grid, st);
    if (e != cudaSuccess) return SASQ_ERR_CUDA;
    if (bwd) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)((K + 63) / 64), 1, 1);
        cfg.blockDim = dim3(kPcThreads, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1] = {pdl_attribute()};
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, fakequant_pc_combine_kernel, static_cast<const float*>(workspace),
                               grad_scales_dev, (int)K, row_groups, accumulate ? 1 : 0) != cudaSuccess)
            return SASQ_ERR_CUDA;
    }
    return SASQ_OK;
}

}  // extern "C"
