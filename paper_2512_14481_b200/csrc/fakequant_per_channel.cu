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

constexpr int kPcMaxTensors = 16;       // tensors of one launch

struct PcTensor {
    const uint4* x;
    const uint4* g;
    uint4* y;
    uint4* dx;
    const float* scales;    // [K]
    float* grad_scales;     // [K]
    float* partials;        // [row_groups][K]
    long long T;
    int K;
    int vec_per_row;        // K / 8
    int col_threads;        // threads of a block that work (equal-width column blocks)
    int col_blocks;
    int row_groups;
    int first_block;        // blocks [first_block, first_block + col_blocks * row_groups) belong to this tensor
    int first_combine_block;
};

struct PcParams {
    PcTensor t[kPcMaxTensors];
    int n;
    float qn, qp;
    int accumulate;
    int* status;
};

__device__ __forceinline__ uint4 pc_load(const uint4* p) {
    uint4 v;
    // coherent path: y may alias x and grad_x may alias grad_y (in-place calls)
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void pc_store(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// All tensors of the launch run side by side: every tensor owns a contiguous range of blocks, sized by its share
// of the elements, arranged as (row group, column block).
template <bool BF, bool FWD, bool BWD>
__global__ void __launch_bounds__(kPcThreads, kPcBlocksPerSM) fakequant_pc_kernel(const __grid_constant__ PcParams p) {
    pdl_launch_dependents();
    pdl_wait();
    int ti = 0;
    while (ti + 1 < p.n && (int)blockIdx.x >= p.t[ti + 1].first_block) ++ti;
    const PcTensor& d = p.t[ti];
    const int local = (int)blockIdx.x - d.first_block;
    const int rg = local / d.col_blocks, n_rg = d.row_groups;
    const int cv = (local - rg * d.col_blocks) * d.col_threads + (int)threadIdx.x;   // which 8-channel vector of a row
    if ((int)threadIdx.x >= d.col_threads || cv >= d.vec_per_row || rg >= n_rg) return;
    const float qn = p.qn, qp = p.qp;
    const long long T = d.T;
    const int vec_per_row = d.vec_per_row;

    float s[8], inv[8];
    {
        const float4 a = __ldg(reinterpret_cast<const float4*>(d.scales) + 2 * cv);
        const float4 b = __ldg(reinterpret_cast<const float4*>(d.scales) + 2 * cv + 1);
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

    for (long long r0 = rg; r0 < T; r0 += (long long)n_rg * UNROLL) {
        uint4 xv[UNROLL], gv[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long r = r0 + (long long)u * n_rg;
            if (r < T) {
                xv[u] = pc_load(d.x + r * vec_per_row + cv);
                if constexpr (BWD) gv[u] = pc_load(d.g + r * vec_per_row + cv);
            }
        }
        // the products of the rows in flight are first added in fp32, in a fixed tree, and reach the double sums
        // once per trip: a float -> double conversion and a double add per ELEMENT kept the conversion pipe busier
        // than the memory system (the per-tensor kernel likewise adds a vector's 8 products in fp32 first)
        float prod[UNROLL][8];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long r = r0 + (long long)u * n_rg;
#pragma unroll
            for (int j = 0; j < 8; ++j) prod[u][j] = 0.0f;
            if (r < T) {
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
                        prod[u][2 * q] = __fmul_rn(gf.x, in0 ? __fsub_rn(r_0, t0) : c0);
                        prod[u][2 * q + 1] = __fmul_rn(gf.y, in1 ? __fsub_rn(r_1, t1) : c1);
                    }
                }
                if constexpr (FWD) pc_store(d.y + r * vec_per_row + cv, make_uint4(yo[0], yo[1], yo[2], yo[3]));
                if constexpr (BWD) pc_store(d.dx + r * vec_per_row + cv, make_uint4(dxo[0], dxo[1], dxo[2], dxo[3]));
            }
        }
        if constexpr (BWD) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float sum = 0.0f;
                if constexpr (UNROLL == 4) {
                    sum = __fadd_rn(__fadd_rn(prod[0][j], prod[1][j]), __fadd_rn(prod[2][j], prod[3][j]));
                } else {
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) sum = __fadd_rn(sum, prod[u][j]);
                }
                acc[j] += (double)sum;
            }
        }
    }
    if constexpr (BWD) {
        float4* out = reinterpret_cast<float4*>(d.partials + (size_t)rg * d.K) + 2 * cv;
        out[0] = make_float4((float)acc[0], (float)acc[1], (float)acc[2], (float)acc[3]);
        out[1] = make_float4((float)acc[4], (float)acc[5], (float)acc[6], (float)acc[7]);
    }
}

// Second stage: 64 channels per block, four threads per channel.  Thread (part, channel) adds a contiguous quarter
// of the row groups in row-group order (16 loads in flight), then the four quarters are added in order: fixed by the
// launch shape, double accumulation throughout.
__global__ void __launch_bounds__(kPcThreads) fakequant_pc_combine_kernel(const __grid_constant__ PcParams p) {
    __shared__ double quarter[4][64];
    pdl_launch_dependents();
    pdl_wait();
    int ti = 0;
    while (ti + 1 < p.n && (int)blockIdx.x >= p.t[ti + 1].first_combine_block) ++ti;
    const PcTensor& d = p.t[ti];
    const int ch = threadIdx.x & 63, part = threadIdx.x >> 6;
    const int k = ((int)blockIdx.x - d.first_combine_block) * 64 + ch;
    const int K = d.K, row_groups = d.row_groups;
    const int rg_begin = (part * row_groups) / 4, rg_end = ((part + 1) * row_groups) / 4;
    double tot = 0.0;
    if (k < K) {
        for (int rg0 = rg_begin; rg0 < rg_end; rg0 += 16) {
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = (rg0 + u < rg_end) ? __ldcg(d.partials + (size_t)(rg0 + u) * K + k) : 0.0f;
#pragma unroll
            for (int u = 0; u < 16; ++u) tot += (double)v[u];
        }
    }
    quarter[part][ch] = tot;
    __syncthreads();
    if (part == 0 && k < K) {
        const double sum = ((quarter[0][ch] + quarter[1][ch]) + quarter[2][ch]) + quarter[3][ch];
        const float prev = p.accumulate ? d.grad_scales[k] : 0.0f;
        d.grad_scales[k] = prev + (float)sum;
    }
}

// threads of a block that work, such that the blocks of a row are equally full: a row of K / 8 vectors is cut into
// the fewest blocks of at most 256 threads, then those blocks are made equally wide and a multiple of 8 threads
// (whole 128-byte lines per block and row; K = 11008: 6 blocks of 232, not 5 x 256 + 96)
int pc_block_threads(int K) {
    const int vec = K / 8;
    const int col_blocks = (vec + kPcThreads - 1) / kPcThreads;
    return ((vec + col_blocks - 1) / col_blocks + 7) & ~7;
}

template <bool BF, bool FWD, bool BWD>
cudaError_t pc_launch(const PcParams& p, int grid, cudaStream_t st) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kPcThreads, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fakequant_pc_kernel<BF, FWD, BWD>, p);
}

template <bool BF>
cudaError_t pc_launch_mode(bool fwd, bool bwd, const PcParams& p, int grid, cudaStream_t st) {
    if (fwd && bwd) return pc_launch<BF, true, true>(p, grid, st);
    if (fwd) return pc_launch<BF, true, false>(p, grid, st);
    return pc_launch<BF, false, true>(p, grid, st);
}

int pc_run(const sasq_pcdesc_t* descs, int n, int accumulate, int dt, int bits, void* workspace, size_t ws_bytes,
           void* stream) {
    if (n < 0 || n > kPcMaxTensors || (n > 0 && descs == nullptr)) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8 || (dt != SASQ_F16 && dt != SASQ_BF16)) return SASQ_ERR_INVALID_ARG;
    if (n == 0) return SASQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the first descriptor that has rows says which passes run; tensors without rows may leave the data pointers NULL
    int lead = 0;
    while (lead + 1 < n && descs[lead].T == 0) ++lead;
    const bool fwd = descs[lead].y != nullptr, bwd = descs[lead].grad_y != nullptr;
    long long total_elems = 0, total_k = 0;
    int live = 0;
    for (int i = 0; i < n; ++i) {
        const sasq_pcdesc_t& d = descs[i];
        if (d.T < 0 || d.K <= 0 || d.scales == nullptr || d.reserved != 0) return SASQ_ERR_INVALID_ARG;
        if (d.K % 8 != 0 || d.K > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
        if (d.T > 0) {
            if ((d.y != nullptr) != fwd || (d.grad_y != nullptr) != bwd) return SASQ_ERR_INVALID_ARG;
            if ((d.grad_y != nullptr) != (d.grad_x != nullptr) || d.x == nullptr) return SASQ_ERR_INVALID_ARG;
        }
        if (bwd && d.T > 0 && d.grad_scales == nullptr) return SASQ_ERR_INVALID_ARG;
        if (!aligned16(d.x) || !aligned16(d.grad_y) || !aligned16(d.y) || !aligned16(d.grad_x) || !aligned16(d.scales))
            return SASQ_ERR_INVALID_ARG;
        if (d.T > 0) { total_elems += d.T * d.K; total_k += d.K; ++live; }
    }
    // tensors without rows: the gradients of an empty sum are zero
    for (int i = 0; i < n; ++i)
        if (descs[i].T == 0 && descs[i].grad_scales != nullptr && !accumulate &&
            cudaMemsetAsync(descs[i].grad_scales, 0, sizeof(float) * (size_t)descs[i].K, st) != cudaSuccess)
            return SASQ_ERR_CUDA;
    if (live == 0) return SASQ_OK;
    if (!fwd && !bwd) return SASQ_ERR_INVALID_ARG;
    if (bwd && (workspace == nullptr || !aligned16(workspace) ||
                ws_bytes < (size_t)kPcMaxRowGroups * (size_t)total_k * sizeof(float)))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = per_channel_status_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;

    PcParams p{};
    p.qn = (float)(1 << (bits - 1));
    p.qp = (float)((1 << (bits - 1)) - 1);
    p.accumulate = accumulate ? 1 : 0;
    p.status = status;
    // Every tensor gets a share of the resident blocks in proportion to its elements (at least one row group), as
    // many row groups as fit that share; the whole grid stays resident at once.
    const long long budget = (long long)kPcBlocksPerSM * sm_count;
    int block = 0, cblock = 0;
    float* part = static_cast<float*>(workspace);
    for (int i = 0; i < n; ++i) {
        const sasq_pcdesc_t& d = descs[i];
        if (d.T == 0) continue;
        PcTensor& t = p.t[p.n++];
        t.x = static_cast<const uint4*>(d.x);
        t.g = static_cast<const uint4*>(d.grad_y);
        t.y = static_cast<uint4*>(d.y);
        t.dx = static_cast<uint4*>(d.grad_x);
        t.scales = d.scales;
        t.grad_scales = d.grad_scales;
        t.T = d.T;
        t.K = (int)d.K;
        t.vec_per_row = (int)(d.K / 8);
        t.col_threads = pc_block_threads((int)d.K);
        t.col_blocks = (t.vec_per_row + kPcThreads - 1) / kPcThreads;
        long long share = (long long)((double)budget * (double)(d.T * d.K) / (double)total_elems);
        long long rg = share / t.col_blocks;
        if (rg > kPcMaxRowGroups) rg = kPcMaxRowGroups;
        if (rg > d.T) rg = d.T;
        if (rg < 1) rg = 1;
        t.row_groups = (int)rg;
        t.first_block = block;
        t.first_combine_block = cblock;
        t.partials = part;
        block += t.col_blocks * t.row_groups;
        cblock += (int)((d.K + 63) / 64);
        part += (size_t)t.row_groups * (size_t)d.K;
    }
    const cudaError_t e = (dt == SASQ_BF16) ? pc_launch_mode<true>(fwd, bwd, p, block, st)
                                            : pc_launch_mode<false>(fwd, bwd, p, block, st);
    if (e != cudaSuccess) return SASQ_ERR_CUDA;
    if (bwd) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)cblock, 1, 1);
        cfg.blockDim = dim3(kPcThreads, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1] = {pdl_attribute()};
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, fakequant_pc_combine_kernel, p) != cudaSuccess) return SASQ_ERR_CUDA;
    }
    return SASQ_OK;
}

}  // namespace
}  // namespace sasq

extern "C" {

size_t sasq_fakequant_per_channel_workspace(int64_t T, int64_t K) {
    (void)T;
    if (K <= 0) return 0;
    return (size_t)sasq::kPcMaxRowGroups * (size_t)K * sizeof(float);
}

size_t sasq_fakequant_per_channel_multi_workspace(int64_t total_K) {
    if (total_K <= 0) return 0;
    return (size_t)sasq::kPcMaxRowGroups * (size_t)total_K * sizeof(float);
}

int sasq_fakequant_fwd_bwd_per_channel(const void* x, const void* grad_y, void* y, void* grad_x,
                                       float* grad_scales_dev, int accumulate, int64_t T, int64_t K, int dt,
                                       const float* scales_dev, int bits, void* workspace, size_t ws_bytes,
                                       void* stream) {
    sasq_pcdesc_t d{};
    d.x = x;
    d.grad_y = grad_y;
    d.y = y;
    d.grad_x = grad_x;
    d.scales = scales_dev;
    d.grad_scales = grad_scales_dev;
    d.T = T;
    d.K = K;
    if (T > 0 && y == nullptr && grad_y == nullptr) return SASQ_ERR_INVALID_ARG;
    return sasq::pc_run(&d, 1, accumulate, dt, bits, workspace, ws_bytes, stream);
}

int sasq_fakequant_fwd_bwd_per_channel_multi(const sasq_pcdesc_t* descs_host, int n_tensors, int accumulate, int dt,
                                             int bits, void* workspace, size_t ws_bytes, void* stream) {
    return sasq::pc_run(descs_host, n_tensors, accumulate, dt, bits, workspace, ws_bytes, stream);
}

}  // extern "C"
