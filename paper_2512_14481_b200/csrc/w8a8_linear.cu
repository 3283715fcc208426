// Static W8A8 linear for sm_100a (Eq. 1 with the fixed learned factor, Eq. 2):
//   X_int = int8(clamp(rint(x * fl32(1/s_x)), -Qn, Qp))
//   acc   = X_int * W_int^T                      int8 x int8 -> int32 on tcgen05 tensor cores, accumulators in TMEM
//   y     = narrow(fl32(acc) * fl32(s_x * s_w[n]) (+ bias[n]))
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0      TMA producer: W tiles (and pre-quantized A tiles) -> 128-byte-swizzled shared memory
//   warp 1      MMA issuer: tcgen05.mma.kind::i8, 128 x 256 x 32 per instruction, TMEM double-buffered
//   warps 2..5  epilogue: tcgen05.ld -> dequant -> 16-bit stores, overlapped with the next tile's mainloop
// Every wait on an mbarrier is bounded; a wait that gives up raises SASQ_ERR_TIMEOUT
// in the sticky status word and all roles fall through to the teardown.
#include "common.cuh"
#include "tcgen05.cuh"

namespace sasq {

SASQ_DEFINE_STATUS_WORD(g_linear_status)
int linear_status_read_and_clear(cudaStream_t st) { return g_linear_status_read_and_clear(st); }

namespace {

constexpr int BM = 128;            // rows of x per tile (UMMA M)
constexpr int BN = 256;            // output channels per tile (UMMA N)
constexpr int BK = 128;            // int8 elements (= bytes) of K per pipeline stage: one 128-byte swizzle row
constexpr int UMMA_K = 32;         // K per tcgen05.mma.kind::i8
constexpr int STAGES = 4;
constexpr int ACC_BUFS = 2;        // TMEM accumulator buffers (2 x 256 columns = all 512)
constexpr int A_STAGE_BYTES = BM * BK;
constexpr int B_STAGE_BYTES = BN * BK;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int NUM_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr uint32_t TMEM_COLS = 512;
constexpr long long kWaitLimit = 1LL << 31;   // clock cycles a single wait may take (about a second)

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
    const float* x_scale;
    const void* bias;
    void* y;
    int32_t* acc_out;
    int T, N, K;
    int m_blocks, n_blocks, k_blocks;
    int* status;
    long long wait_limit;
};

// Bounded wait: false (and the abort flag raised) if the phase did not complete in time
// or another role already gave up.
__device__ __forceinline__ bool wait_bounded(uint64_t* bar, uint32_t parity, SharedTail* tail, const LinearParams& p) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int polls = 0;
    while (!ptx::mbar_try_wait(bar, parity)) {
        if ((++polls & 63) == 0) {
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

template <bool BF>
__global__ void __launch_bounds__(NUM_THREADS, 1)
w8a8_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                 const __grid_constant__ LinearParams p) {
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
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int m_blk = tile % p.m_blocks, n_blk = tile / p.m_blocks;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                if (lane == 0) {
                    ok = wait_bounded(&tail->empty[stage], phase ^ 1u, tail, p);
                    if (ok) {
                        uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
                        uint8_t* b_dst = a_dst + A_STAGE_BYTES;
                        ptx::mbar_arrive_expect_tx(&tail->full[stage], STAGE_BYTES);
                        ptx::tma_load_2d(a_dst, &tmap_a, &tail->full[stage], kb * BK, m_blk * BM);
                        ptx::tma_load_2d(b_dst, &tmap_w, &tail->full[stage], kb * BK, n_blk * BN);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        // teardown: copies still in flight must land before the CTA's shared memory goes away.
        // Every armed full barrier either was consumed already (wait returns at once) or completes here.
        if (lane == 0 && !ok) {
            for (int s = 0; s < STAGES; ++s) {
                const long long t0 = clock64();
                // the phase armed last for stage s: stages before `stage` are in `phase`, the others in phase^1
                const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
                while (!ptx::mbar_try_wait(&tail->full[s], par)) {
                    if (clock64() - t0 > (1LL << 24)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            if (lane == 0) ok = wait_bounded(&tail->tmem_empty[buf], acc_phase ^ 1u, tail, p);
            ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                if (lane == 0) {
                    ok = wait_bounded(&tail->full[stage], phase, tail, p);
                    if (ok) {
                        ptx::tc_fence_after_sync();
                        const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)stage * STAGE_BYTES);
                        const uint32_t b_addr = a_addr + A_STAGE_BYTES;
                        const uint64_t a_desc = ptx::smem_desc_k_major_sw128(a_addr);
                        const uint64_t b_desc = ptx::smem_desc_k_major_sw128(b_addr);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            // advance both operands by 32 bytes of K inside the swizzled row
                            ptx::mma_i8_ss(d_tmem, a_desc + (uint64_t)(k * (UMMA_K >> 4)),
                                           b_desc + (uint64_t)(k * (UMMA_K >> 4)), idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                        ptx::mma_commit(&tail->empty[stage]);          // stage reusable once these MMAs are done
                        if (kb == p.k_blocks - 1) ptx::mma_commit(&tail->tmem_full[buf]);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue (warps 2..5) ----------------
        const int quad = warp & 3;                      // TMEM lane quadrant this warp may read
        const int et = threadIdx.x - 64;                // 0..127
        const float sx = __ldg(p.x_scale);
        if (blockIdx.x == 0 && et == 0 && scale_is_bad(sx)) atomicMax(p.status, (int)SASQ_ERR_BAD_SCALE);
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
                tail->scale[j] = (n < p.N) ? __fmul_rn(sx, __ldg(p.w_scale + n)) : 0.0f;
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
                            float f0 = __fmul_rn(__int2float_rn((int)v[j + 2 * q]), tail->scale[c + j + 2 * q]);
                            float f1 = __fmul_rn(__int2float_rn((int)v[j + 2 * q + 1]), tail->scale[c + j + 2 * q + 1]);
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

// Eq. 1 with the fixed factor, written once to int8 (operand A of the GEMM).
// 16 elements per thread: two 128-bit loads, one 128-bit store.
template <bool BF>
__global__ void __launch_bounds__(256) quantize_act_kernel(const uint4* __restrict__ x, uint4* __restrict__ out,
                                                           long long n16, const float* __restrict__ x_scale,
                                                           float qn, float qp) {
    const float inv = __fdiv_rn(1.0f, __ldg(x_scale));
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) {
        const uint4 a = x[2 * i], b = x[2 * i + 1];
        const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t packed = 0;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float2 f = widen2<BF>(w[2 * q + h]);
                const int c0 = __float2int_rn(fminf(fmaxf(__fmul_rn(f.x, inv), -qn), qp));
                const int c1 = __float2int_rn(fminf(fmaxf(__fmul_rn(f.y, inv), -qn), qp));
                packed |= ((uint32_t)(c0 & 0xFF) | ((uint32_t)(c1 & 0xFF) << 8)) << (16 * h);
            }
            o[q] = packed;
        }
        out[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
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

// int8 [rows, K] row-major -> tiles of box_rows x 128 bytes, 128-byte swizzle, zero fill outside
bool make_tmap(CUtensorMap* m, const void* base, long long rows, long long K, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int* status_word_ptr() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_linear_status) != cudaSuccess) return nullptr;
    return p;
}

}  // namespace
}  // namespace sasq

extern "C" {

size_t sasq_static_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K) {
    (void)N;
    if (T <= 0 || K <= 0) return 0;
    // int8 copy of the activations, padded to whole 16-element groups
    return (size_t)(((T * K + 15) / 16) * 16 + 256);
}

int sasq_static_w8a8_linear(const void* x, const int8_t* w, const float* w_scale, const float* x_scale_dev,
                            const void* bias, void* y, int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt,
                            int bits, void* workspace, size_t ws_bytes, void* stream) {
    using namespace sasq;
    if (T < 0 || N <= 0 || K <= 0) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (w == nullptr || w_scale == nullptr || x_scale_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (T > 0 && (x == nullptr || y == nullptr)) return SASQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(acc_out) ||
        (reinterpret_cast<uintptr_t>(w_scale) & 3u) || (reinterpret_cast<uintptr_t>(bias) & 1u))
        return SASQ_ERR_INVALID_ARG;
    if (K % 16 != 0 || N % 8 != 0 || K > 131072 || T > (1 << 24) || N > (1 << 24)) return SASQ_ERR_UNSUPPORTED;
    if (T == 0) return SASQ_OK;
    if (workspace == nullptr || !aligned16(workspace) || ws_bytes < sasq_static_w8a8_linear_workspace(T, N, K))
        return SASQ_ERR_WORKSPACE;
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // 1. Eq. 1 with the fixed factor -> int8 activations in the workspace
    uint8_t* a_int8 = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(workspace) + 127) & ~uintptr_t(127));
    const long long n16 = (T * K) / 16;     // K % 16 == 0
    const float qn = (float)(1 << (bits - 1)), qp = (float)((1 << (bits - 1)) - 1);
    {
        long long blocks = (n16 + 255) / 256;
        if (blocks > (long long)sm_count * 8) blocks = (long long)sm_count * 8;
        if (dt == SASQ_BF16)
            quantize_act_kernel<true><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                                   reinterpret_cast<uint4*>(a_int8), n16,
                                                                   x_scale_dev, qn, qp);
        else
            quantize_act_kernel<false><<<(int)blocks, 256, 0, st>>>(static_cast<const uint4*>(x),
                                                                    reinterpret_cast<uint4*>(a_int8), n16,
                                                                    x_scale_dev, qn, qp);
        if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    }

    // 2. TMA-fed tcgen05 GEMM with the dequant epilogue
    CUtensorMap tmap_a, tmap_w;
    if (!make_tmap(&tmap_a, a_int8, T, K, BM) || !make_tmap(&tmap_w, w, N, K, BN)) return SASQ_ERR_CUDA;
    LinearParams p{};
    p.w_scale = w_scale;
    p.x_scale = x_scale_dev;
    p.bias = bias;
    p.y = y;
    p.acc_out = acc_out;
    p.T = (int)T; p.N = (int)N; p.K = (int)K;
    p.m_blocks = (int)((T + BM - 1) / BM);
    p.n_blocks = (int)((N + BN - 1) / BN);
    p.k_blocks = (int)((K + BK - 1) / BK);
    p.status = status;
    p.wait_limit = kWaitLimit;
    const long long tiles = (long long)p.m_blocks * p.n_blocks;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    cudaError_t e;
    if (dt == SASQ_BF16) {
        e = cudaFuncSetAttribute(w8a8_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return SASQ_ERR_CUDA;
        w8a8_gemm_kernel<true><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
    } else {
        e = cudaFuncSetAttribute(w8a8_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e != cudaSuccess) return SASQ_ERR_CUDA;
        w8a8_gemm_kernel<false><<<grid, NUM_THREADS, kSmemBytes, st>>>(tmap_a, tmap_w, p);
    }
    if (cudaGetLastError() != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

}  // extern "C"
