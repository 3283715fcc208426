// C-ABI entry points of the fake-quant forward / backward / fused path.
#include <atomic>

#include "fakequant_kernels.cuh"

namespace sasq {

SASQ_DEFINE_STATUS_WORD(g_fakequant_status)

int fakequant_status_read_and_clear(cudaStream_t st) { return g_fakequant_status_read_and_clear(st); }

// device address of the fake-quant status word on the current device (shared with the per-channel kernels)
int* per_channel_status_ptr() {
    static int* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (cache[dev] == nullptr) {
        int* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_fakequant_status) != cudaSuccess) return nullptr;
        cache[dev] = p;
    }
    return cache[dev];
}

namespace {

// launch shape of the streaming kernel
constexpr int kThreads = 256;
constexpr int kUnroll = 2;             // 128-bit vectors of x (and of g) in flight per thread
constexpr int kUnrollFwdOnly = 4;      // the forward alone loads half as much per vector: keep as many bytes in flight
constexpr int kBlocksPerSM = 4;
// streaming loads through the coherent path (hint 3): y may alias x and grad_x may alias grad_y, so the launch may
// store to the addresses it loads from, which rules out the non-coherent (.nc) form; measured at the same speed
#ifndef SASQ_FQ_LOAD_HINT
#define SASQ_FQ_LOAD_HINT 3
#endif
constexpr int kLoadHint = SASQ_FQ_LOAD_HINT;
constexpr int kStoreHint = 1;

int* status_word_ptr() {
    static int* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (cache[dev] == nullptr) {
        int* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_fakequant_status) != cudaSuccess) return nullptr;
        cache[dev] = p;
    }
    return cache[dev];
}

// Ticket counters of the second reduction stage.  They are zero when the library is loaded and every launch
// leaves the one it used at zero again.  Launches made directly draw them round-robin, so two of them share a counter
// only if more than kTicketSlots launches of this library were executing at the same time, which no GPU does.  A
// launch that is being captured into a CUDA graph keeps its counter's address for every replay, at times the library
// does not see: it gets a counter of its own from a second pool that is never handed out twice (kCaptureTickets
// captured launches per process), so a replay can overlap other launches of the library on other streams.
constexpr unsigned kTicketSlots = 256;
constexpr unsigned kCaptureTickets = 4096;
static __device__ unsigned g_tickets[kTicketSlots + kCaptureTickets];

// SASQ_OK and *ticket, or SASQ_ERR_UNSUPPORTED when a captured launch finds the capture pool used up
int next_ticket(cudaStream_t st, unsigned** ticket) {
    static unsigned* base[64] = {nullptr};
    static std::atomic<unsigned> next{0};
    static std::atomic<unsigned> capture_next{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SASQ_ERR_CUDA;
    if (base[dev] == nullptr) {
        unsigned* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_tickets) != cudaSuccess) return SASQ_ERR_CUDA;
        base[dev] = p;
    }
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &capturing) != cudaSuccess) return SASQ_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) {
        const unsigned at = capture_next.fetch_add(1u, std::memory_order_relaxed);
        if (at >= kCaptureTickets) return SASQ_ERR_UNSUPPORTED;
        *ticket = base[dev] + kTicketSlots + at;
        return SASQ_OK;
    }
    *ticket = base[dev] + (next.fetch_add(1u, std::memory_order_relaxed) % kTicketSlots);
    return SASQ_OK;
}

template <bool BF, bool FWD, bool BWD, int VARIANT = 0>
cudaError_t launch_stream(const QParams& p, int grid, cudaStream_t st) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fakequant_kernel<BF, FWD, BWD, kThreads, (BWD ? kUnroll : kUnrollFwdOnly), kBlocksPerSM, kLoadHint, kStoreHint, VARIANT>, p);
}

template <bool BF, int VARIANT = 0>
cudaError_t launch_mode(bool fwd, bool bwd, const QParams& p, int grid, cudaStream_t st) {
    if (fwd && bwd) return launch_stream<BF, true, true, VARIANT>(p, grid, st);
    if (fwd) return launch_stream<BF, true, false, VARIANT>(p, grid, st);
    return launch_stream<BF, false, true, VARIANT>(p, grid, st);
}

int grid_for(long long max_numel, int sm_count) {
    long long g = (long long)sm_count * kBlocksPerSM;
    const long long need = ((max_numel >> 3) + kThreads - 1) / kThreads;
    if (g > need) g = need;
    if (g > kMaxGrid) g = kMaxGrid;
    if (g < 1) g = 1;
    return (int)g;
}

template <bool BF>
cudaError_t launch_variant(int variant, bool fwd, bool bwd, const QParams& p, int grid, cudaStream_t st) {
    if (variant == SASQ_WITHOUT_ROUND) return launch_mode<BF, 1>(fwd, bwd, p, grid, st);
    if (variant == SASQ_WITHOUT_CLAMP) return launch_mode<BF, 2>(fwd, bwd, p, grid, st);
    return launch_mode<BF, 0>(fwd, bwd, p, grid, st);
}

int run_multi(const sasq_qdesc_t* descs, int n_tensors, const float* scales_dev, float* grad_scales_dev,
              int n_scales, int accumulate, int dt, int bits, void* workspace, size_t ws_bytes, void* stream,
              int variant = SASQ_FULL_OPERATOR) {
    if (variant != SASQ_FULL_OPERATOR && variant != SASQ_WITHOUT_ROUND && variant != SASQ_WITHOUT_CLAMP)
        return SASQ_ERR_INVALID_ARG;
    if (n_tensors < 0 || n_scales <= 0 || (n_tensors > 0 && descs == nullptr)) return SASQ_ERR_INVALID_ARG;
    if (scales_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (n_tensors == 0) return SASQ_OK;

    // the first descriptor that holds elements says which passes run; empty ones (numel == 0) may leave every
    // pointer NULL and are skipped by the kernel
    int lead = 0;
    while (lead + 1 < n_tensors && descs[lead].numel == 0) ++lead;
    const bool fwd = descs[lead].y != nullptr;
    const bool bwd = descs[lead].grad_y != nullptr;
    long long max_numel = 0;
    for (int i = 0; i < n_tensors; ++i) {
        const sasq_qdesc_t& d = descs[i];
        if (d.numel < 0 || d.reserved != 0) return SASQ_ERR_INVALID_ARG;
        if (d.scale_index < 0 || d.scale_index >= n_scales) return SASQ_ERR_INVALID_ARG;
        if (d.numel > 0 && ((d.y != nullptr) != fwd || (d.grad_y != nullptr) != bwd)) return SASQ_ERR_INVALID_ARG;
        if (d.numel > 0 && (d.grad_y != nullptr) != (d.grad_x != nullptr)) return SASQ_ERR_INVALID_ARG;
        if (d.numel > 0 && d.x == nullptr) return SASQ_ERR_INVALID_ARG;
        if (!aligned16(d.x) || !aligned16(d.y) || !aligned16(d.grad_y) || !aligned16(d.grad_x))
            return SASQ_ERR_INVALID_ARG;
        if (d.numel > max_numel) max_numel = d.numel;
    }
    if (!fwd && !bwd) return SASQ_ERR_INVALID_ARG;
    if (bwd) {
        if (grad_scales_dev == nullptr) return SASQ_ERR_INVALID_ARG;
        if (workspace == nullptr || !aligned16(workspace) ||
            ws_bytes < sasq_fakequant_multi_workspace(n_tensors))
            return SASQ_ERR_WORKSPACE;
    }
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = grid_for(max_numel, sm_count);
    // slots already written by an earlier chunk of this call are added to afterwards
    // (only possible when n_tensors > kMaxDescsPerLaunch)
    for (int base = 0; base < n_tensors; base += kMaxDescsPerLaunch) {
        const int n = (n_tensors - base < kMaxDescsPerLaunch) ? (n_tensors - base) : kMaxDescsPerLaunch;
        QParams p{};
        for (int i = 0; i < n; ++i) {
            const sasq_qdesc_t& d = descs[base + i];
            p.d[i].x = static_cast<const uint4*>(d.x);
            p.d[i].g = static_cast<const uint4*>(d.grad_y);
            p.d[i].y = static_cast<uint4*>(d.y);
            p.d[i].dx = static_cast<uint4*>(d.grad_x);
            p.d[i].numel = d.numel;
            p.d[i].scale_index = d.scale_index;
            bool seen_before = false;
            for (int k = 0; k < base && !seen_before; ++k) seen_before = (descs[k].scale_index == d.scale_index);
            if (accumulate || seen_before) p.accumulate_mask |= (1u << i);
        }
        p.n = n;
        p.scales = scales_dev;
        p.partials = static_cast<double*>(workspace) + (size_t)base * kMaxGrid;
        p.qn = (float)(1 << (bits - 1));
        p.qp = (float)((1 << (bits - 1)) - 1);
        p.status = status;
        p.grad_scales = grad_scales_dev;
        if (bwd) {
            const int ticket_rc = next_ticket(st, &p.ticket);
            if (ticket_rc != SASQ_OK) return ticket_rc;
        }
        cudaError_t e = (dt == SASQ_BF16) ? launch_variant<true>(variant, fwd, bwd, p, grid, st)
                                          : launch_variant<false>(variant, fwd, bwd, p, grid, st);
        if (e != cudaSuccess) return SASQ_ERR_CUDA;
    }
    return SASQ_OK;
}

int run_single(const void* x, const void* grad_y, void* y, void* grad_x, float* grad_scale_dev, int accumulate,
               int64_t numel, int dt, const float* scale_dev, int bits, void* workspace, size_t ws_bytes,
               void* stream, bool fwd, bool bwd, int variant = SASQ_FULL_OPERATOR) {
    if (numel < 0) return SASQ_ERR_INVALID_ARG;
    if (scale_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return SASQ_ERR_INVALID_ARG;
    if (dt != SASQ_F16 && dt != SASQ_BF16) return SASQ_ERR_INVALID_ARG;
    if (bwd && grad_scale_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (numel > 0) {
        if (x == nullptr || (fwd && y == nullptr) || (bwd && (grad_y == nullptr || grad_x == nullptr)))
            return SASQ_ERR_INVALID_ARG;
    }
    if (numel == 0) {
        if (bwd && !accumulate) {
            if (cudaMemsetAsync(grad_scale_dev, 0, sizeof(float), static_cast<cudaStream_t>(stream)) != cudaSuccess)
                return SASQ_ERR_CUDA;
        }
        return SASQ_OK;
    }
    sasq_qdesc_t d{};
    d.x = x;
    d.grad_y = bwd ? grad_y : nullptr;
    d.y = fwd ? y : nullptr;
    d.grad_x = bwd ? grad_x : nullptr;
    d.numel = numel;
    d.scale_index = 0;
    return run_multi(&d, 1, scale_dev, grad_scale_dev, 1, accumulate, dt, bits, workspace, ws_bytes, stream, variant);
}

// ---------------------------------------------------------------------------
// Variant for callers that cannot allocate: the block partials live in a
// file-scope device array instead of a caller-provided workspace.
// ---------------------------------------------------------------------------
constexpr int kStaticPartials = 1024;                      // doubles: 8 KiB held by every device that loads the library
constexpr int64_t kStaticMaxNumel = (int64_t)1 << 30;      // largest tensor the static-scratch call accepts
static __device__ __align__(256) double g_static_partials[kStaticPartials];

// Device address of the static scratch on the current device.  In host code the
// array's name is only a handle; the address a kernel can use comes from the
// runtime, once per device, with that device current.
double* static_partials_ptr(int* err) {
    static double* cache[64] = {nullptr};
    *err = SASQ_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *err = SASQ_ERR_CUDA; return nullptr; }
    if (cache[dev] == nullptr) {
        double* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials) != cudaSuccess || p == nullptr) {
            *err = SASQ_ERR_CUDA;
            return nullptr;
        }
        cache[dev] = p;
    }
    return cache[dev];
}

}  // namespace
}  // namespace sasq

extern "C" {

int sasq_fakequant_fwd_bwd_static(const void* x, const void* grad_y, void* y, void* grad_x, float* grad_scale_dev,
                                  int accumulate, int64_t numel, int dt, const float* scale_dev, int bits,
                                  void* stream) {
    using namespace sasq;
    if (numel > kStaticMaxNumel) return SASQ_ERR_UNSUPPORTED;
    if (numel < 0 || scale_dev == nullptr || grad_scale_dev == nullptr) return SASQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8 || (dt != SASQ_F16 && dt != SASQ_BF16)) return SASQ_ERR_INVALID_ARG;
    if (numel > 0 && (x == nullptr || grad_y == nullptr || y == nullptr || grad_x == nullptr))
        return SASQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(grad_y) || !aligned16(y) || !aligned16(grad_x)) return SASQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (numel == 0) {
        if (!accumulate && cudaMemsetAsync(grad_scale_dev, 0, sizeof(float), st) != cudaSuccess) return SASQ_ERR_CUDA;
        return SASQ_OK;
    }
    const int sm_count = device_sm_count_if_sm100();
    if (sm_count <= 0) return SASQ_ERR_UNSUPPORTED;
    const int grid = grid_for(numel, sm_count);
    if (grid > kStaticPartials) return SASQ_ERR_UNSUPPORTED;      // more blocks than the static scratch holds
    int err = SASQ_OK;
    double* partials = static_partials_ptr(&err);                   // first call on a device resolves the address
    if (partials == nullptr) return err;
    int* status = status_word_ptr();
    if (status == nullptr) return SASQ_ERR_CUDA;

    QParams p{};
    p.d[0].x = static_cast<const uint4*>(x);
    p.d[0].g = static_cast<const uint4*>(grad_y);
    p.d[0].y = static_cast<uint4*>(y);
    p.d[0].dx = static_cast<uint4*>(grad_x);
    p.d[0].numel = numel;
    p.d[0].scale_index = 0;
    p.n = 1;
    p.scales = scale_dev;
    p.partials = partials;      // every block overwrites its own slot: nothing has to start at zero
    p.qn = (float)(1 << (bits - 1));
    p.qp = (float)((1 << (bits - 1)) - 1);
    p.status = status;
    p.grad_scales = grad_scale_dev;
    p.accumulate_mask = accumulate ? 1u : 0u;
    const int ticket_rc = next_ticket(st, &p.ticket);
    if (ticket_rc != SASQ_OK) return ticket_rc;
    const cudaError_t e = (dt == SASQ_BF16) ? launch_mode<true>(true, true, p, grid, st)
                                            : launch_mode<false>(true, true, p, grid, st);
    if (e != cudaSuccess) return SASQ_ERR_CUDA;
    return SASQ_OK;
}

size_t sasq_fakequant_bwd_workspace(int64_t numel) {
    (void)numel;
    return sasq_fakequant_multi_workspace(1);
}

size_t sasq_fakequant_multi_workspace(int n_tensors) {
    if (n_tensors < 1) n_tensors = 1;
    return (size_t)n_tensors * sasq::kMaxGrid * sizeof(double);
}

int sasq_fakequant_fwd(const void* x, void* y, int64_t numel, int dt, const float* scale_dev, int bits,
                       void* stream) {
    return sasq::run_single(x, nullptr, y, nullptr, nullptr, 0, numel, dt, scale_dev, bits, nullptr, 0, stream,
                            true, false);
}

int sasq_fakequant_bwd(const void* x, const void* grad_y, void* grad_x, float* grad_scale_dev, int accumulate,
                       int64_t numel, int dt, const float* scale_dev, int bits, void* workspace, size_t ws_bytes,
                       void* stream) {
    return sasq::run_single(x, grad_y, nullptr, grad_x, grad_scale_dev, accumulate, numel, dt, scale_dev, bits,
                            workspace, ws_bytes, stream, false, true);
}

int sasq_fakequant_fwd_bwd(const void* x, const void* grad_y, void* y, void* grad_x, float* grad_scale_dev,
                           int accumulate, int64_t numel, int dt, const float* scale_dev, int bits,
                           void* workspace, size_t ws_bytes, void* stream) {
    return sasq::run_single(x, grad_y, y, grad_x, grad_scale_dev, accumulate, numel, dt, scale_dev, bits,
                            workspace, ws_bytes, stream, true, true);
}

int sasq_fakequant_fwd_bwd_ablation(const void* x, const void* grad_y, void* y, void* grad_x, float* grad_scale_dev,
                                    int accumulate, int64_t numel, int dt, const float* scale_dev, int bits,
                                    int variant, void* workspace, size_t ws_bytes, void* stream) {
    return sasq::run_single(x, grad_y, y, grad_x, grad_scale_dev, accumulate, numel, dt, scale_dev, bits, workspace,
                            ws_bytes, stream, true, true, variant);
}

int sasq_fakequant_fwd_bwd_multi(const sasq_qdesc_t* descs_host, int n_tensors, const float* scales_dev,
                                 float* grad_scales_dev, int n_scales, int accumulate, int dt, int bits,
                                 void* workspace, size_t ws_bytes, void* stream) {
    return sasq::run_multi(descs_host, n_tensors, scales_dev, grad_scales_dev, n_scales, accumulate, dt, bits,
                           workspace, ws_bytes, stream);
}

}  // extern "C"
