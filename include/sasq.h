/* sasq.h -- C ABI of the B200 (sm_100a) SASQ hot-path library.
 *
 * SASQ (Static Activation Scaling for Quantization-aware training) inserts a
 * fake-quantization operator in front of every frozen linear layer, trains only
 * the activation quantization factors (Sec. 4.2), and at inference applies the
 * learned factors statically in front of an integer GEMM (Fig. 1, Eq. 2).
 *
 * Notation (Eq. 1):  b = bits, Qn = 2^(b-1), Qp = 2^(b-1) - 1, s = factor.
 *   inv = fl32(1 / s)            one IEEE fp32 division per factor
 *   t   = fl32(x * inv)          one fp32 multiply, never fused with anything
 *   r   = rint(t)                round to nearest, ties to even
 *   c   = min(max(r, -Qn), Qp)   the integer code of Eq. 1
 *   m   = (-Qn <= r <= Qp)       Eq. 4: clamp passes the gradient, ends included
 *
 * General rules
 *   - Every data pointer is a DEVICE pointer unless its comment says "host".
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  All work is enqueued on it; no call synchronises except
 *     sasq_device_status.
 *   - The caller owns every buffer.  The library allocates no device memory.
 *   - Tensors are dense, row-major, 16-bit floating point (sasq_dtype_t) and
 *     16-byte aligned.  Factors are fp32 and live in device memory so that an
 *     optimizer can update them without a host round trip.
 *   - A factor may be any finite non-zero fp32 whose reciprocal is finite,
 *     negative values included (the paper puts no constraint on the update
 *     range, Sec. 4.2).  A zero / NaN / Inf factor is detected on the device:
 *     the sticky status word becomes SASQ_ERR_BAD_SCALE and outputs are
 *     unspecified.
 *   - Non-finite activations are outside the contract.  What happens anyway:
 *     +-Inf saturates (m = 0); NaN gives code -Qn, m = 0.
 *   - Host-detectable errors (NULL or misaligned pointers, sizes, bits,
 *     workspace too small, wrong device architecture) return a code and launch
 *     nothing.  There is no CPU fallback.
 *   - numel == 0 / T == 0 is SASQ_OK without a launch (grad_scale is zeroed
 *     unless accumulating).
 */
#ifndef SASQ_H_
#define SASQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SASQ_API __attribute__((visibility("default")))
#else
#define SASQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SASQ_OK = 0,
    SASQ_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, negative size, bits outside [2, 8] ... */
    SASQ_ERR_UNSUPPORTED = 2,   /* shape constraint of a kernel not met, or device is not sm_100 */
    SASQ_ERR_WORKSPACE = 3,     /* workspace NULL or smaller than the matching *_workspace() query */
    SASQ_ERR_BAD_SCALE = 4,     /* device-detected: factor is 0, NaN, Inf or has a non-finite reciprocal */
    SASQ_ERR_TIMEOUT = 5,       /* device-detected: a bounded wait inside a kernel gave up */
    SASQ_ERR_CUDA = 6           /* a CUDA runtime / driver call failed */
} sasq_status_t;

typedef enum { SASQ_F16 = 0, SASQ_BF16 = 1 } sasq_dtype_t;

/* The fake-quant operator and the two ablations of Table 3. */
typedef enum {
    SASQ_FULL_OPERATOR = 0,   /* quant, round, clamp, dequant (Sec. 4.2) */
    SASQ_WITHOUT_ROUND = 1,   /* "w/o round": r = t, so y = clamp(x / s) * s and the factor gradient inside the range is 0 */
    SASQ_WITHOUT_CLAMP = 2    /* "w/o clamp": c = r, every element passes the gradient, term = r - t */
} sasq_variant_t;

/* One tensor of a multi-tensor fake-quant launch (host struct).  y == NULL skips
 * the forward output; grad_y == grad_x == NULL skips the backward; at least one
 * part must be present and every descriptor of one call must have the same
 * parts.  scale_index selects the factor (and the gradient slot) in the arrays
 * passed to the call; several tensors may share one index, which is how one
 * factor per decoder layer is expressed. */
typedef struct {
    const void* x;        /* [numel] activations */
    const void* grad_y;   /* [numel] upstream gradient, or NULL */
    void* y;              /* [numel] fake-quantized output, or NULL */
    void* grad_x;         /* [numel] input gradient, or NULL (must be non-NULL iff grad_y is) */
    int64_t numel;
    int32_t scale_index;
    int32_t reserved;     /* must be 0 */
} sasq_qdesc_t;

SASQ_API const char* sasq_status_string(int status);

/* Fake-quant forward (Sec. 4.2: quant, round, clamp, dequant; Eq. 1):
 *   y[i] = narrow( fl32(c_i * s) ),  one round-to-nearest-even narrowing to `dt`.
 * x, y: [numel] of `dt`; y may alias x.  scale_dev: one fp32.  bits in [2, 8]. */
SASQ_API int sasq_fakequant_fwd(const void* x, void* y, int64_t numel, int dt, const float* scale_dev, int bits,
                       void* stream);

/* Bytes of scratch the backward / fused calls need for a single tensor. */
SASQ_API size_t sasq_fakequant_bwd_workspace(int64_t numel);

/* Straight-through backward (Eq. 4) and the factor gradient that follows from it
 * by the chain rule, summed over EVERY element of the tensor:
 *   grad_x[i]  = m_i ? grad_y[i] : +0                        (bit copy or zero)
 *   grad_scale = sum_i grad_y[i] * (m_i ? (r_i - t_i) : c_i)  (no normalisation)
 * The sum is taken as fp32 products, fixed-shape fp32 trees of 8, then double
 * accumulation per thread, a fixed-order block reduction and a fixed-order
 * second-stage combine: the result is bit-identical from run to run and within
 * 1e-4 relative of a double-precision sum.
 * grad_scale_dev: one fp32, overwritten (accumulate == 0) or added to (!= 0).
 * workspace: >= sasq_fakequant_bwd_workspace(numel) bytes, 16-byte aligned; its
 * contents need no initialisation and are garbage afterwards.  Calls that share
 * a workspace must be ordered on the stream. grad_x may alias grad_y. */
SASQ_API int sasq_fakequant_bwd(const void* x, const void* grad_y, void* grad_x, float* grad_scale_dev, int accumulate,
                       int64_t numel, int dt, const float* scale_dev, int bits, void* workspace,
                       size_t ws_bytes, void* stream);

/* Forward and backward in one pass over x and grad_y (what one scale-only
 * training step does per quantizer): same results as the two calls above. */
SASQ_API int sasq_fakequant_fwd_bwd(const void* x, const void* grad_y, void* y, void* grad_x, float* grad_scale_dev,
                           int accumulate, int64_t numel, int dt, const float* scale_dev, int bits,
                           void* workspace, size_t ws_bytes, void* stream);

/* The fused pass with one of the operator's steps removed (Table 3's ablations; SASQ_FULL_OPERATOR gives
 * sasq_fakequant_fwd_bwd).  Same arguments and conventions otherwise. */
SASQ_API int sasq_fakequant_fwd_bwd_ablation(const void* x, const void* grad_y, void* y, void* grad_x,
                                             float* grad_scale_dev, int accumulate, int64_t numel, int dt,
                                             const float* scale_dev, int bits, int variant, void* workspace,
                                             size_t ws_bytes, void* stream);

/* The same fused pass for callers that can neither allocate device memory nor
 * hand over a workspace: for instance a plugin hook of an inference runtime that
 * forbids allocation inside its execute call, or a process whose device memory
 * is entirely owned by another allocator, so that a cudaMalloc here would fail
 * or break its budget.  (The paper has no counterpart; this is a deployment
 * convenience of the library.)  The block partials of the scale-gradient
 * reduction live in a fixed 8 KiB array inside the library's device image, which
 * every GPU that loads the library holds until the process exits.  The call
 * itself performs no allocation of any kind.
 *   - Results are identical, bit for bit, to sasq_fakequant_fwd_bwd.
 *   - numel may be at most 2^30; larger tensors (or a device with more thread
 *     blocks than the array has slots) give SASQ_ERR_UNSUPPORTED and no launch.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Its previous contents never
 *     matter (every slot that is read is written first, nothing needs zeroing),
 *     but two calls that overlap on the GPU -- different streams, or different
 *     host threads without ordering -- race on it and corrupt each other's
 *     grad_scale.  Order them on one stream or with events. */
SASQ_API int sasq_fakequant_fwd_bwd_static(const void* x, const void* grad_y, void* y, void* grad_x,
                                           float* grad_scale_dev, int accumulate, int64_t numel, int dt,
                                           const float* scale_dev, int bits, void* stream);

/* Bytes of scratch for a multi-tensor call with n_tensors descriptors. */
SASQ_API size_t sasq_fakequant_multi_workspace(int n_tensors);

/* Several quantizers in one call (e.g. the seven linear inputs of a decoder
 * layer).  descs_host: HOST array of n_tensors descriptors, copied into the
 * launch parameters (it may be freed on return).  scales_dev[n_scales] fp32,
 * grad_scales_dev[n_scales] fp32 (may be NULL when no descriptor has a backward
 * part).  Every slot of grad_scales_dev that some descriptor with a backward
 * part refers to is overwritten (or accumulated into); other slots are left
 * alone.  A slot shared by several tensors receives the sum over all of them,
 * combined in descriptor order (one factor per layer). */
SASQ_API int sasq_fakequant_fwd_bwd_multi(const sasq_qdesc_t* descs_host, int n_tensors, const float* scales_dev,
                                 float* grad_scales_dev, int n_scales, int accumulate, int dt, int bits,
                                 void* workspace, size_t ws_bytes, void* stream);

/* Bytes of scratch the per-channel call needs when it has a backward part. */
SASQ_API size_t sasq_fakequant_per_channel_workspace(int64_t T, int64_t K);

/* The fake-quant operator with one factor per channel (per column of x[T, K]), the granularity of the paper's
 * experiments (Fig. 2b; Sec. 5.1: activations and weights both per channel).  Per element the arithmetic is that
 * of the per-tensor calls with s = scales[k]; the gradient of factor k is summed over the T rows of column k:
 *   y[t,k]  = narrow( fl32(c * scales[k]) ),   grad_x[t,k] = m ? grad_y[t,k] : +0,
 *   grad_scales[k] = sum_t grad_y[t,k] * (m ? (r - t') : c)       (t' = fl32(x * fl32(1/scales[k])))
 * x, y, grad_y, grad_x: [T, K] of `dt`; y == NULL skips the forward output, grad_y == grad_x == NULL skips the
 * backward; y may alias x and grad_x may alias grad_y.  scales_dev, grad_scales_dev: [K] fp32, 16-byte aligned;
 * grad_scales_dev is overwritten (accumulate == 0) or added to.  The sum runs in double per thread down the rows
 * of a row group, then over the row groups in a fixed order: bit-identical from run to run, within 1e-4 relative
 * of a double-precision sum.  workspace: >= sasq_fakequant_per_channel_workspace(T, K) bytes when there is a
 * backward part.  K % 8 == 0, otherwise SASQ_ERR_UNSUPPORTED.  Any zero / non-finite factor sets
 * SASQ_ERR_BAD_SCALE in the status word. */
SASQ_API int sasq_fakequant_fwd_bwd_per_channel(const void* x, const void* grad_y, void* y, void* grad_x,
                                                float* grad_scales_dev, int accumulate, int64_t T, int64_t K, int dt,
                                                const float* scales_dev, int bits, void* workspace, size_t ws_bytes,
                                                void* stream);

/* One tensor of a multi-tensor per-channel launch (host struct); fields as the arguments of
 * sasq_fakequant_fwd_bwd_per_channel.  All descriptors of a call have the same parts (forward and / or backward). */
typedef struct {
    const void* x;          /* [T, K] */
    const void* grad_y;     /* [T, K] or NULL */
    void* y;                /* [T, K] or NULL */
    void* grad_x;           /* [T, K] or NULL (non-NULL iff grad_y is) */
    const float* scales;    /* [K] fp32, device */
    float* grad_scales;     /* [K] fp32, device (needed with a backward part) */
    int64_t T, K;
    int64_t reserved;       /* must be 0 */
} sasq_pcdesc_t;

/* Bytes of scratch for a multi-tensor per-channel call whose tensors have total_K channels in all. */
SASQ_API size_t sasq_fakequant_per_channel_multi_workspace(int64_t total_K);

/* Up to 16 per-channel quantizers in one launch (e.g. the seven linear inputs of a decoder layer): the tensors run
 * side by side, each on a share of the GPU in proportion to its size.  descs_host: HOST array, copied into the launch
 * parameters.  Results are those of n_tensors separate calls. */
SASQ_API int sasq_fakequant_fwd_bwd_per_channel_multi(const sasq_pcdesc_t* descs_host, int n_tensors, int accumulate,
                                                      int dt, int bits, void* workspace, size_t ws_bytes,
                                                      void* stream);

/* Bytes of scratch sasq_static_w8a8_linear needs for this shape (may be 0). */
SASQ_API size_t sasq_static_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K);

/* Static W8A8 linear (Eq. 1 with the fixed learned factor, then Eq. 2):
 *   X_int[t,k] = int8(c(x[t,k]))                 no max / scale pass at run time
 *   acc[t,n]   = sum_k X_int[t,k] * w[n,k]       int32, exact
 *   y[t,n]     = narrow( fl32(acc) * fl32(s_x * w_scale[n]) (+ bias[n]) )
 * x: [T, K] of `dt`.  w: [N, K] int8, one row per output channel (the paper's W
 * is its transpose).  w_scale: [N] fp32 per-output-channel weight factors.
 * x_scale_dev: one fp32.  bias: [N] of `dt` or NULL (bias is never quantized,
 * Sec. 3).  y: [T, N] of `dt`.  acc_out: [T, N] int32 or NULL; when given, the
 * raw accumulators are also written (parity / debugging).
 * Constraints: K % 16 == 0, N % 8 == 0, K <= 131072 (int32 cannot overflow),
 * bits in [2, 8]; otherwise SASQ_ERR_UNSUPPORTED.
 * The weights are frozen (Sec. 4.2): `w` is read as soon as the kernel is resident, which, for a call that follows
 * another call of this library on the same stream, can be before that earlier kernel has finished.  No call of this
 * library writes int8 weights on that fast path (sasq_quantize_weight does not let its successor start early), so
 * this matters only to a caller that hands `w` a buffer some other SASQ call on the stream is still writing as
 * its 16-bit output: do not.  x, x_scale_dev, w_scale, bias and y are touched only after every earlier kernel of
 * the stream has completed. */
SASQ_API int sasq_static_w8a8_linear(const void* x, const int8_t* w, const float* w_scale, const float* x_scale_dev,
                            const void* bias, void* y, int32_t* acc_out, int64_t T, int64_t N, int64_t K,
                            int dt, int bits, void* workspace, size_t ws_bytes, void* stream);

/* Bytes of scratch sasq_static_w8a8_linear_per_channel needs for this shape. */
SASQ_API size_t sasq_static_w8a8_linear_per_channel_workspace(int64_t T, int64_t N, int64_t K);

/* Static W8A8 linear with one learned activation factor per CHANNEL (column of x), the granularity of the paper's
 * experiments (Sec. 5.1).  Because the factors are static, they are absorbed into the frozen weights ahead of time
 * instead of being carried through Eq. 3's groups: the caller quantizes w'[n,k] = w_fp[n,k] * s_x[k] per output
 * channel (sasq_quantize_weight) and passes the result as w, w_scale.  The call then computes
 *   X_int[t,k] = int8(c(x[t,k])) with s = x_scales_dev[k]        (Eq. 1 per channel, no run-time scale pass)
 *   acc[t,n]   = sum_k X_int[t,k] * w[n,k]                        (= sum_k X_int s_x[k] w_fp[n,k] / w_scale[n], up to the
 *                                                                  weight rounding)
 *   y[t,n]     = narrow( fl32(acc) * w_scale[n] (+ bias[n]) )
 * x_scales_dev: [K] fp32.  Other arguments as for sasq_static_w8a8_linear. */
SASQ_API int sasq_static_w8a8_linear_per_channel(const void* x, const int8_t* w, const float* w_scale,
                                                 const float* x_scales_dev, const void* bias, void* y,
                                                 int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt, int bits,
                                                 void* workspace, size_t ws_bytes, void* stream);

/* Bytes of scratch sasq_fakequant_linear_fp_weights needs for this shape. */
SASQ_API size_t sasq_fakequant_linear_fp_weights_workspace(int64_t T, int64_t N, int64_t K);

/* The "FP weights" form of the quantized linear (Table 3; Eq. 5 and 6: quantization seen as a transform of the
 * activations alone): the activations go through the fake-quant operator, the weights stay 16-bit floating point:
 *   x'[t,k] = narrow( fl32(c(x[t,k]) * s) )                       (sasq_fakequant_fwd, bit for bit)
 *   y[t,n]  = narrow( sum_k x'[t,k] * w[n,k] (+ bias[n]) )        products exact, fp32 accumulation on the tensor
 *                                                                  cores (order unspecified), bias added in fp32
 * x: [T, K], w: [N, K], bias: [N] or NULL, y: [T, N], all of `dt`; x_scale_dev: one fp32.  Constraints: K % 8 == 0,
 * N % 8 == 0 (otherwise SASQ_ERR_UNSUPPORTED).  The workspace receives x'.  Two launches. */
SASQ_API int sasq_fakequant_linear_fp_weights(const void* x, const void* w, const float* x_scale_dev, const void* bias,
                                              void* y, int64_t T, int64_t N, int64_t K, int dt, int bits,
                                              void* workspace, size_t ws_bytes, void* stream);

/* Bytes of scratch sasq_static_w8a8_linear_grouped needs for this shape. */
SASQ_API size_t sasq_static_w8a8_linear_grouped_workspace(int64_t T, int64_t N, int64_t K);

/* Static W8A8 linear in the grouped form of Eq. 3: the K axis is cut into K / group groups of `group` consecutive
 * columns, each with its own static activation factor; a group's integer partial product is scaled by its factor
 * and the partials are accumulated in fp32, in group order:
 *   X_int[t,k] = int8(c(x[t,k])) with s = s_group[k / group]                       (Eq. 1 per group)
 *   acc_g[t,n] = sum_{k in group g} X_int[t,k] * w[n,k]                            (int32)
 *   y[t,n]     = narrow( sum_g fl32(acc_g) * fl32(s_group[g] * w_scale[n]) (+ bias[n]) )   (fp32 adds, g ascending,
 *                                                                                   starting from +0, no FMA)
 * s_group_dev: [K / group] fp32 in DEVICE memory.  group must be a multiple of 128 and divide K (otherwise
 * SASQ_ERR_UNSUPPORTED).  Other arguments, alignment, ownership and errors as for sasq_static_w8a8_linear; there is
 * no acc_out (no single integer accumulator exists).  Three launches: reciprocals, activation quantizer, GEMM. */
SASQ_API int sasq_static_w8a8_linear_grouped(const void* x, const int8_t* w, const float* w_scale,
                                             const float* s_group_dev, int64_t group, const void* bias, void* y,
                                             int64_t T, int64_t N, int64_t K, int dt, int bits, void* workspace,
                                             size_t ws_bytes, void* stream);

/* Bytes of scratch sasq_dynamic_w8a8_linear needs for this shape. */
SASQ_API size_t sasq_dynamic_w8a8_linear_workspace(int64_t T, int64_t N, int64_t K);

/* W8A8 linear with DYNAMIC per-token activation factors: the generation phase of the paper's phased quantization
 * (Sec. 4.4; one token per sequence, so per-token equals per-tensor on that row).  For every row t:
 *   s_t        = max_k |x[t,k]| / Qp                  (Eq. 1 on the row; an all-zero row takes s_t = 1)
 *   X_int[t,k] = int8(c(x[t,k])) with s = s_t,   acc[t,n] = sum_k X_int[t,k] * w[n,k]
 *   y[t,n]     = narrow( fl32(acc) * fl32(s_t * w_scale[n]) (+ bias[n]) )
 * Arguments as for sasq_static_w8a8_linear, without x_scale_dev.  row_scale_out: [T] fp32 that receives the
 * factors, or NULL (they are then kept in the workspace).  For T <= 128 (the generation phase) everything runs in
 * one launch: the rows are dealt to the CTAs of the GEMM kernel, whose quantizer warps find a row's factor and write
 * its codes.  For larger T one extra launch computes the factors and the codes (a row's factor needs the whole row
 * first). */
SASQ_API int sasq_dynamic_w8a8_linear(const void* x, const int8_t* w, const float* w_scale, const void* bias, void* y,
                                      float* row_scale_out, int32_t* acc_out, int64_t T, int64_t N, int64_t K, int dt,
                                      int bits, void* workspace, size_t ws_bytes, void* stream);

/* One linear of sasq_static_w8a8_linear_multi: the arguments of sasq_static_w8a8_linear for one problem.  The
 * struct lives in HOST memory; the pointers in it are DEVICE pointers with the layouts, alignment and ownership
 * stated there (bias may be NULL). */
typedef struct sasq_linear_desc {
    const void* x;          /* [T, K] 16-bit activations */
    const int8_t* w;        /* [N, K] int8 weights */
    const float* w_scale;   /* [N] fp32 */
    const float* x_scale;   /* 1 fp32: the static factor of this linear's quantizer */
    const void* bias;       /* [N] 16-bit, or NULL */
    void* y;                /* [T, N] 16-bit output */
    int64_t T, N, K;
} sasq_linear_desc_t;

/* Bytes of scratch sasq_static_w8a8_linear_multi needs for these problems (descs_host: HOST memory, count entries). */
SASQ_API size_t sasq_static_w8a8_linear_multi_workspace(int count, const sasq_linear_desc_t* descs_host);

/* Several independent static W8A8 linears (Sec. 4.2 static factors, Eq. 1 + Eq. 2, each exactly as sasq_static_w8a8_linear
 * computes it: the results are bit-identical to `count` separate calls) submitted together, e.g. the q/k/v or the
 * gate/up projections of a decoder layer, which do not depend on one another.  Consecutive problems with T > 128 run
 * in ONE launch (up to 8 problems, 1024 256-row blocks and 80 MiB of int8 activation codes, i.e. sum of T x K,
 * per launch, so that the codes stay in L2 until they are used; more are cut into several launches): the CTA
 * pairs walk one tile list over all of them and the quantizer warps one chunk list, so the activation quantization
 * of a problem and the drain of its last tiles overlap with the MMAs of its neighbours instead of idling the tensor
 * cores at every launch boundary.  A run that contains problems with T <= 128 shares a launch only if it has at
 * least two problems whose output tiles fill every resident CTA pair (the weights then stream through one launch
 * instead of one latency chain per linear); otherwise consecutive problems with the same T <= 128 whose 128-channel
 * output tiles all fit the device at once (one CTA each; e.g. the q/k/v projections of a decode step) share one
 * launch of the small-T kernel, and what is left is launched one by one, in order.  No problem may read another's
 * output.  descs_host: HOST memory, read before the call returns.  All problems share dt and bits.
 * Returns SASQ_ERR_INVALID_ARG / UNSUPPORTED / WORKSPACE as sasq_static_w8a8_linear does, checked for every problem
 * before anything is launched. */
SASQ_API int sasq_static_w8a8_linear_multi(int count, const sasq_linear_desc_t* descs_host, int dt, int bits,
                                           void* workspace, size_t ws_bytes, void* stream);

/* How many kernels sasq_static_w8a8_linear_multi launches for these problems (only T, N, K of each descriptor are
 * read) on a device with `num_pairs` resident CTA pairs (74 on a B200): introspection for launch counting and tests;
 * runs on the host, touches no device.  Returns -1 for invalid arguments. */
SASQ_API int sasq_static_w8a8_linear_multi_launches(int count, const sasq_linear_desc_t* descs_host, int num_pairs);

/* How sasq_static_w8a8_linear splits a [T, N] output over `num_pairs` co-operating CTA pairs when T > 128
 * (introspection for tests and tuning; runs on the host, touches no device).  Every 256-row block is cut into the
 * same number of column tiles, widths multiples of 16 that differ by at most 16; the number is chosen so that the
 * tiles fill whole waves of the pairs; tile t goes to pair t % num_pairs, column tiles fastest.  Writes up to `cap`
 * triples (first row, first column, width in columns) of pair `pair_id` to tiles_host (HOST memory, [cap][3]
 * int32) and returns how many tiles the pair has, or -1 for invalid arguments. */
SASQ_API int sasq_static_w8a8_linear_tiles(int64_t T, int64_t N, int num_pairs, int pair_id, int32_t* tiles_host,
                                           int cap);

/* ---- PTQ initialisation (Sec. 4.1), set-up only, not on the hot path ---- */

/* Bytes of scratch sasq_absmax_scale needs. */
SASQ_API size_t sasq_absmax_scale_workspace(int64_t numel);

/* Max-based factor of one calibration batch (Eq. 1): scale_out_dev[0] =
 * max_i |x[i]| / Qp in fp32.  The paper initialises each factor with the average
 * of these values over the calibration batches; the caller averages.  x:
 * [numel] of `dt`; an all-zero or empty x gives 0 (not a usable factor). */
SASQ_API int sasq_absmax_scale(const void* x, int64_t numel, int dt, int bits, float* scale_out_dev, void* workspace,
                               size_t ws_bytes, void* stream);

/* The same per channel (column of x[T, K]), the granularity of the paper's experiments (Sec. 5.1):
 * scales_out_dev[k] = max_t |x[t,k]| / Qp in fp32 (0 for an all-zero column or T == 0).  x: [T, K] of `dt`,
 * K % 8 == 0; scales_out_dev: [K] fp32, also used as scratch while the call runs. */
SASQ_API int sasq_absmax_scale_per_channel(const void* x, int64_t T, int64_t K, int dt, int bits,
                                           float* scales_out_dev, void* stream);

/* Running mean for the initialisation of Sec. 4.1 ("the average of the factors of the calibration batches"),
 * kept on the device: fed the factors of batch number `count` (1, 2, ...) it turns the mean of the first
 * count - 1 batches into the mean of the first count:
 *   mean[i] = value[i]                                   if count == 1
 *   mean[i] = mean[i] + (value[i] - mean[i]) / count     otherwise (fp32)
 * mean_dev, value_dev: [n] fp32 (one entry per tensor, or per channel). */
SASQ_API int sasq_running_mean(float* mean_dev, const float* value_dev, int n, int count, void* stream);

/* Per-output-channel symmetric weight quantizer (Eq. 1 applied to each column of
 * the paper's K x N weight, i.e. each row of w[N, K]; weights are always
 * quantized per channel, Sec. 5.1):  w_scale[n] = max_k |w[n,k]| / Qp (1 for an
 * all-zero row), w_int[n,k] = clamp(rint(w[n,k] * fl32(1 / w_scale[n])), -Qn, Qp).
 * w: [N, K] fp32; w_int: [N, K] int8; w_scale: [N] fp32. */
SASQ_API int sasq_quantize_weight(const float* w, int8_t* w_int, float* w_scale, int64_t N, int64_t K, int bits,
                                  void* stream);

/* One AdamW step on n factors (the factors are the only trainable parameters, Sec. 4.2; AdamW, lr 2e-4, Sec. 5.1),
 * consuming the gradients the backward calls wrote, all in device memory, fp32:
 *   m = beta1 m + (1 - beta1) g;   v = beta2 v + (1 - beta2) g^2;
 *   s = s - lr * ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay * s )
 * scales_dev, exp_avg_dev (m), exp_avg_sq_dev (v): [n] fp32, updated in place; grad_scales_dev: [n] fp32.
 * step counts from 1.  No constraint is put on the updated factors (Sec. 4.2). */
SASQ_API int sasq_adamw_scales(float* scales_dev, const float* grad_scales_dev, float* exp_avg_dev,
                               float* exp_avg_sq_dev, int n, int step, float lr, float beta1, float beta2, float eps,
                               float weight_decay, void* stream);

/* Concurrency of the linear entry points.  When the activation quantizer runs inside the GEMM launch (every static
 * linear with T <= 262144 whose tiles fit the device), CTAs of that launch wait for codes that other CTAs of the
 * same launch write, so all of its CTAs must be resident together.  By default (on != 0) these launches are
 * therefore made as co-operative grids, which the driver starts only when every CTA can be resident: linears may
 * then run on several streams of one device at once, or beside other kernels, and merely queue behind one another.
 * A caller that submits all of its linears on ONE stream of an otherwise idle device may switch this off
 * (on == 0): plain launches let a launch's set-up overlap its predecessor's tail, about 2 us per launch on a B200.
 * With it off, two such launches that overlap on different streams can each hold the SMs the other is waiting for;
 * their bounded waits then give up after about a second with SASQ_ERR_TIMEOUT in the status word (outputs
 * unspecified, nothing hangs).  Applies to launches made afterwards, process-wide; returns the previous setting.
 * The paper has no counterpart. */
SASQ_API int sasq_set_gang_launch(int on);

/* Test hook.  Every wait inside the GEMM kernels (on an mbarrier, on the activation quantizer's counters) gives up
 * after this many SM clock cycles, raises SASQ_ERR_TIMEOUT in the status word and lets the kernel finish in an
 * orderly way (outputs are then unspecified).  The default is 2^31 cycles, about a second; a negative value restores
 * it.  Returns the previous limit.  Applies to launches made afterwards.  sasq_device_status clears the library's
 * internal counters when it reports a timeout, so the next call starts clean. */
SASQ_API long long sasq_debug_set_wait_limit(long long cycles);

/* Measurement aid (the paper has no counterpart; Sec. 2 only names integer GEMM kernels as usable).  Runs, on every
 * resident CTA pair of the device, `mma_per_pair` (>= 32, rounded down to a multiple of 32) back-to-back
 * tcgen05.mma.cta_group::2.kind::i8 instructions of shape 256 x n_cols x 32 (n_cols a multiple of 32 in [32, 256])
 * on pseudo-random int8 operands held in shared memory: the instruction the static W8A8 linear is built from, with no loads and no
 * epilogue around it.  Synchronises `stream`.  Writes to HOST memory: *ops_per_second_host = integer operations
 * (2 per multiply-accumulate) of the whole device over the CUDA-event time of the launch, and *mac_per_clk_sm_host
 * = multiply-accumulates per SM clock cycle per SM on the slowest pair.  A few ms of MMAs give the burst rate, a
 * second or more the rate under the power cap.  Allocates nothing.  Errors: SASQ_ERR_INVALID_ARG,
 * SASQ_ERR_UNSUPPORTED (not sm_100), SASQ_ERR_TIMEOUT (a bounded wait gave up), SASQ_ERR_CUDA. */
SASQ_API int sasq_debug_int8_issue_rate(int mma_per_pair, int n_cols, double* ops_per_second_host,
                                        double* mac_per_clk_sm_host, void* stream);

/* Synchronises `stream`, returns the sticky device status word of the current
 * device (SASQ_OK, SASQ_ERR_BAD_SCALE or SASQ_ERR_TIMEOUT) and clears it. */
SASQ_API int sasq_device_status(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SASQ_H_ */
