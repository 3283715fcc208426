// SASQ CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
//
// A plain, slow, obviously-correct CPU statement of what the static-scale
// activation quantizer and the static W8A8 linear compute.  Only the test
// suite, the smoke check and the benchmark's CPU-baseline leg may call it.
// It shares no code, header, table or helper with the CUDA library.
//
// Every function follows a definition in the SASQ paper:
//   * symmetric b-bit quantizer, clamp(round(X/S), -2^(b-1), 2^(b-1)-1)   -- Eq. 1
//   * max-based factor S = max|X| / (2^(b-1)-1)                             -- Eq. 1
//   * quantized linear  Y = S_x (X_int W_int) S_w                           -- Eq. 2
//   * grouped form      Y = sum_i (S_xi S_w)(X_int,i W_int)                 -- Eq. 3
//   * straight-through gradients of round and clamp                        -- Eq. 4
//   * fake quantization = quant, round, truncation, dequant, output float  -- Sec. 4.2 / 4.3
//   * ablation variants "w/o round", "w/o clamp"                           -- Table 3
//   * bias is left unquantized                                             -- Sec. 3
//
// Readings where the paper is silent (each listed in the design notes):
//   rounding is ties-to-even; X/S is evaluated as x * fl32(1/s) in fp32 with
//   two roundings and no fused multiply-add; Eq. 4's range test is applied to
//   the rounded value, inclusive at both ends; the scale gradient is the plain
//   chain-rule sum with no normalisation; accumulation is in double.
//
// Pins (tests/test_oracle_*.py): idempotence, clip bounds, power-of-two
// identities, fp64 finite differences of the STE surrogate, torch-autograd
// float64 on tiny tensors, closed forms, int64 brute force for the GEMM,
// exhaustive checks of the 16-bit conversions against numpy / torch.
//
// Build: g++ -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC
// (contraction off is load-bearing: x*inv must round before anything else).

#include <cfenv>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------
// 16-bit storage formats.  dtype: 0 = IEEE binary16, 1 = bfloat16.
// Widening is exact; narrowing is one round-to-nearest-even step.
// ---------------------------------------------------------------------------
inline float bits_to_f32(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }
inline uint32_t f32_to_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }

float half_to_f32(uint16_t h) {
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    const uint32_t exp = (h >> 10) & 0x1Fu;
    const uint32_t man = h & 0x3FFu;
    if (exp == 0x1Fu) return bits_to_f32(sign | 0x7F800000u | (man << 13));   // inf / nan
    if (exp == 0) {
        // zero or subnormal: value = man * 2^-24, exact in fp32
        const float v = std::ldexp((float)man, -24);
        return sign ? -v : v;
    }
    return bits_to_f32(sign | ((exp + 112u) << 23) | (man << 13));
}

uint16_t f32_to_half_rne(float f) {
    const uint32_t u = f32_to_bits(f);
    const uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    const uint32_t absu = u & 0x7FFFFFFFu;
    if (absu > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);               // nan
    if (absu == 0x7F800000u) return (uint16_t)(sign | 0x7C00u);              // inf
    const double a = std::fabs((double)f);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7C00u);                     // rounds to inf
    if (a < std::ldexp(1.0, -14)) {
        // subnormal target: units of 2^-24, ties to even (nearbyint in FE_TONEAREST)
        const double q = std::nearbyint(std::ldexp(a, 24));
        return (uint16_t)(sign | (uint16_t)q);                               // q == 1024 becomes the smallest normal
    }
    int e;
    const double m = std::frexp(a, &e);            // a = m * 2^e, m in [0.5, 1)
    // normal half: 1.mmmmmmmmmm * 2^(e-1); 11 significant bits
    double q = std::nearbyint(std::ldexp(m, 11));  // in [1024, 2048]
    int ee = e - 1;
    if (q == 2048.0) { q = 1024.0; ee += 1; }
    const uint32_t biased = (uint32_t)(ee + 15);
    return (uint16_t)(sign | (biased << 10) | ((uint32_t)q - 1024u));
}

float bf16_to_f32(uint16_t h) { return bits_to_f32((uint32_t)h << 16); }

uint16_t f32_to_bf16_rne(float f) {
    const uint32_t u = f32_to_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);   // quiet nan
    const uint32_t lsb = (u >> 16) & 1u;
    return (uint16_t)((u + 0x7FFFu + lsb) >> 16);
}

inline float widen(uint16_t h, int dtype) { return dtype == 0 ? half_to_f32(h) : bf16_to_f32(h); }
inline uint16_t narrow(float f, int dtype) { return dtype == 0 ? f32_to_half_rne(f) : f32_to_bf16_rne(f); }

// ---------------------------------------------------------------------------
// One element of the quantizer, in the paper's order: quant, round, clamp.
// variant 0 = full, 1 = "w/o round", 2 = "w/o clamp" (Table 3).
// ---------------------------------------------------------------------------
struct Q1 {
    float t;      // x * (1/s)           (the "quant" step of Eq. 1)
    float r;      // after rounding      (or t itself without round)
    float c;      // after clamping      (or r itself without clamp)
    bool inside;  // Eq. 4: clamp passes the gradient iff its argument is in [min, max]
};

inline Q1 quant1(float x, float inv, float qn, float qp, int variant) {
    Q1 q;
    q.t = x * inv;                                        // one fp32 multiply, rounded once
    q.r = (variant == 1) ? q.t : std::nearbyintf(q.t);     // FE_TONEAREST: ties to even
    if (variant == 2) {
        q.c = q.r;
        q.inside = true;
    } else {
        q.c = std::fminf(std::fmaxf(q.r, -qn), qp);        // Eq. 1 clamp
        q.inside = (q.r >= -qn) && (q.r <= qp);            // Eq. 4, inclusive
    }
    return q;
}

inline bool bits_ok(int bits) { return bits >= 2 && bits <= 8; }

}  // namespace

extern "C" {

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// 16-bit conversions, exposed so the tests can pin them against numpy / torch.
void oracle_widen(const uint16_t* in, float* out, int64_t n, int dtype) {
    for (int64_t i = 0; i < n; ++i) out[i] = widen(in[i], dtype);
}
void oracle_narrow(const float* in, uint16_t* out, int64_t n, int dtype) {
    for (int64_t i = 0; i < n; ++i) out[i] = narrow(in[i], dtype);
}

// Eq. 1, second half: S = max|X| / (2^(b-1) - 1), in fp32.
float oracle_absmax_scale(const uint16_t* x, int64_t numel, int dtype, int bits) {
    float amax = 0.0f;
    for (int64_t i = 0; i < numel; ++i) {
        const float a = std::fabs(widen(x[i], dtype));
        if (a > amax) amax = a;
    }
    const float qp = (float)((1 << (bits - 1)) - 1);
    return amax / qp;
}

// Fake-quant forward (Sec. 4.2): y = s * clamp(round(x / s)).  x is [rows, cols]
// row-major; codes (optional) receives the integer of Eq. 1 for every element
// (for variant 1 the value is not an integer and codes must be NULL).
int oracle_fakequant_fwd(const uint16_t* x, uint16_t* y, int32_t* codes, int64_t rows, int64_t cols,
                         int dtype, float s, int bits, int variant) {
    if (!bits_ok(bits) || variant < 0 || variant > 2) return 1;
    if (codes && variant == 1) return 1;
    std::fesetround(FE_TONEAREST);
    const float inv = 1.0f / s;                            // fp32 IEEE division, once per scale
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < rows; ++row) {
        std::fesetround(FE_TONEAREST);
        for (int64_t col = 0; col < cols; ++col) {
            const int64_t i = row * cols + col;
            const Q1 q = quant1(widen(x[i], dtype), inv, qn, qp, variant);
            if (y) y[i] = narrow(q.c * s, dtype);          // dequant: fp32 multiply, one narrowing
            if (codes) codes[i] = (int32_t)q.c;
        }
    }
    return 0;
}

// STE backward (Eq. 4) and the scale gradient that follows from it by the chain
// rule:  y = s*c, c = clamp(r), r = round(u), u = x/s
//   dy/dx = [inside]                         -> dx = g or 0
//   dy/ds = c + s*[inside]*(-x/s^2) = c - [inside]*u
//         = r - u inside the range, the clamp bound outside.
// ds is the sum over every element, accumulated in double: each row
// sequentially, then the row sums sequentially in row order.
int oracle_fakequant_bwd(const uint16_t* x, const uint16_t* g, uint16_t* dx, double* ds_out,
                         int64_t rows, int64_t cols, int dtype, float s, int bits, int variant) {
    if (!bits_ok(bits) || variant < 0 || variant > 2) return 1;
    std::fesetround(FE_TONEAREST);
    const float inv = 1.0f / s;
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
    double* row_sum = new double[rows > 0 ? rows : 1];
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < rows; ++row) {
        std::fesetround(FE_TONEAREST);
        double acc = 0.0;
        for (int64_t col = 0; col < cols; ++col) {
            const int64_t i = row * cols + col;
            const Q1 q = quant1(widen(x[i], dtype), inv, qn, qp, variant);
            const float gi = widen(g[i], dtype);
            if (dx) dx[i] = q.inside ? g[i] : (uint16_t)0;  // exactly g, or +0
            const float term = q.inside ? (q.r - q.t) : q.c;
            acc += (double)gi * (double)term;
        }
        row_sum[row] = acc;
    }
    double ds = 0.0;
    for (int64_t row = 0; row < rows; ++row) ds += row_sum[row];
    delete[] row_sum;
    if (ds_out) *ds_out = ds;
    return 0;
}

// Per-channel activation factors (Fig. 2b; the granularity of the paper's
// experiments): one factor per column of x.  ds[col] sums over the rows.
int oracle_fakequant_fwd_per_channel(const uint16_t* x, uint16_t* y, int32_t* codes, int64_t rows,
                                     int64_t cols, int dtype, const float* s, int bits) {
    if (!bits_ok(bits)) return 1;
    std::fesetround(FE_TONEAREST);
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < rows; ++row) {
        std::fesetround(FE_TONEAREST);
        for (int64_t col = 0; col < cols; ++col) {
            const int64_t i = row * cols + col;
            const float inv = 1.0f / s[col];
            const Q1 q = quant1(widen(x[i], dtype), inv, qn, qp, 0);
            if (y) y[i] = narrow(q.c * s[col], dtype);
            if (codes) codes[i] = (int32_t)q.c;
        }
    }
    return 0;
}

int oracle_fakequant_bwd_per_channel(const uint16_t* x, const uint16_t* g, uint16_t* dx, double* ds_out,
                                     int64_t rows, int64_t cols, int dtype, const float* s, int bits) {
    if (!bits_ok(bits)) return 1;
    std::fesetround(FE_TONEAREST);
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
    for (int64_t col = 0; col < cols; ++col) ds_out[col] = 0.0;
    for (int64_t row = 0; row < rows; ++row) {
        for (int64_t col = 0; col < cols; ++col) {
            const int64_t i = row * cols + col;
            const float inv = 1.0f / s[col];
            const Q1 q = quant1(widen(x[i], dtype), inv, qn, qp, 0);
            const float gi = widen(g[i], dtype);
            if (dx) dx[i] = q.inside ? g[i] : (uint16_t)0;
            const float term = q.inside ? (q.r - q.t) : q.c;
            ds_out[col] += (double)gi * (double)term;
        }
    }
    return 0;
}

// Eq. 1 applied to the activation with the fixed (static) factor: the integer
// operand of the GEMM.  codes are int8; valid for bits <= 8.
int oracle_quantize_act(const uint16_t* x, int8_t* codes, int64_t rows, int64_t cols, int dtype,
                        float s, int bits) {
    if (!bits_ok(bits)) return 1;
    std::fesetround(FE_TONEAREST);
    const float inv = 1.0f / s;
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t row = 0; row < rows; ++row) {
        std::fesetround(FE_TONEAREST);
        for (int64_t col = 0; col < cols; ++col) {
            const int64_t i = row * cols + col;
            codes[i] = (int8_t)quant1(widen(x[i], dtype), inv, qn, qp, 0).c;
        }
    }
    return 0;
}

// Per-output-channel symmetric weight quantizer (Eq. 1 per column of the
// paper's K x N weight; stored here as w[N, K], one factor per row n).
// A row of zeros gets factor 1 and codes 0.
int oracle_quantize_weight(const float* w, int8_t* w_int, float* w_scale, int64_t N, int64_t K, int bits) {
    if (!bits_ok(bits)) return 1;
    std::fesetround(FE_TONEAREST);
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        std::fesetround(FE_TONEAREST);
        float amax = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            const float a = std::fabs(w[n * K + k]);
            if (a > amax) amax = a;
        }
        const float sc = amax > 0.0f ? amax / qp : 1.0f;
        const float inv = 1.0f / sc;
        w_scale[n] = sc;
        for (int64_t k = 0; k < K; ++k) {
            const float r = std::nearbyintf(w[n * K + k] * inv);
            w_int[n * K + k] = (int8_t)std::fminf(std::fmaxf(r, -qn), qp);
        }
    }
    return 0;
}

// Integer GEMM of Eq. 2: acc[t, n] = sum_k X_int[t, k] * W_int[n, k], int32.
// Only rows [row_begin, row_end) of X_int are computed (the caller may sample).
int oracle_int_gemm(const int8_t* x_int, const int8_t* w_int, int32_t* acc, int64_t T, int64_t N, int64_t K,
                    int64_t row_begin, int64_t row_end) {
    if (row_begin < 0 || row_end > T || row_begin > row_end) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = row_begin; t < row_end; ++t) {
        for (int64_t n = 0; n < N; ++n) {
            int32_t a = 0;
            for (int64_t k = 0; k < K; ++k) a += (int32_t)x_int[t * K + k] * (int32_t)w_int[n * K + k];
            acc[t * N + n] = a;
        }
    }
    return 0;
}

// Brute-force twin with 64-bit products and sums (self-check of the above).
int oracle_int_gemm_i64(const int8_t* x_int, const int8_t* w_int, int64_t* acc, int64_t T, int64_t N, int64_t K) {
    for (int64_t t = 0; t < T; ++t)
        for (int64_t n = 0; n < N; ++n) {
            int64_t a = 0;
            for (int64_t k = 0; k < K; ++k) a += (int64_t)x_int[t * K + k] * (int64_t)w_int[n * K + k];
            acc[t * N + n] = a;
        }
    return 0;
}

// Dequantisation of Eq. 2: y = S_x * acc * S_w[n] (+ bias[n]), evaluated as
// fl32(acc) * fl32(s_x * s_w[n]), bias added in fp32, one narrowing at the end.
// y32 (optional) receives the fp32 value before narrowing.
int oracle_dequant(const int32_t* acc, const float* w_scale, float s_x, const uint16_t* bias, uint16_t* y,
                   float* y32, int64_t T, int64_t N, int dtype, int64_t row_begin, int64_t row_end) {
    if (row_begin < 0 || row_end > T || row_begin > row_end) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = row_begin; t < row_end; ++t) {
        for (int64_t n = 0; n < N; ++n) {
            const float sc = s_x * w_scale[n];
            float v = (float)acc[t * N + n] * sc;
            if (bias) v = v + widen(bias[n], dtype);
            if (y32) y32[t * N + n] = v;
            if (y) y[t * N + n] = narrow(v, dtype);
        }
    }
    return 0;
}

// The whole static W8A8 linear (Eq. 1 with the fixed factor, Eq. 2), rows
// [row_begin, row_end) of the output.  x_int_scratch is [T, K] int8.
int oracle_w8a8_linear(const uint16_t* x, const int8_t* w_int, const float* w_scale, float s_x,
                       const uint16_t* bias, uint16_t* y, float* y32, int32_t* acc, int8_t* x_int_scratch,
                       int64_t T, int64_t N, int64_t K, int dtype, int bits, int64_t row_begin, int64_t row_end) {
    if (row_begin < 0 || row_end > T || row_begin > row_end) return 1;
    int rc = oracle_quantize_act(x + row_begin * K, x_int_scratch + row_begin * K, row_end - row_begin, K,
                                 dtype, s_x, bits);
    if (rc) return rc;
    rc = oracle_int_gemm(x_int_scratch, w_int, acc, T, N, K, row_begin, row_end);
    if (rc) return rc;
    return oracle_dequant(acc, w_scale, s_x, bias, y, y32, T, N, dtype, row_begin, row_end);
}

// Eq. 3, grouped form for per-channel activation factors: the K axis is cut
// into G = K / group groups; x is quantized with s_x[k] (one factor per
// column), each group's int32 partial product is scaled by the group's factor
// and the partials are accumulated in fp32 in group order.  For the product to
// factor out of a group, every column of a group must share one factor: the
// caller passes s_group[G].
int oracle_w8a8_linear_grouped(const uint16_t* x, const int8_t* w_int, const float* w_scale,
                               const float* s_group, int64_t group, const uint16_t* bias, uint16_t* y,
                               float* y32, int64_t T, int64_t N, int64_t K, int dtype, int bits) {
    if (!bits_ok(bits) || group <= 0 || K % group != 0) return 1;
    std::fesetround(FE_TONEAREST);
    const int64_t G = K / group;
    const float qn = (float)(1 << (bits - 1));
    const float qp = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        std::fesetround(FE_TONEAREST);
        int8_t* row = new int8_t[K];
        for (int64_t k = 0; k < K; ++k) {
            const float inv = 1.0f / s_group[k / group];
            row[k] = (int8_t)quant1(widen(x[t * K + k], dtype), inv, qn, qp, 0).c;
        }
        for (int64_t n = 0; n < N; ++n) {
            float v = 0.0f;
            for (int64_t gi = 0; gi < G; ++gi) {
                int32_t a = 0;
                for (int64_t k = gi * group; k < (gi + 1) * group; ++k)
                    a += (int32_t)row[k] * (int32_t)w_int[n * K + k];
                v = v + (float)a * (s_group[gi] * w_scale[n]);
            }
            if (bias) v = v + widen(bias[n], dtype);
            if (y32) y32[t * N + n] = v;
            if (y) y[t * N + n] = narrow(v, dtype);
        }
        delete[] row;
    }
    return 0;
}

}  // extern "C"
