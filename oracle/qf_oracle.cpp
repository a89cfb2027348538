// CPU oracle for the fake-quantization hot path (NVFP4 / MXFP4 / Q4_K quantize-dequantize,
// the BF16 matmul on fake-quantized operands and its straight-through backward).
//
// THIS IS TEST INFRASTRUCTURE. It is deliberately plain and slow: one scalar loop per step,
// steps in the order the paper's Section 3.2 gives them, no blocking, no fusion, no vector code.
// Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it; the CUDA
// library never does, and the two share no source.
//
// Arithmetic contract (the paper fixes formats, not operation order, so the order is fixed here):
// every FP32 operation below is a single IEEE-754 binary32 operation with round-to-nearest-even.
// Build with -ffp-contract=off and without -ffast-math so the compiler neither fuses nor
// reassociates. BF16 inputs widen to FP32 exactly. Matmuls accumulate in FP64.
//
// Parity pins (tests/test_oracle_*.py): E2M1 value set (Eq. e2m1-values), threshold table and
// ml_dtypes casts for the 4- and 8-bit float encoders, numpy.float16 for the FP16 rounding,
// gguf's Q4_K reader for the record layout and dequantization (Eq. q4k-dequant), closed forms,
// sign / power-of-two invariances, idempotence, brute-force nearest-grid search on tiny blocks.
// "parity unpinned": the *choice* of the Q4_K quantizer rule (plain min/max affine rounding); the
// paper gives only the format and the dequantization formula for Q4_K.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <cstddef>
#include <vector>
#include <omp.h>

namespace {

// ---------------------------------------------------------------------------------------------
// Scalar number formats
// ---------------------------------------------------------------------------------------------

inline float bf16_to_f32(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

// FP32 -> BF16, round to nearest, ties to even. Finite inputs only (precondition of the path).
inline uint16_t f32_to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

// FP32 -> FP16 (IEEE binary16, subnormals kept), round to nearest even, saturating at 65504.
inline uint16_t f32_to_fp16_sat(float f) {
    if (f > 65504.0f) f = 65504.0f;
    if (f < -65504.0f) f = -65504.0f;
    _Float16 h = static_cast<_Float16>(f);
    uint16_t b;
    std::memcpy(&b, &h, 2);
    return b;
}

inline float fp16_to_f32(uint16_t b) {
    _Float16 h;
    std::memcpy(&h, &b, 2);
    return static_cast<float>(h);
}

// E2M1 (Eq. e2m1-values): sign bit 3, magnitudes indexed by the low three bits.
const double kE2M1Mag[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

inline float e2m1_value(uint8_t code) {
    float m = static_cast<float>(kE2M1Mag[code & 7]);
    return (code & 8) ? -m : m;
}

// Nearest representable magnitude; a tie goes to the even code; anything above 6 lands on 6.
// The sign bit is copied from v even when the magnitude rounds to zero.
inline uint8_t e2m1_encode(float v) {
    double a = std::fabs(static_cast<double>(v));
    if (a > 6.0) a = 6.0;      // saturate first: for huge |v| every distance |a - grid| rounds to the same double
    int best = 0;
    double best_d = std::fabs(a - kE2M1Mag[0]);
    for (int c = 1; c < 8; ++c) {
        double d = std::fabs(a - kE2M1Mag[c]);
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    uint8_t sign = std::signbit(v) ? 8 : 0;
    return static_cast<uint8_t>(sign | best);
}

// E4M3 "fn" (bias 7, no infinities, 0x7F is NaN), non-negative half: codes 0x00..0x7E.
inline double e4m3_value_d(uint8_t code) {
    int e = (code >> 3) & 0xF;
    int m = code & 7;
    if (e == 0) return std::ldexp(static_cast<double>(m), -9);        // subnormal: m * 2^-9
    return std::ldexp(1.0 + m / 8.0, e - 7);
}

inline float e4m3_value(uint8_t code) { return static_cast<float>(e4m3_value_d(code)); }

// Clamp to 448, then the nearest of the 127 finite codes, ties to the even code.
inline uint8_t e4m3_encode(float q) {
    double a = static_cast<double>(q);
    if (a > 448.0) a = 448.0;
    if (!(a > 0.0)) return 0;
    int best = 0;
    double best_d = a;
    for (int c = 1; c <= 0x7E; ++c) {
        double d = std::fabs(a - e4m3_value_d(static_cast<uint8_t>(c)));
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    return static_cast<uint8_t>(best);
}

// 2^p for integer p in [-127, 127], exact in FP32 (2^-127 is an FP32 subnormal).
inline float exp2i(int p) { return std::ldexp(1.0f, p); }

// ---------------------------------------------------------------------------------------------
// NVFP4  (Eq. nvfp4, Eq. nvfp4-dequant): E2M1 codes, blocks of 16, E4M3 block scale, FP32 tensor
// scale. x_hat_i = s_FP32 * s_E4M3,b * C_i.
// ---------------------------------------------------------------------------------------------

float tensor_amax(const uint16_t* x, int64_t n) {
    float amax = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float a = std::fabs(bf16_to_f32(x[i]));
        if (a > amax) amax = a;
    }
    return amax;
}

void nvfp4_row(const uint16_t* x, int64_t cols, float s_t, uint16_t* out, uint8_t* codes, uint8_t* scales) {
    const int B = 16;
    for (int64_t b = 0; b < cols / B; ++b) {
        const uint16_t* xb = x + b * B;
        float amax_b = 0.0f;
        for (int i = 0; i < B; ++i) {
            float a = std::fabs(bf16_to_f32(xb[i]));
            if (a > amax_b) amax_b = a;
        }
        float denom = 6.0f * s_t;
        float q = amax_b / denom;
        uint8_t sb_code = e4m3_encode(q);
        float sb = e4m3_value(sb_code);
        float S = s_t * sb;
        if (scales) scales[b] = sb_code;
        uint8_t c[B];
        for (int i = 0; i < B; ++i) {
            float xv = bf16_to_f32(xb[i]);
            float xhat;
            if (S == 0.0f) {
                c[i] = 0;
                xhat = 0.0f;
            } else {
                float v = xv / S;
                c[i] = e2m1_encode(v);
                float inner = sb * e2m1_value(c[i]);
                xhat = inner * s_t;
            }
            if (out) out[b * B + i] = f32_to_bf16(xhat);
        }
        if (codes)
            for (int i = 0; i < B; i += 2) codes[(b * B + i) / 2] = static_cast<uint8_t>(c[i] | (c[i + 1] << 4));
    }
}

// ---------------------------------------------------------------------------------------------
// MXFP4 (Eq. mxfp4, Eq. mxfp4-dequant): E2M1 codes, blocks of 32, power-of-two E8M0 block scale.
// x_hat_i = 2^{p_b} * C_i.  Scale rule: p = floor(log2 amax) - 2, clamped to [-127, 127]; block
// maxima in (6, 8) * 2^p then saturate at 6 * 2^p. The paper does not fix the rule; the variant
// `noclip` takes instead the smallest p in [-127, 127] with amax <= 6 * 2^p, so nothing saturates.
// ---------------------------------------------------------------------------------------------

void mxfp4_row(const uint16_t* x, int64_t cols, uint16_t* out, uint8_t* codes, uint8_t* scales, bool noclip) {
    const int B = 32;
    for (int64_t b = 0; b < cols / B; ++b) {
        const uint16_t* xb = x + b * B;
        float amax_b = 0.0f;
        for (int i = 0; i < B; ++i) {
            float a = std::fabs(bf16_to_f32(xb[i]));
            if (a > amax_b) amax_b = a;
        }
        uint8_t c[B];
        int p = -127;
        if (amax_b == 0.0f) {
            for (int i = 0; i < B; ++i) c[i] = 0;
        } else {
            int e;
            std::frexp(amax_b, &e);          // amax_b = f * 2^e, f in [0.5, 1)  =>  floor(log2) = e - 1
            p = (e - 1) - 2;
            if (p < -127) p = -127;
            if (p > 127) p = 127;
            if (noclip) {
                p = -127;
                while (p < 127 && static_cast<double>(amax_b) > 6.0 * std::ldexp(1.0, p)) ++p;
            }
            float inv = exp2i(-p);
            for (int i = 0; i < B; ++i) c[i] = e2m1_encode(bf16_to_f32(xb[i]) * inv);
        }
        if (scales) scales[b] = static_cast<uint8_t>(p + 127);
        float sc = exp2i(p);
        for (int i = 0; i < B; ++i) {
            float xhat = (amax_b == 0.0f) ? 0.0f : sc * e2m1_value(c[i]);
            if (out) out[b * B + i] = f32_to_bf16(xhat);
        }
        if (codes)
            for (int i = 0; i < B; i += 2) codes[(b * B + i) / 2] = static_cast<uint8_t>(c[i] | (c[i + 1] << 4));
    }
}

// ---------------------------------------------------------------------------------------------
// Q4_K (Eq. q4k, Eq. q4k-dequant): 256-weight super-block = 8 sub-blocks of 32, unsigned 4-bit
// codes, 6-bit sub-block scale s6 and offset m6 under FP16 super-block factors d and dmin.
// x_hat_i = (d * s6_b) * C_i - (dmin * m6_b).  Quantizer rule: min/max affine, round to nearest.
// ---------------------------------------------------------------------------------------------

inline float rint_even(float v) { return std::nearbyintf(v); }   // default rounding mode = nearest even

void q4k_row(const uint16_t* x, int64_t cols, uint16_t* out, uint8_t* codes, uint8_t* scales) {
    for (int64_t sb = 0; sb < cols / 256; ++sb) {
        const uint16_t* xs = x + sb * 256;
        float sc[8], off[8];
        float max_sc = 0.0f, max_off = 0.0f;
        for (int b = 0; b < 8; ++b) {
            float lo = 0.0f, hi = bf16_to_f32(xs[b * 32]);
            for (int i = 0; i < 32; ++i) {
                float v = bf16_to_f32(xs[b * 32 + i]);
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            sc[b] = (hi - lo) / 15.0f;
            off[b] = -lo;
            if (sc[b] > max_sc) max_sc = sc[b];
            if (off[b] > max_off) max_off = off[b];
        }
        uint16_t d_h = f32_to_fp16_sat(max_sc / 63.0f);
        uint16_t dmin_h = f32_to_fp16_sat(max_off / 63.0f);
        float d = fp16_to_f32(d_h), dmin = fp16_to_f32(dmin_h);
        int s6[8], m6[8];
        for (int b = 0; b < 8; ++b) {
            float s = (d == 0.0f) ? 0.0f : rint_even(sc[b] / d);
            float m = (dmin == 0.0f) ? 0.0f : rint_even(off[b] / dmin);
            s6[b] = static_cast<int>(std::fmin(std::fmax(s, 0.0f), 63.0f));
            m6[b] = static_cast<int>(std::fmin(std::fmax(m, 0.0f), 63.0f));
        }
        uint8_t c[256];
        for (int b = 0; b < 8; ++b) {
            float es = d * static_cast<float>(s6[b]);
            float em = dmin * static_cast<float>(m6[b]);
            for (int i = 0; i < 32; ++i) {
                float xv = bf16_to_f32(xs[b * 32 + i]);
                float cf = 0.0f;
                if (es > 0.0f) {
                    float t = (xv + em) / es;
                    cf = std::fmin(std::fmax(rint_even(t), 0.0f), 15.0f);
                }
                c[b * 32 + i] = static_cast<uint8_t>(cf);
                float prod = es * cf;
                float xhat = prod - em;
                if (out) out[sb * 256 + b * 32 + i] = f32_to_bf16(xhat);
            }
        }
        if (scales) {
            uint8_t* r = scales + sb * 16;
            std::memcpy(r, &d_h, 2);
            std::memcpy(r + 2, &dmin_h, 2);
            uint8_t* pk = r + 4;
            for (int j = 0; j < 4; ++j) {
                pk[j]     = static_cast<uint8_t>((s6[j] & 63) | ((s6[j + 4] >> 4) << 6));
                pk[j + 4] = static_cast<uint8_t>((m6[j] & 63) | ((m6[j + 4] >> 4) << 6));
                pk[j + 8] = static_cast<uint8_t>((s6[j + 4] & 15) | ((m6[j + 4] & 15) << 4));
            }
        }
        if (codes) {
            uint8_t* q = codes + sb * 128;
            for (int j = 0; j < 4; ++j)
                for (int l = 0; l < 32; ++l)
                    q[j * 32 + l] = static_cast<uint8_t>(c[j * 64 + l] | (c[j * 64 + 32 + l] << 4));
        }
    }
}

void q4k_unpack_meta(const uint8_t* r, float* d, float* dmin, int s6[8], int m6[8]) {
    uint16_t d_h, dmin_h;
    std::memcpy(&d_h, r, 2);
    std::memcpy(&dmin_h, r + 2, 2);
    *d = fp16_to_f32(d_h);
    *dmin = fp16_to_f32(dmin_h);
    const uint8_t* pk = r + 4;
    for (int j = 0; j < 4; ++j) {
        s6[j] = pk[j] & 63;
        m6[j] = pk[j + 4] & 63;
        s6[j + 4] = (pk[j + 8] & 15) | ((pk[j] >> 6) << 4);
        m6[j + 4] = (pk[j + 8] >> 4) | ((pk[j + 4] >> 6) << 4);
    }
}

}  // namespace

extern "C" {

enum { ORC_FMT_NONE = 0, ORC_FMT_NVFP4 = 1, ORC_FMT_MXFP4 = 2, ORC_FMT_Q4_K = 3 };

// Scalar helpers, exported so the tests can pin each one on its own.
uint8_t orc_e2m1_encode(float v) { return e2m1_encode(v); }
float orc_e2m1_value(uint8_t c) { return e2m1_value(c); }
uint8_t orc_e4m3_encode(float q) { return e4m3_encode(q); }
float orc_e4m3_value(uint8_t c) { return e4m3_value(c); }
uint16_t orc_bf16_round(float f) { return f32_to_bf16(f); }
uint16_t orc_fp16_round_sat(float f) { return f32_to_fp16_sat(f); }
float orc_fp16_value(uint16_t h) { return fp16_to_f32(h); }
int orc_num_threads(void) { return omp_get_max_threads(); }

float orc_amax(const uint16_t* x, int64_t n) { return tensor_amax(x, n); }

// Quantize-dequantize of a row-major BF16 [rows, cols] tensor, blocks along cols.
// out / codes / scales may be null. NVFP4: *tensor_scale is read when tscale_given != 0, otherwise
// derived from the tensor's absolute maximum and written back. mxfp4_noclip != 0 selects the MXFP4
// scale rule without saturation. Returns 0, or -1 on a bad shape.
int orc_qdq(int fmt, const uint16_t* in, int64_t rows, int64_t cols, uint16_t* out, uint8_t* codes,
            uint8_t* scales, float* tensor_scale, int tscale_given, int mxfp4_noclip) {
    int block = fmt == ORC_FMT_NVFP4 ? 16 : fmt == ORC_FMT_MXFP4 ? 32 : fmt == ORC_FMT_Q4_K ? 256 : 0;
    if (block == 0 || rows < 0 || cols < 0 || cols % block) return -1;
    float s_t = 1.0f;
    if (fmt == ORC_FMT_NVFP4) {
        if (tscale_given) {
            s_t = *tensor_scale;
        } else {
            float amax_t = tensor_amax(in, rows * cols);
            s_t = (amax_t == 0.0f) ? 1.0f : amax_t / 2688.0f;     // 2688 = 6 * 448
            if (tensor_scale) *tensor_scale = s_t;
        }
    }
    const int64_t code_stride = cols / 2;
    const int64_t scale_stride = fmt == ORC_FMT_Q4_K ? (cols / 256) * 16 : cols / block;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const uint16_t* x = in + r * cols;
        uint16_t* o = out ? out + r * cols : nullptr;
        uint8_t* c = codes ? codes + r * code_stride : nullptr;
        uint8_t* s = scales ? scales + r * scale_stride : nullptr;
        if (fmt == ORC_FMT_NVFP4) nvfp4_row(x, cols, s_t, o, c, s);
        else if (fmt == ORC_FMT_MXFP4) mxfp4_row(x, cols, o, c, s, mxfp4_noclip != 0);
        else q4k_row(x, cols, o, c, s);
    }
    return 0;
}

// The inverse half of the quantizer interface: codes + metadata -> BF16.
int orc_dequant(int fmt, const uint8_t* codes, const uint8_t* scales, const float* tensor_scale,
                int64_t rows, int64_t cols, uint16_t* out) {
    int block = fmt == ORC_FMT_NVFP4 ? 16 : fmt == ORC_FMT_MXFP4 ? 32 : fmt == ORC_FMT_Q4_K ? 256 : 0;
    if (block == 0 || cols % block) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t k = 0; k < cols; ++k) {
            float xhat;
            if (fmt == ORC_FMT_Q4_K) {
                int64_t sb = k / 256;
                int within = static_cast<int>(k % 256);
                float d, dmin;
                int s6[8], m6[8];
                q4k_unpack_meta(scales + (r * (cols / 256) + sb) * 16, &d, &dmin, s6, m6);
                int b = within / 32;
                int j = within / 64, l = within % 32;
                uint8_t byte = codes[(r * (cols / 256) + sb) * 128 + j * 32 + l];
                int c = ((within % 64) < 32) ? (byte & 15) : (byte >> 4);
                float es = d * static_cast<float>(s6[b]);
                float em = dmin * static_cast<float>(m6[b]);
                float prod = es * static_cast<float>(c);
                xhat = prod - em;
            } else {
                uint8_t byte = codes[(r * cols + k) / 2];
                uint8_t c = (k & 1) ? (byte >> 4) : (byte & 15);
                uint8_t sc = scales[r * (cols / block) + k / block];
                if (fmt == ORC_FMT_NVFP4) {
                    float inner = e4m3_value(sc) * e2m1_value(c);
                    xhat = inner * (*tensor_scale);
                } else {
                    xhat = exp2i(static_cast<int>(sc) - 127) * e2m1_value(c);
                }
            }
            out[r * cols + k] = f32_to_bf16(xhat);
        }
    }
    return 0;
}

// LoRA merge ahead of the quantizer (Eq. qad-lora): merged = bf16(W + scale * B A), W [rows, cols],
// B [rows, rank], A [rank, cols]. FP32 accumulation in a fixed order, one fused multiply-add per rank
// step (std::fmaf rounds once), then one rounding to BF16.
void orc_lora_merge(const uint16_t* W, const uint16_t* B, const uint16_t* A, int64_t rows, int64_t cols, int64_t rank,
                    float scale, uint16_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < rows; ++n)
    for (int64_t k = 0; k < cols; ++k) {
      float acc = bf16_to_f32(W[n * cols + k]);
      for (int64_t r = 0; r < rank; ++r) {
        const float b = scale * bf16_to_f32(B[n * rank + r]);
        acc = std::fmaf(b, bf16_to_f32(A[r * cols + k]), acc);
      }
      out[n * cols + k] = f32_to_bf16(acc);
    }
}

// Y[m,n] = sum_k Xh[m,k] * Wh[n,k]   (Eq. fakequant: O = W_hat A_hat, written for row-major
// activations [M,K] and weights [N,K]). BF16 operands, FP64 accumulation, FP32 result.
void orc_matmul_fwd(const uint16_t* Xh, const uint16_t* Wh, int64_t M, int64_t N, int64_t K, float* Y) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += static_cast<double>(bf16_to_f32(Xh[m * K + k])) * static_cast<double>(bf16_to_f32(Wh[n * K + k]));
            Y[m * N + n] = static_cast<float>(acc);
        }
}

// dX[m,k] = sum_n dY[m,n] * Wh[n,k]   (Eq. activation-ste: dL/dA = W_hat^T dL/dO).
void orc_matmul_dgrad(const uint16_t* dY, const uint16_t* Wh, int64_t M, int64_t N, int64_t K, float* dX) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        std::vector<double> acc(static_cast<size_t>(K), 0.0);
        for (int64_t n = 0; n < N; ++n) {
            double g = static_cast<double>(bf16_to_f32(dY[m * N + n]));
            for (int64_t k = 0; k < K; ++k) acc[k] += g * static_cast<double>(bf16_to_f32(Wh[n * K + k]));
        }
        for (int64_t k = 0; k < K; ++k) dX[m * K + k] = static_cast<float>(acc[k]);
    }
}

// dW[n,k] = sum_m dY[m,n] * Xh[m,k]   (Eq. ste: dL/dW = dL/dO A_hat^T), for the output rows
// n_idx[0..n_rows) only (pass n_idx = null for all N rows). dW_out is [n_rows, K].
void orc_matmul_wgrad(const uint16_t* dY, const uint16_t* Xh, int64_t M, int64_t N, int64_t K,
                      const int64_t* n_idx, int64_t n_rows, float* dW_out) {
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n_rows; ++j) {
        int64_t n = n_idx ? n_idx[j] : j;
        std::vector<double> acc(static_cast<size_t>(K), 0.0);
        for (int64_t m = 0; m < M; ++m) {
            double g = static_cast<double>(bf16_to_f32(dY[m * N + n]));
            for (int64_t k = 0; k < K; ++k) acc[k] += g * static_cast<double>(bf16_to_f32(Xh[m * K + k]));
        }
        for (int64_t k = 0; k < K; ++k) dW_out[j * K + k] = static_cast<float>(acc[k]);
    }
}

}  // extern "C"
