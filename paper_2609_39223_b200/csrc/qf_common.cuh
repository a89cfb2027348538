// Internal declarations shared by the translation units of libqf.so (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qf.h"

namespace qf {

constexpr int kNumSMs = 148;            // B200: 2 dies x 74 SMs
constexpr size_t kWsHeader = 256;       // workspace header: status word, amax slots, scale slots

// Layout of the 256-byte workspace header (32-bit words).
enum WsWord : int {
  kWsStatus = 0,      // qf_status_t written by a device-side wait that gave up
  kWsAmaxW = 4,       // max|W| as FP32 bits (unsigned-integer max is order preserving for x >= 0)
  kWsAmaxA = 5,       // max|X|
  kWsAmaxReport = 6,  // max|X| gathered for the caller's a_amax_out when the quantize pass over X does not derive a scale
  kWsScaleW = 8,      // derived NVFP4 tensor scale of W (float)
  kWsScaleA = 9,      // derived NVFP4 tensor scale of X (float)
  kWsGuessW = 10,     // the caller's guess of W's tensor scale (float bits), kept for the conditional second pass
  kWsClkCycles = 12,  // 64-bit: SM clock cycles the last matmul launch ran for (first CTA, start to end)
  kWsClkNanos = 14,   // 64-bit: the same interval in nanoseconds of the global timer; cycles / ns = SM clock in GHz
};

// ---- device helpers -----------------------------------------------------------------------

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// E2M1 pair: lo -> low nibble, hi -> high nibble; round to nearest even, saturate to +-6.
__device__ __forceinline__ uint32_t e2m1x2_encode(float lo, float hi) {
  return static_cast<uint32_t>(__nv_cvt_float2_to_fp4x2(make_float2(lo, hi), __NV_E2M1, cudaRoundNearest)) & 0xFFu;
}

// packed E2M1 byte -> the two represented values as floats (exact)
__device__ __forceinline__ float2 e2m1x2_decode(uint32_t byte) {
  __half2_raw h = __nv_cvt_fp4x2_to_halfraw2(static_cast<__nv_fp4x2_storage_t>(byte), __NV_E2M1);
  return __half22float2(*reinterpret_cast<__half2*>(&h));
}

// non-negative float -> E4M3 code (round to nearest even, saturate to 448)
__device__ __forceinline__ uint32_t e4m3_encode(float q) {
  return static_cast<uint32_t>(__nv_cvt_float_to_fp8(q, __NV_SATFINITE, __NV_E4M3)) & 0x7Fu;
}

// E4M3 code (sign bit clear) -> float, exact for normals and subnormals: the 7 code bits placed at
// the top of an FP32 exponent/mantissa give value * 2^-120.
__device__ __forceinline__ float e4m3_decode(uint32_t code) {
  return __fmul_rn(__uint_as_float(code << 20), 0x1p120f);
}

// E8M0 code (p + 127) -> 2^p (code 0 = 2^-127, an FP32 subnormal) and 2^-p.
__device__ __forceinline__ float e8m0_scale(uint32_t code) {
  return __uint_as_float(code ? (code << 23) : 0x00400000u);
}
__device__ __forceinline__ float e8m0_inv_scale(uint32_t code) { return __uint_as_float((254u - code) << 23); }

// MXFP4 block-scale code from the block's max |x| given as BF16 bits (sign clear):
// p = floor(log2 amax) - 2 clamped to [-127, 127]; code = p + 127 = biased exponent - 2.
// noclip: the smallest p with amax <= 6 * 2^p instead. amax * 2^-p = 4 * (1 + mantissa / 128) under the
// first rule, so that is one more exactly when the mantissa exceeds 64 (and the first rule did not clamp:
// below biased exponent 2 the ratio is under 4 already).
__device__ __forceinline__ uint32_t mxfp4_scale_code(uint32_t amax_bf16_bits, bool noclip) {
  const int e = static_cast<int>(amax_bf16_bits >> 7);
  const int bump = (noclip && e >= 2 && (amax_bf16_bits & 0x7Fu) > 0x40u) ? 1 : 0;
  return static_cast<uint32_t>(max(e - 2, 0) + bump);
}

__device__ __forceinline__ float2 splat(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 unpack2(uint32_t w) { return make_float2(bf16_lo(w), bf16_hi(w)); }
__device__ __forceinline__ uint32_t bf2_bits(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ __nv_bfloat162 bits_bf2(uint32_t v) { return *reinterpret_cast<__nv_bfloat162*>(&v); }

// max |x| over the 8 BF16 values of one 16-byte chunk, as BF16 bits (sign clear)
__device__ __forceinline__ uint32_t chunk8_amax_bits(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
  const __nv_bfloat162 a = __hmax2(__habs2(bits_bf2(w0)), __habs2(bits_bf2(w1)));
  const __nv_bfloat162 b = __hmax2(__habs2(bits_bf2(w2)), __habs2(bits_bf2(w3)));
  const uint32_t m = bf2_bits(__hmax2(a, b));
  return max(m & 0xFFFFu, m >> 16);
}

// MXFP4 quantize-dequantize of one packed BF16 pair given its block's max |x| (BF16 bits):
// x_hat = 2^p * E2M1(x * 2^-p), p = floor(log2 amax) - 2 (Eq. mxfp4-dequant). Every product is exact.
__device__ __forceinline__ uint32_t mxfp4_qdq_pair(uint32_t w, float2 inv, float2 sc, uint32_t keep) {
  const float2 v = __fmul2_rn(unpack2(w), inv);
  const uint32_t byte = e2m1x2_encode(v.x, v.y) & keep;
  const float2 o = __fmul2_rn(e2m1x2_decode(byte), sc);
  return pack_bf16x2(o.x, o.y);
}

// The same MXFP4 rounding done entirely in packed BF16 arithmetic (no format conversions, which run
// on a narrow pipe): for |x| in the binade [2^e, 2^(e+1)) the E2M1 grid scaled by 2^p has spacing
// 2^(e-1) (one mantissa bit), and below 2^p it has the spacing of the first binade, 2^(p-1). Adding
// and subtracting 1.5 * 2^(e+6) in BF16 (8 significant bits) therefore rounds |x| to that spacing with
// round-to-nearest-even, and "even multiple of the spacing" coincides with "even E2M1 code"; the
// result is then clamped to 6 * 2^p and the sign of x restored. `one2` is 2^p and `six2` 6 * 2^p as
// packed BF16 pairs. Valid while all of these are normal BF16 numbers: scale code in [8, 240].
__device__ __forceinline__ bool mxfp4_bf16_path_ok(uint32_t scale_code) { return scale_code >= 8u && scale_code <= 240u; }
__device__ __forceinline__ uint32_t mxfp4_one2(uint32_t scale_code) { return (scale_code << 7) | (scale_code << 23); }
__device__ __forceinline__ uint32_t mxfp4_six2(uint32_t scale_code) { return mxfp4_one2(scale_code + 2u) | 0x00400040u; }
__device__ __forceinline__ uint32_t mxfp4_qdq_pair_bf16(uint32_t w, uint32_t one2, uint32_t six2) {
  const uint32_t a = w & 0x7FFF7FFFu;
  const uint32_t t = bf2_bits(__hmax2(bits_bf2(a), bits_bf2(one2)));
  const uint32_t magic = (t & 0x7F807F80u) + 0x03400340u;            // 1.5 * 2^(e+6) per lane
  __nv_bfloat162 r = __hadd2(bits_bf2(a), bits_bf2(magic));           // one rounding: nearest multiple of the spacing
  r = __hsub2(r, bits_bf2(magic));                                    // exact
  r = __hmin2(r, bits_bf2(six2));
  return bf2_bits(r) | (w & 0x80008000u);
}

// ---- host-side launchers implemented in the .cu files ---------------------------------------

// NVFP4 with a speculated tensor scale: the first pass quantizes with the caller's guess while it accumulates the true
// maximum; the second pass derives the scale from that maximum and does nothing when it equals the guess.
struct Nvfp4Speculation {
  uint32_t* amax_accum;          // where the maximum of everything read is accumulated (FP32 bits); also used on its own,
                                 // by either FP4 format, to report max|x| from the quantize pass
  uint32_t* guess_out;           // first pass: receives the bits of the scale it used
  const uint32_t* skip_guess;    // second pass: leave at once if the derived scale has these bits
};

struct QdqArgs {
  int fmt;
  const void* in;
  int64_t rows, cols;
  void* out;
  void* codes;
  void* scales;
  const float* tscale_in;        // NVFP4: tensor scale to read (device), or
  const uint32_t* amax_bits;     // NVFP4: tensor amax as FP32 bits (device) to derive it from
  float* tscale_out;             // NVFP4: where the derived scale is written (nullable)
  bool reverse;                  // walk the tensor back to front (after an amax pass: L2 holds the tail)
  bool mxfp4_noclip;             // MXFP4: smallest block exponent without saturation (QF_MXFP4_NO_CLIP)
  int groups;                    // NVFP4: > 1 = that many equal tensors back to back, each with its own tensor scale
  Nvfp4Speculation spec;         // all null unless launch_qdq_nvfp4_speculative() fills it in
  // LoRA merge ahead of the quantizer (lora_rank > 0): the input is W + lora_scale * B A, formed on the fly
  const void* lora_B;            // [rows, rank] BF16
  const void* lora_A;            // [rank, cols] BF16
  int lora_rank;
  float lora_scale;
};

// Many tensors in one call (host arrays of device pointers and shapes); see launch_qdq_batched in qf_qdq.cu.
struct QdqBatchArgs {
  int fmt;
  int n;
  const void* const* in;
  const int64_t* rows;
  const int64_t* cols;
  void* const* out;              // each array nullable as a whole, and entry by entry
  void* const* codes;
  void* const* scales;
  float* tscales;                // NVFP4: device float[n], read (given / guesses) or written (derived)
  bool given, speculative, noclip;
  uint32_t* ws_words;            // NVFP4 without given scales: device uint32[2n], zeroed on the stream beforehand
};
cudaError_t launch_qdq_batched(const QdqBatchArgs& a, cudaStream_t st);

cudaError_t launch_amax(const void* in, int64_t n, uint32_t* amax_bits, cudaStream_t st);
cudaError_t launch_qdq_nvfp4_speculative(const QdqArgs& a, uint32_t* header, int amax_word, int guess_word, cudaStream_t st);
cudaError_t launch_amax_to_float(const uint32_t* amax_bits, float* out, cudaStream_t st);
cudaError_t launch_amax_to_scale(const uint32_t* amax_bits, float* scale, cudaStream_t st);
cudaError_t launch_qdq(const QdqArgs& a, cudaStream_t st);
cudaError_t launch_qdq_nvfp4_derive(const QdqArgs& a, uint32_t* header, int amax_word, cudaStream_t st);
cudaError_t launch_dequant(int fmt, const void* codes, const void* scales, const float* tscale, int64_t rows,
                           int64_t cols, void* out, cudaStream_t st);
cudaError_t launch_selftest_div(const float* xs, int64_t nx, const float* ys, int64_t ny, unsigned long long* mismatches,
                                cudaStream_t st);
cudaError_t launch_selftest_mxfp4_bf16(unsigned long long* mismatches, cudaStream_t st);
cudaError_t launch_selftest_cvt(const float* in, int64_t n, uint8_t* e2m1, uint8_t* e4m3, cudaStream_t st);

// C[Mo, No] (+)= sum_c A(m, c) * B(n, c). Operand storage: K-major = [rows, contraction] row-major,
// MN-major = [contraction, rows] row-major. ld* are row pitches in elements. Optional grouping:
// see qf_gemm.cu.
struct GemmArgs {
  const void* A;
  const void* B;
  void* C;
  int64_t Mo, No, Kc;            // output rows, output cols, contraction length
  int64_t lda, ldb, ldc;
  bool a_mn_major, b_mn_major;
  int c_dtype;                   // qf_dtype_t
  bool accumulate;
  // grouped modes (0 = plain)
  int group_mode;                // 1: rows of A/C segmented, B per group [G, No, Kc] (fwd / dgrad)
                                 // 2: contraction segmented, C per group [G, Mo, No] (wgrad)
  const int32_t* group_offsets;  // device int32[G+1]
  int G;
  int64_t b_group_stride;        // elements between consecutive groups of B (mode 1)
  int64_t c_group_stride;        // elements between consecutive groups of C (mode 2)
  int64_t rows_padded;           // mode 1: total rows of A / C; mode 2: total contraction rows
  uint32_t* status_word;         // device word receiving QF_ERR_TIMEOUT if a wait expires
  bool fuse_a_mxfp4, fuse_b_mxfp4;   // apply the MXFP4 quantize-dequantize to the staged tiles inside the kernel
  bool mxfp4_noclip;                 // scale rule of that in-kernel quantizer (QF_MXFP4_NO_CLIP)
};

cudaError_t launch_pack_q4k(const void* codes, const void* scales, int64_t nsb, void* records, bool unpack, void* codes_out,
                            void* scales_out, cudaStream_t st);
cudaError_t launch_swizzle_scales(const void* scales, int64_t rows, int64_t nblk, void* out, bool unswizzle, cudaStream_t st);
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st);

// Operands of the native block-scaled FP4 product (qf_fp4_gemm.cu): codes and block scales as the quantizer emits them.
struct Fp4GemmArgs {
  int fmt;                           // QF_FMT_MXFP4 or QF_FMT_NVFP4
  const void* a_codes;               // [M, K/2] bytes
  const void* a_scales;              // [M, K/block] bytes
  const void* b_codes;               // [N, K/2]
  const void* b_scales;              // [N, K/block]
  const float* a_tscale;             // NVFP4: device tensor scales
  const float* b_tscale;
  float* Y;                          // [M, N] FP32
  int64_t M, N, K;
  bool scales_tiled;                 // scales in the tiled engine layout (qf_pack, QF_LAYOUT_FP4_SWIZZLED_SCALES)
  uint32_t* status_word;
};
cudaError_t launch_fp4_native(const Fp4GemmArgs& a, cudaStream_t st);
bool gemm_can_fuse(const GemmArgs& a);
cudaError_t launch_selftest_timeout(uint32_t* status, long long limit_cycles, int* gave_up, cudaStream_t st);

}  // namespace qf
