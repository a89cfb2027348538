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
  kWsTileSync = 24,   // 16 words: arrival counters of the matmul launches of one call (tile-start rendezvous)
  kWsTileSyncCount = 16,
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

// ---------------------------------------------------------------------------------------------
// Exact division without the per-element IEEE divide sequence.
//
// The formats need v = x / S (NVFP4) and t = (x + em) / es (Q4_K) as correctly rounded FP32
// quotients, because the quotient decides a code. One divisor serves a whole block, so its correctly
// rounded reciprocal rc = RN(1/y) is computed once and every quotient is then
//     q0 = RN(x * rc);  q1 = RN(q0 + rc * (x - y*q0))          (x - y*q0 is exact in a fused multiply-add)
// (two elements per instruction). With an exactly rounded reciprocal and no overflow / underflow in
// the residual, q1 is the correctly rounded quotient (Markstein's division theorem); the range guard
// below keeps operands where that holds and the caller falls back to the IEEE divide otherwise.
// qf_selftest_div compares it with the IEEE divide (tens of billions of pairs, including every BF16
// numerator and divisors with an all-ones significand, without a difference).
//
// The residual is formed rounding toward minus infinity. Being exact, its value does not depend on the
// rounding mode, but its sign when it is zero does: an exactly cancelling sum is -0 in that mode, so the
// correction step adds -0 to q0 and leaves q0's sign alone. That makes x = -0 come out as -0, like the
// IEEE quotient (with round-to-nearest the residual would be +0 and (+0) + (-0) = +0).
// ---------------------------------------------------------------------------------------------

#ifndef QF_DIV_STEPS
#define QF_DIV_STEPS 1      // residual corrections after the first product (1 suffices with an exact reciprocal)
#endif


__device__ __forceinline__ float2 div2_fast(float2 x, float y, float rc) {
  const float2 ny = splat(-y), r = splat(rc);
  float2 q = __fmul2_rn(x, r);
  q = __ffma2_rn(__ffma2_rd(ny, q, x), r, q);
#if QF_DIV_STEPS > 1
  q = __ffma2_rn(__ffma2_rd(ny, q, x), r, q);
#endif
  return q;
}
__device__ __forceinline__ float div1_fast(float x, float y, float rc) {
  float q = __fmul_rn(x, rc);
  q = __fmaf_rn(__fmaf_rd(-y, q, x), rc, q);
#if QF_DIV_STEPS > 1
  q = __fmaf_rn(__fmaf_rd(-y, q, x), rc, q);
#endif
  return q;
}
// divisor magnitudes for which the iteration above is used
__device__ __forceinline__ bool div_safe(float y) { return y >= 0x1p-60f && y <= 0x1p60f; }

// NVFP4 per-tensor constants derived from the tensor scale: the divisor 6 * s_t of the block-scale quotient and its
// exactly rounded reciprocal (when the divisor lies in the range where the reciprocal-based division is exact).
struct Nvfp4Tensor {
  float s_t, denom, rc_denom;
  bool denom_safe;
};
__device__ __forceinline__ Nvfp4Tensor nvfp4_tensor(float s_t) {
  Nvfp4Tensor t;
  t.s_t = s_t;
  t.denom = __fmul_rn(6.0f, s_t);
  t.denom_safe = div_safe(t.denom);
  t.rc_denom = t.denom_safe ? __frcp_rn(t.denom) : 0.0f;
  return t;
}

// NVFP4 quantize-dequantize of NW packed BF16 pairs that belong to one 16-element block whose max |x| is amax_b
// (Eq. nvfp4, Eq. nvfp4-dequant): block scale sb = E4M3(min(amax_b / (6 s_t), 448)), S = s_t * sb, codes from
// x / S (the correctly rounded quotient by either route), x_hat = bf16((sb * value(code)) * s_t). `scale_code`
// receives the E4M3 code and `codes` one byte per pair (low nibble = first element). Both division routes give the
// IEEE quotient, so the choice between them never changes a result.
template <int NW>
__device__ __forceinline__ void nvfp4_block_words(const uint32_t (&w)[NW], float amax_b, const Nvfp4Tensor nt, uint32_t (&xhat)[NW],
                                                  uint32_t (&codes)[NW], uint32_t& scale_code) {
  // A supplied tensor scale can be far too small for a block: the quotient then exceeds every E4M3 value and may
  // even overflow FP32, which the reciprocal-based form does not survive (inf - inf). 512 * denom is exact there;
  // at or beyond it the scale is the largest code whatever the quotient.
  const bool fast = nt.denom_safe && (amax_b == 0.0f || amax_b >= 0x1p-60f);
  const float q = fast ? (amax_b >= __fmul_rn(512.0f, nt.denom) ? 512.0f : div1_fast(amax_b, nt.denom, nt.rc_denom))
                       : __fdiv_rn(amax_b, nt.denom);
  scale_code = e4m3_encode(q);
  const float sb = e4m3_decode(scale_code);
  const float S = __fmul_rn(nt.s_t, sb);
  const float2 sb2 = splat(sb), st2 = splat(nt.s_t);
  if (S == 0.0f) {
#pragma unroll
    for (int j = 0; j < NW; ++j) { xhat[j] = 0u; codes[j] = 0u; }
  } else if (fast && div_safe(S) && amax_b <= __fmul_rn(8.0f, S)) {
    const float rc = __frcp_rn(S);
#pragma unroll
    for (int j = 0; j < NW; ++j) {
      const float2 v = div2_fast(unpack2(w[j]), S, rc);
      codes[j] = e2m1x2_encode(v.x, v.y);
      const float2 o = __fmul2_rn(__fmul2_rn(sb2, e2m1x2_decode(codes[j])), st2);
      xhat[j] = pack_bf16x2(o.x, o.y);
    }
  } else {
#pragma unroll
    for (int j = 0; j < NW; ++j) {
      const float2 x = unpack2(w[j]);
      codes[j] = e2m1x2_encode(__fdiv_rn(x.x, S), __fdiv_rn(x.y, S));
      const float2 o = __fmul2_rn(__fmul2_rn(sb2, e2m1x2_decode(codes[j])), st2);
      xhat[j] = pack_bf16x2(o.x, o.y);
    }
  }
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
// the first half of that alone: *a.tscale_out (a.groups floats) receives the derived tensor scale(s); nothing is quantized
cudaError_t launch_nvfp4_scales_only(const QdqArgs& a, uint32_t* header, int amax_word, cudaStream_t st);
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
  uint32_t* tile_sync_word;      // device word, zero before the launch: arrival counter of the tile-start rendezvous (nullable)
  int fuse_a_fmt, fuse_b_fmt;        // QF_FMT_MXFP4 / QF_FMT_NVFP4: quantize-dequantize the staged tiles of that operand
                                     // inside the kernel (QF_FMT_NONE: the operand is used as it is)
  const float* fuse_a_tscale;        // NVFP4: device tensor scale of A (one float), final before the launch
  const float* fuse_b_tscale;        // NVFP4: device tensor scale(s) of B: one float, or one per group (mode 1)
  bool fuse_b_tscale_per_group;
  bool mxfp4_noclip;                 // scale rule of the in-kernel MXFP4 quantizer (QF_MXFP4_NO_CLIP)
  // Side jobs: flat FP4 quantize-dequantize passes (BF16 copy only) that spare warps of the matmul kernel run while the
  // tensor cores work, for operands of the NEXT product. Nothing in this launch reads what they write.
  struct Side {
    const void* in;                  // BF16, nelem elements (a multiple of 32)
    void* out;
    int64_t nelem;                   // 0: no job
    int fmt;                         // QF_FMT_MXFP4, or QF_FMT_NVFP4 with a final tensor scale at *tscale
    const float* tscale;
    bool mxfp4_noclip;
  } side[2];
};
bool gemm_side_supported(const GemmArgs& a);

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
