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
  kWsScaleW = 8,      // derived NVFP4 tensor scale of W (float)
  kWsScaleA = 9,      // derived NVFP4 tensor scale of X (float)
};

// ---- device helpers -----------------------------------------------------------------------

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ uint32_t habs2_bits(uint32_t w) { return w & 0x7FFF7FFFu; }

// max of two packed pairs of non-negative BF16 values (bit patterns of non-negative floats are
// ordered like unsigned integers)
__device__ __forceinline__ uint32_t umax2_bits(uint32_t a, uint32_t b) { return __vmaxu2(a, b); }

__device__ __forceinline__ uint32_t hmax_of_pair(uint32_t w) { return max(w & 0xFFFFu, w >> 16); }

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
__device__ __forceinline__ uint32_t mxfp4_scale_code(uint32_t amax_bf16_bits) {
  int e = static_cast<int>(amax_bf16_bits >> 7);
  return static_cast<uint32_t>(max(e - 2, 0));
}

// ---- host-side launchers implemented in the .cu files ---------------------------------------

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
};

cudaError_t launch_amax(const void* in, int64_t n, uint32_t* amax_bits, cudaStream_t st);
cudaError_t launch_amax_to_float(const uint32_t* amax_bits, float* out, cudaStream_t st);
cudaError_t launch_qdq(const QdqArgs& a, cudaStream_t st);
cudaError_t launch_qdq_nvfp4_derive(const QdqArgs& a, uint32_t* header, int amax_word, cudaStream_t st);
cudaError_t launch_dequant(int fmt, const void* codes, const void* scales, const float* tscale, int64_t rows,
                           int64_t cols, void* out, cudaStream_t st);
cudaError_t launch_selftest_div(const float* xs, int64_t nx, const float* ys, int64_t ny, unsigned long long* mismatches,
                                cudaStream_t st);
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
};

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st);

}  // namespace qf
