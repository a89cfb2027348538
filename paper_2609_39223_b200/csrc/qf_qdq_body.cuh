// Device code of the FP4 quantize-dequantize pass shared by the stand-alone quantizer kernels (qf_qdq.cu) and by the
// matmul kernel, which can run the same loop as a side job for the operand of the NEXT product (qf_gemm.cu).
#pragma once

#include "qf_common.cuh"

namespace qf {

constexpr int kQdqThreads = 256;       // threads per block of the stand-alone quantizer kernels

// Where a kernel's 16-byte input chunks come from: the tensor itself.
struct PlainLoader {
  const uint4* in;
  __device__ __forceinline__ uint4 chunk(int64_t c) const { return __ldg(in + c); }
  __device__ __forceinline__ PlainLoader slice(int64_t chunks) const { return PlainLoader{in + chunks}; }
};


// chunk = 8 BF16 values
__device__ __forceinline__ uint32_t chunk_amax_bits(const uint4& v) { return chunk8_amax_bits(v.x, v.y, v.z, v.w); }

// max |x| over 16 BF16 values held in 8 words, as BF16 bits (sign clear)
__device__ __forceinline__ uint32_t unit_amax_bits(const uint32_t (&w)[8]) {
  __nv_bfloat162 m0 = __hmax2(__habs2(bits_bf2(w[0])), __habs2(bits_bf2(w[1])));
  __nv_bfloat162 m1 = __hmax2(__habs2(bits_bf2(w[2])), __habs2(bits_bf2(w[3])));
  __nv_bfloat162 m2 = __hmax2(__habs2(bits_bf2(w[4])), __habs2(bits_bf2(w[5])));
  __nv_bfloat162 m3 = __hmax2(__habs2(bits_bf2(w[6])), __habs2(bits_bf2(w[7])));
  const uint32_t m = bf2_bits(__hmax2(__hmax2(m0, m1), __hmax2(m2, m3)));
  return max(m & 0xFFFFu, m >> 16);
}

// ---------------------------------------------------------------------------------------------
// FP4 formats: one lane owns 16 consecutive elements (two 16-byte loads): a whole NVFP4 block, or
// half an MXFP4 block (one shuffle with the neighbouring lane).
// ---------------------------------------------------------------------------------------------

struct UnitOut {
  uint32_t xhat[8];   // 16 BF16
  uint2 codes;        // 16 x 4 bit, element i in nibble i
};

// MXFP4: x_hat = 2^p * C with p = floor(log2 amax_block) - 2 (Eq. mxfp4-dequant). All products exact.
__device__ __forceinline__ UnitOut mxfp4_unit(const uint32_t (&w)[8], uint32_t block_amax_bits, bool noclip,
                                              uint32_t& scale_code) {
  scale_code = mxfp4_scale_code(block_amax_bits, noclip);
  const float2 inv = splat(e8m0_inv_scale(scale_code));
  const float2 sc = splat(e8m0_scale(scale_code));
  const uint32_t keep = block_amax_bits == 0 ? 0u : 0xFFu;       // an all-zero block drops the sign of -0
  UnitOut r;
  uint32_t c[2] = {0, 0};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float2 v = __fmul2_rn(unpack2(w[j]), inv);
    const uint32_t byte = e2m1x2_encode(v.x, v.y) & keep;
    const float2 o = __fmul2_rn(e2m1x2_decode(byte), sc);
    r.xhat[j] = pack_bf16x2(o.x, o.y);
    c[j >> 2] |= byte << (8 * (j & 3));
  }
  r.codes = make_uint2(c[0], c[1]);
  return r;
}

// NVFP4: x_hat = s_FP32 * s_E4M3 * C (Eq. nvfp4-dequant); block scale = E4M3(amax_block / (6 s_FP32)).
// FAST selects the reciprocal-based exact division; otherwise the IEEE divide.
template <bool FAST>
__device__ __forceinline__ UnitOut nvfp4_unit(const uint32_t (&w)[8], float amax_b, float s_t, float denom, float rc_denom,
                                              uint32_t& scale_code) {
  // A supplied tensor scale can be far too small for a block: the quotient then exceeds every E4M3 value and may
  // even overflow FP32, which the reciprocal-based form does not survive (inf - inf). 512 * denom is exact
  // (denom lies in [2^-60, 2^60] on this path); at or beyond it the scale is the largest code whatever the quotient.
  const float q = FAST ? (amax_b >= __fmul_rn(512.0f, denom) ? 512.0f : div1_fast(amax_b, denom, rc_denom))
                       : __fdiv_rn(amax_b, denom);
  scale_code = e4m3_encode(q);
  const float sb = e4m3_decode(scale_code);
  const float S = __fmul_rn(s_t, sb);
  UnitOut r;
  uint32_t c[2] = {0, 0};
  const float2 sb2 = splat(sb), st2 = splat(s_t);
  // Three whole-block cases, chosen once (not per element): scale rounded to zero; the
  // reciprocal-based division (sane divisor, quotients bounded by 8); the IEEE divide.
  if (S == 0.0f) {
#pragma unroll
    for (int j = 0; j < 8; ++j) r.xhat[j] = 0u;
  } else if (FAST && div_safe(S) && amax_b <= __fmul_rn(8.0f, S)) {
    const float rc = __frcp_rn(S);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float2 x = unpack2(w[j]);
      const float2 v = div2_fast(x, S, rc);          // signed zeros included: x = -0 gives -0
      const uint32_t byte = e2m1x2_encode(v.x, v.y);
      const float2 o = __fmul2_rn(__fmul2_rn(sb2, e2m1x2_decode(byte)), st2);
      r.xhat[j] = pack_bf16x2(o.x, o.y);
      c[j >> 2] |= byte << (8 * (j & 3));
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float2 x = unpack2(w[j]);
      const uint32_t byte = e2m1x2_encode(__fdiv_rn(x.x, S), __fdiv_rn(x.y, S));
      const float2 o = __fmul2_rn(__fmul2_rn(sb2, e2m1x2_decode(byte)), st2);
      r.xhat[j] = pack_bf16x2(o.x, o.y);
      c[j >> 2] |= byte << (8 * (j & 3));
    }
  }
  r.codes = make_uint2(c[0], c[1]);
  return r;
}

constexpr int kUnitsPerThread = 2;

// The grid-stride loop shared by the single-tensor and the batched FP4 kernels: this thread's units are
// first, first + stride, ... (two in flight per iteration). Every thread of the block must call it (the optional
// maximum reduction at the end synchronises the block).
template <int FMT, typename Loader, bool ACCUM = true>
__device__ __forceinline__ void qdq_fp4_body(const Loader& in, int64_t nunits, uint4* __restrict__ out, uint2* __restrict__ codes,
                                             uint8_t* __restrict__ scales, const Nvfp4Tensor nt, bool reverse, bool noclip,
                                             uint32_t* __restrict__ amax_accum, int64_t first, int64_t stride) {
  const float s_t = nt.s_t, denom = nt.denom, rc_denom = nt.rc_denom;
  const bool denom_safe = nt.denom_safe;
  const int lane = threadIdx.x & 31;
  const int64_t warp_first = first - lane;                    // warp-uniform trip count (shuffles below)
  const int64_t nunits_up = (nunits + 31) & ~static_cast<int64_t>(31);
  uint32_t seen = 0;                                          // largest block maximum this thread met (speculative first pass)
  for (int64_t base = 0; warp_first + base < nunits_up; base += kUnitsPerThread * stride) {
    uint4 v[kUnitsPerThread][2];
    bool ok[kUnitsPerThread];
#pragma unroll
    for (int u = 0; u < kUnitsPerThread; ++u) {
      const int64_t lin = first + base + u * stride;
      // reverse: walk whole warps' worth of units from the end (block pairs of lanes stay adjacent)
      const int64_t i = reverse ? (nunits_up - 32 - (lin - lane)) + lane : lin;
      ok[u] = lin < nunits_up && i < nunits;      // lin past the end would map to a negative index in reverse
      v[u][0] = ok[u] ? in.chunk(2 * i) : make_uint4(0, 0, 0, 0);
      v[u][1] = ok[u] ? in.chunk(2 * i + 1) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kUnitsPerThread; ++u) {
      const int64_t lin = first + base + u * stride;
      const int64_t i = reverse ? (nunits_up - 32 - (lin - lane)) + lane : lin;
      if (warp_first + base + u * stride >= nunits_up) break;              // warp-uniform
      const uint32_t w[8] = {v[u][0].x, v[u][0].y, v[u][0].z, v[u][0].w, v[u][1].x, v[u][1].y, v[u][1].z, v[u][1].w};
      uint32_t m = unit_amax_bits(w);
      uint32_t scale_code;
      UnitOut r;
      seen = max(seen, m);
      if (FMT == QF_FMT_MXFP4) {
        m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
        r = mxfp4_unit(w, m, noclip, scale_code);
      } else {
        const float amax_b = __uint_as_float(m << 16);
        // quotients near the bottom of the FP32 range take the IEEE divide (warp-uniform choice)
        const bool fast_ok = denom_safe && (amax_b == 0.0f || amax_b >= 0x1p-60f);
        if (__all_sync(0xFFFFFFFFu, fast_ok)) r = nvfp4_unit<true>(w, amax_b, s_t, denom, rc_denom, scale_code);
        else r = nvfp4_unit<false>(w, amax_b, s_t, denom, rc_denom, scale_code);
      }
      if (ok[u]) {
        if (out) {
          out[2 * i] = make_uint4(r.xhat[0], r.xhat[1], r.xhat[2], r.xhat[3]);
          out[2 * i + 1] = make_uint4(r.xhat[4], r.xhat[5], r.xhat[6], r.xhat[7]);
        }
        if (codes) codes[i] = r.codes;
        if (scales) {
          if (FMT == QF_FMT_NVFP4) scales[i] = static_cast<uint8_t>(scale_code);
          else if ((threadIdx.x & 1) == 0) scales[i >> 1] = static_cast<uint8_t>(scale_code);
        }
      }
    }
  }
  if constexpr (!ACCUM) return;            // (no block-wide synchronisation on this path: safe inside a warp-specialised kernel)
  if (amax_accum) {
    // the maximum of everything this pass read (padding lanes contributed zeros): for the pass that checks a
    // guessed tensor scale, or for a caller that wants max|x| reported without a separate read
    seen = __reduce_max_sync(0xFFFFFFFFu, seen);
    __shared__ uint32_t warp_seen[kQdqThreads / 32];
    if (lane == 0) warp_seen[threadIdx.x >> 5] = seen;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t m = 0;
#pragma unroll
      for (int k = 0; k < kQdqThreads / 32; ++k) m = max(m, warp_seen[k]);
      if (m) atomicMax(amax_accum, m << 16);             // BF16 bits -> FP32 bits
    }
  }
}

}  // namespace qf
