// Memory-bound quantize-dequantize kernels for NVFP4, MXFP4 and Q4_K (the paper's Section 3.2.3
// formats; Eq. nvfp4 / mxfp4 / q4k and their dequantization equations), plus the tensor-amax
// pre-pass NVFP4 needs and the stand-alone dequantizers.
//
// Work decomposition: one thread owns one 16-byte chunk (8 BF16 values); a warp reads 512
// contiguous bytes per load instruction. A quantization block is 2 (NVFP4), 4 (MXFP4) or 32
// (Q4_K super-block) neighbouring lanes, so block statistics are warp shuffles. Every FP32
// operation that decides a code is written with an explicit round-to-nearest intrinsic so that
// the compiler can neither contract it into an FMA nor replace a division by a reciprocal.
#include "qf_common.cuh"

namespace qf {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;          // independent 16-byte loads in flight per thread

__device__ __forceinline__ uint4 ld_chunk(const uint4* p) { return __ldg(p); }

// max |x| over the 8 BF16 values of a chunk, as BF16 bits (sign clear)
__device__ __forceinline__ uint32_t chunk_amax_bits(const uint4& v) {
  uint32_t m = umax2_bits(umax2_bits(habs2_bits(v.x), habs2_bits(v.y)),
                          umax2_bits(habs2_bits(v.z), habs2_bits(v.w)));
  return hmax_of_pair(m);
}

// ---------------------------------------------------------------------------------------------
// tensor amax
// ---------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kThreads) amax_kernel(const uint4* __restrict__ in, int64_t nchunks,
                                                        const __nv_bfloat16* __restrict__ tail, int ntail,
                                                        uint32_t* __restrict__ amax_bits) {
  uint32_t m = 0;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  for (; i + 3 * stride < nchunks; i += 4 * stride) {
    uint4 a = ld_chunk(in + i), b = ld_chunk(in + i + stride), c = ld_chunk(in + i + 2 * stride),
          d = ld_chunk(in + i + 3 * stride);
    m = max(m, max(max(chunk_amax_bits(a), chunk_amax_bits(b)), max(chunk_amax_bits(c), chunk_amax_bits(d))));
  }
  for (; i < nchunks; i += stride) m = max(m, chunk_amax_bits(ld_chunk(in + i)));
  if (blockIdx.x == 0 && threadIdx.x < ntail)
    m = max(m, static_cast<uint32_t>(__bfloat16_as_ushort(tail[threadIdx.x])) & 0x7FFFu);
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  __shared__ uint32_t warp_max[kThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (threadIdx.x == 0 && m) atomicMax(amax_bits, m << 16);     // BF16 bits -> FP32 bits
  }
}

__global__ void amax_to_float_kernel(const uint32_t* amax_bits, float* out) { *out = __uint_as_float(*amax_bits); }

// ---------------------------------------------------------------------------------------------
// per-chunk quantize-dequantize, FP4 formats
// ---------------------------------------------------------------------------------------------

struct ChunkOut {
  uint4 xhat;        // 8 BF16
  uint32_t codes;    // 8 x 4 bit, element i in nibble i
};

// MXFP4: x_hat = 2^p * C with p = floor(log2 amax_block) - 2 (Eq. mxfp4-dequant).
__device__ __forceinline__ ChunkOut mxfp4_chunk(const uint4& v, uint32_t block_amax_bits, uint32_t& scale_code) {
  scale_code = mxfp4_scale_code(block_amax_bits);
  const float inv = e8m0_inv_scale(scale_code);
  const float sc = e8m0_scale(scale_code);
  const bool zero_block = block_amax_bits == 0;
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t o[4];
  ChunkOut r;
  r.codes = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t byte = e2m1x2_encode(__fmul_rn(bf16_lo(w[j]), inv), __fmul_rn(bf16_hi(w[j]), inv));
    if (zero_block) byte = 0;                       // an all-zero block drops the sign of -0
    float2 c = e2m1x2_decode(byte);
    o[j] = pack_bf16x2(__fmul_rn(c.x, sc), __fmul_rn(c.y, sc));
    r.codes |= byte << (8 * j);
  }
  r.xhat = make_uint4(o[0], o[1], o[2], o[3]);
  return r;
}

// NVFP4: x_hat = s_FP32 * s_E4M3 * C (Eq. nvfp4-dequant); block scale = E4M3(amax_block / (6 s_FP32)).
__device__ __forceinline__ ChunkOut nvfp4_chunk(const uint4& v, uint32_t block_amax_bits, float s_t,
                                                uint32_t& scale_code) {
  const float amax_b = __uint_as_float(block_amax_bits << 16);
  const float q = __fdiv_rn(amax_b, __fmul_rn(6.0f, s_t));
  scale_code = e4m3_encode(q);
  const float sb = e4m3_decode(scale_code);
  const float S = __fmul_rn(s_t, sb);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t o[4];
  ChunkOut r;
  r.codes = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint32_t byte = 0;
    if (S != 0.0f) byte = e2m1x2_encode(__fdiv_rn(bf16_lo(w[j]), S), __fdiv_rn(bf16_hi(w[j]), S));
    float2 c = e2m1x2_decode(byte);
    o[j] = pack_bf16x2(__fmul_rn(__fmul_rn(sb, c.x), s_t), __fmul_rn(__fmul_rn(sb, c.y), s_t));
    r.codes |= byte << (8 * j);
  }
  r.xhat = make_uint4(o[0], o[1], o[2], o[3]);
  return r;
}

template <int FMT>
__global__ void __launch_bounds__(kThreads) qdq_fp4_kernel(const uint4* __restrict__ in, int64_t nchunks,
                                                           uint4* __restrict__ out, uint32_t* __restrict__ codes,
                                                           uint8_t* __restrict__ scales,
                                                           const float* __restrict__ tscale_in,
                                                           const uint32_t* __restrict__ amax_bits,
                                                           float* __restrict__ tscale_out) {
  constexpr int kLanesPerBlock = FMT == QF_FMT_NVFP4 ? 2 : 4;
  float s_t = 1.0f;
  if (FMT == QF_FMT_NVFP4) {
    if (amax_bits) {
      const float amax_t = __uint_as_float(*amax_bits);
      s_t = amax_t == 0.0f ? 1.0f : __fdiv_rn(amax_t, 2688.0f);            // 2688 = 6 * 448
      if (tscale_out && blockIdx.x == 0 && threadIdx.x == 0) *tscale_out = s_t;
    } else {
      s_t = *tscale_in;
    }
  }
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  const int64_t first = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  // warp-uniform trip count: every lane of a warp takes part in the shuffles
  const int64_t warp_first = first - (threadIdx.x & 31);
  for (int64_t base = 0; warp_first + base < nchunks; base += kUnroll * stride) {
    uint4 v[kUnroll];
    bool ok[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t i = first + base + u * stride;
      ok[u] = i < nchunks;
      v[u] = ok[u] ? ld_chunk(in + i) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t i = first + base + u * stride;
      if (warp_first + base + u * stride >= nchunks) break;                 // warp-uniform
      uint32_t m = chunk_amax_bits(v[u]);
      m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
      if (kLanesPerBlock == 4) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
      uint32_t scale_code;
      ChunkOut r = FMT == QF_FMT_NVFP4 ? nvfp4_chunk(v[u], m, s_t, scale_code) : mxfp4_chunk(v[u], m, scale_code);
      if (ok[u]) {
        if (out) out[i] = r.xhat;
        if (codes) codes[i] = r.codes;
        if (scales && (threadIdx.x & (kLanesPerBlock - 1)) == 0) scales[i / kLanesPerBlock] = static_cast<uint8_t>(scale_code);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Q4_K: one warp per 256-weight super-block; lane t owns elements 8t..8t+7, sub-block t/4.
// x_hat = (d * s6) * C - (dmin * m6)  (Eq. q4k-dequant); min/max affine rule for the quantizer.
// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ float clampf(float v, float lo, float hi) { return fminf(fmaxf(v, lo), hi); }

__global__ void __launch_bounds__(kThreads) qdq_q4k_kernel(const uint4* __restrict__ in, int64_t nchunks,
                                                           uint4* __restrict__ out, uint32_t* __restrict__ codes,
                                                           uint4* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  // nchunks is a multiple of 32, so a warp is either entirely inside the tensor or entirely outside
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < nchunks; i += stride) {
    const uint4 v = ld_chunk(in + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float x[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      x[2 * j] = bf16_lo(w[j]);
      x[2 * j + 1] = bf16_hi(w[j]);
    }
    float lo = fminf(fminf(fminf(x[0], x[1]), fminf(x[2], x[3])), fminf(fminf(x[4], x[5]), fminf(x[6], x[7])));
    float hi = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])), fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, 1));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, 1));
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, 2));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, 2));
    lo = fminf(lo, 0.0f);
    const float sc = __fdiv_rn(__fsub_rn(hi, lo), 15.0f);
    const float off = __fsub_rn(0.0f, lo);             // >= +0: a sub-block with no negative value has offset +0
    float max_sc = sc, max_off = off;
#pragma unroll
    for (int s = 4; s < 32; s <<= 1) {
      max_sc = fmaxf(max_sc, __shfl_xor_sync(0xFFFFFFFFu, max_sc, s));
      max_off = fmaxf(max_off, __shfl_xor_sync(0xFFFFFFFFu, max_off, s));
    }
    const __half d_h = __float2half_rn(fminf(__fdiv_rn(max_sc, 63.0f), 65504.0f));
    const __half dmin_h = __float2half_rn(fminf(__fdiv_rn(max_off, 63.0f), 65504.0f));
    const float d = __half2float(d_h), dmin = __half2float(dmin_h);
    const float s6f = d == 0.0f ? 0.0f : clampf(rintf(__fdiv_rn(sc, d)), 0.0f, 63.0f);
    const float m6f = dmin == 0.0f ? 0.0f : clampf(rintf(__fdiv_rn(off, dmin)), 0.0f, 63.0f);
    const float es = __fmul_rn(d, s6f), em = __fmul_rn(dmin, m6f);
    uint32_t c8 = 0;
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float c0 = 0.0f, c1 = 0.0f;
      if (es > 0.0f) {
        c0 = clampf(rintf(__fdiv_rn(__fadd_rn(x[2 * j], em), es)), 0.0f, 15.0f);
        c1 = clampf(rintf(__fdiv_rn(__fadd_rn(x[2 * j + 1], em), es)), 0.0f, 15.0f);
      }
      o[j] = pack_bf16x2(__fsub_rn(__fmul_rn(es, c0), em), __fsub_rn(__fmul_rn(es, c1), em));
      c8 |= (static_cast<uint32_t>(c0) | (static_cast<uint32_t>(c1) << 4)) << (8 * j);
    }
    if (out) out[i] = make_uint4(o[0], o[1], o[2], o[3]);
    // code bytes: within a 64-element chunk (8 lanes), byte l = element l | element l+32 << 4.
    // Lanes 0-3 of the 8 hold elements l, lanes 4-7 the elements l+32; the pair (t, t^4) splits the
    // 8 bytes it can form: the low lane writes bytes for its elements 0-3, the high lane for 4-7.
    const uint32_t partner = __shfl_xor_sync(0xFFFFFFFFu, c8, 4);
    if (codes) {
      const bool high = (lane & 4) != 0;
      const uint32_t lo_src = high ? partner : c8, hi_src = high ? c8 : partner;
      const int sh = high ? 16 : 0;
      uint32_t word = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        word |= (((lo_src >> (sh + 4 * k)) & 15u) | (((hi_src >> (sh + 4 * k)) & 15u) << 4)) << (8 * k);
      // super-block i/32 owns 32 words; chunk (lane/8) owns 8 of them; low lane q writes word 2q, high 2q+1
      const int q = lane & 3;
      codes[(i - lane) + (lane >> 3) * 8 + 2 * q + (high ? 1 : 0)] = word;
    }
    if (scales) {
      // gather the eight 6-bit (s6, m6) pairs: each sub-block leader contributes its byte lanes
      const uint32_t s6 = static_cast<uint32_t>(s6f), m6 = static_cast<uint32_t>(m6f);
      const int b = lane >> 2;
      const bool leader = (lane & 3) == 0;
      // words of the 12 packed bytes: w0 = bytes 0-3, w1 = bytes 4-7, w2 = bytes 8-11
      uint32_t w0 = 0, w1 = 0, w2 = 0;
      if (leader) {
        if (b < 4) {
          w0 = (s6 & 63u) << (8 * b);
          w1 = (m6 & 63u) << (8 * b);
        } else {
          w0 = ((s6 >> 4) << 6) << (8 * (b - 4));
          w1 = ((m6 >> 4) << 6) << (8 * (b - 4));
          w2 = ((s6 & 15u) | ((m6 & 15u) << 4)) << (8 * (b - 4));
        }
      }
      w0 = __reduce_or_sync(0xFFFFFFFFu, w0);
      w1 = __reduce_or_sync(0xFFFFFFFFu, w1);
      w2 = __reduce_or_sync(0xFFFFFFFFu, w2);
      if (lane == 0) {
        const uint32_t hdr = static_cast<uint32_t>(__half_as_ushort(d_h)) | (static_cast<uint32_t>(__half_as_ushort(dmin_h)) << 16);
        scales[i >> 5] = make_uint4(hdr, w0, w1, w2);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// stand-alone dequantizers: one thread per 8 outputs
// ---------------------------------------------------------------------------------------------

template <int FMT>
__global__ void __launch_bounds__(kThreads) dequant_fp4_kernel(const uint32_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales,
                                                               const float* __restrict__ tscale, int64_t nchunks,
                                                               uint4* __restrict__ out) {
  constexpr int kLanesPerBlock = FMT == QF_FMT_NVFP4 ? 2 : 4;
  const float s_t = FMT == QF_FMT_NVFP4 ? *tscale : 1.0f;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < nchunks; i += stride) {
    const uint32_t c = codes[i];
    const uint32_t sc = scales[i / kLanesPerBlock];
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float2 val = e2m1x2_decode((c >> (8 * j)) & 0xFFu);
      if (FMT == QF_FMT_NVFP4) {
        const float sb = e4m3_decode(sc & 0x7Fu);
        o[j] = pack_bf16x2(__fmul_rn(__fmul_rn(sb, val.x), s_t), __fmul_rn(__fmul_rn(sb, val.y), s_t));
      } else {
        const float s = e8m0_scale(sc);
        o[j] = pack_bf16x2(__fmul_rn(val.x, s), __fmul_rn(val.y, s));
      }
    }
    out[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

__global__ void __launch_bounds__(kThreads) dequant_q4k_kernel(const uint8_t* __restrict__ codes,
                                                               const uint8_t* __restrict__ scales, int64_t nchunks,
                                                               uint4* __restrict__ out) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < nchunks; i += stride) {
    const int64_t sb = i >> 5;
    const int t = static_cast<int>(i & 31);           // chunk within the super-block: elements 8t..8t+7
    const int b = t >> 2;                             // sub-block
    const uint8_t* r = scales + sb * 16;
    const float d = __half2float(__ushort_as_half(static_cast<unsigned short>(r[0] | (r[1] << 8))));
    const float dmin = __half2float(__ushort_as_half(static_cast<unsigned short>(r[2] | (r[3] << 8))));
    const uint8_t* pk = r + 4;
    uint32_t s6, m6;
    if (b < 4) {
      s6 = pk[b] & 63u;
      m6 = pk[b + 4] & 63u;
    } else {
      s6 = (pk[b + 4] & 15u) | ((pk[b - 4] >> 6) << 4);
      m6 = (pk[b + 4] >> 4) | ((pk[b] >> 6) << 4);
    }
    const float es = __fmul_rn(d, static_cast<float>(s6)), em = __fmul_rn(dmin, static_cast<float>(m6));
    const uint8_t* q = codes + sb * 128 + (t >> 3) * 32 + (t & 3) * 8;
    const int sh = (t & 4) ? 4 : 0;
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float c0 = static_cast<float>((q[2 * j] >> sh) & 15u), c1 = static_cast<float>((q[2 * j + 1] >> sh) & 15u);
      o[j] = pack_bf16x2(__fsub_rn(__fmul_rn(es, c0), em), __fsub_rn(__fmul_rn(es, c1), em));
    }
    out[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

__global__ void selftest_cvt_kernel(const float* __restrict__ in, int64_t n, uint8_t* __restrict__ e2m1,
                                    uint8_t* __restrict__ e4m3) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float x = in[i];
  if (e2m1) e2m1[i] = static_cast<uint8_t>(e2m1x2_encode(x, 0.0f) & 15u);
  if (e4m3) e4m3[i] = static_cast<uint8_t>(e4m3_encode(fabsf(x)));
}

int grid_for(int64_t nchunks, int per_thread) {
  int64_t blocks = (nchunks + static_cast<int64_t>(kThreads) * per_thread - 1) / (static_cast<int64_t>(kThreads) * per_thread);
  const int64_t cap = static_cast<int64_t>(kNumSMs) * 8;       // 8 resident blocks of 256 threads per SM
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

}  // namespace

cudaError_t launch_amax(const void* in, int64_t n, uint32_t* amax_bits, cudaStream_t st) {
  const int64_t nchunks = n / 8;
  const int ntail = static_cast<int>(n % 8);
  amax_kernel<<<grid_for(nchunks, 4), kThreads, 0, st>>>(static_cast<const uint4*>(in), nchunks,
                                                         static_cast<const __nv_bfloat16*>(in) + nchunks * 8, ntail,
                                                         amax_bits);
  return cudaGetLastError();
}

cudaError_t launch_amax_to_float(const uint32_t* amax_bits, float* out, cudaStream_t st) {
  amax_to_float_kernel<<<1, 1, 0, st>>>(amax_bits, out);
  return cudaGetLastError();
}

cudaError_t launch_qdq(const QdqArgs& a, cudaStream_t st) {
  const int64_t nchunks = a.rows * a.cols / 8;
  // an empty NVFP4 tensor still has a tensor scale to report (1.0): let one block write it
  if (nchunks == 0 && !(a.fmt == QF_FMT_NVFP4 && a.tscale_out)) return cudaSuccess;
  const uint4* in = static_cast<const uint4*>(a.in);
  uint4* out = static_cast<uint4*>(a.out);
  uint32_t* codes = static_cast<uint32_t*>(a.codes);
  if (a.fmt == QF_FMT_NVFP4) {
    qdq_fp4_kernel<QF_FMT_NVFP4><<<grid_for(nchunks, kUnroll), kThreads, 0, st>>>(
        in, nchunks, out, codes, static_cast<uint8_t*>(a.scales), a.tscale_in, a.amax_bits, a.tscale_out);
  } else if (a.fmt == QF_FMT_MXFP4) {
    qdq_fp4_kernel<QF_FMT_MXFP4><<<grid_for(nchunks, kUnroll), kThreads, 0, st>>>(
        in, nchunks, out, codes, static_cast<uint8_t*>(a.scales), nullptr, nullptr, nullptr);
  } else {
    qdq_q4k_kernel<<<grid_for(nchunks, 2), kThreads, 0, st>>>(in, nchunks, out, codes, static_cast<uint4*>(a.scales));
  }
  return cudaGetLastError();
}

cudaError_t launch_dequant(int fmt, const void* codes, const void* scales, const float* tscale, int64_t rows,
                           int64_t cols, void* out, cudaStream_t st) {
  const int64_t nchunks = rows * cols / 8;
  if (nchunks == 0) return cudaSuccess;
  const int grid = grid_for(nchunks, 2);
  if (fmt == QF_FMT_NVFP4)
    dequant_fp4_kernel<QF_FMT_NVFP4><<<grid, kThreads, 0, st>>>(static_cast<const uint32_t*>(codes),
                                                                static_cast<const uint8_t*>(scales), tscale, nchunks,
                                                                static_cast<uint4*>(out));
  else if (fmt == QF_FMT_MXFP4)
    dequant_fp4_kernel<QF_FMT_MXFP4><<<grid, kThreads, 0, st>>>(static_cast<const uint32_t*>(codes),
                                                                static_cast<const uint8_t*>(scales), nullptr, nchunks,
                                                                static_cast<uint4*>(out));
  else
    dequant_q4k_kernel<<<grid, kThreads, 0, st>>>(static_cast<const uint8_t*>(codes),
                                                  static_cast<const uint8_t*>(scales), nchunks, static_cast<uint4*>(out));
  return cudaGetLastError();
}

cudaError_t launch_selftest_cvt(const float* in, int64_t n, uint8_t* e2m1, uint8_t* e4m3, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  selftest_cvt_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(in, n, e2m1, e4m3);
  return cudaGetLastError();
}

}  // namespace qf
