// Memory-bound quantize-dequantize kernels for NVFP4, MXFP4 and Q4_K (the paper's Section 3.2.3
// formats; Eq. nvfp4 / mxfp4 / q4k and their dequantization equations), plus the tensor-amax
// pre-pass NVFP4 needs and the stand-alone dequantizers.
//
// Work decomposition: FP4 formats: a lane owns 16 consecutive elements (two 16-byte loads): a whole
// NVFP4 block, or half an MXFP4 block (one shuffle with the neighbouring lane). Q4_K: a lane owns one
// 32-weight sub-block (four 16-byte loads), eight neighbouring lanes a super-block, whose statistics are
// warp shuffles. The tensor-amax pass reads one 16-byte chunk per lane and load. Every FP32
// operation that decides a code is written with an explicit round-to-nearest intrinsic so that
// the compiler can neither contract it into an FMA nor replace a division by a reciprocal.
#include "qf_common.cuh"
#include "qf_ptx.cuh"
#include "qf_qdq_body.cuh"

namespace qf {
namespace {

constexpr int kThreads = kQdqThreads;


// Where a kernel's 16-byte input chunks come from. PlainLoader reads the tensor. LoraLoader produces
// the chunk of the merged weight W + s * B A (Eq. qad-lora) on the fly, so the merged tensor is never
// written to memory: per element acc = W; acc = fma(s * B[n,r], A[r,k], acc) for r = 0 .. rank-1 in FP32
// (one rounding per step, in this order), then one rounding to BF16.
struct LoraLoader {
  const uint4* W;                 // [rows, cols] BF16
  const __nv_bfloat16* B;         // [rows, rank] BF16
  const uint4* A;                 // [rank, cols] BF16
  int rank;
  float scale;
  int64_t chunks_per_row;         // cols / 8
  __device__ __forceinline__ uint4 chunk(int64_t c) const {
    const int64_t row = c / chunks_per_row;
    const int64_t kc = c - row * chunks_per_row;
    const uint4 w = __ldg(W + c);
    float acc[8] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y), bf16_lo(w.z), bf16_hi(w.z), bf16_lo(w.w), bf16_hi(w.w)};
    const __nv_bfloat16* brow = B + row * rank;
    for (int r = 0; r < rank; ++r) {
      const float b = __fmul_rn(scale, __bfloat162float(brow[r]));
      const uint4 a = __ldg(A + r * chunks_per_row + kc);
      acc[0] = __fmaf_rn(b, bf16_lo(a.x), acc[0]); acc[1] = __fmaf_rn(b, bf16_hi(a.x), acc[1]);
      acc[2] = __fmaf_rn(b, bf16_lo(a.y), acc[2]); acc[3] = __fmaf_rn(b, bf16_hi(a.y), acc[3]);
      acc[4] = __fmaf_rn(b, bf16_lo(a.z), acc[4]); acc[5] = __fmaf_rn(b, bf16_hi(a.z), acc[5]);
      acc[6] = __fmaf_rn(b, bf16_lo(a.w), acc[6]); acc[7] = __fmaf_rn(b, bf16_hi(a.w), acc[7]);
    }
    return make_uint4(pack_bf16x2(acc[0], acc[1]), pack_bf16x2(acc[2], acc[3]), pack_bf16x2(acc[4], acc[5]), pack_bf16x2(acc[6], acc[7]));
  }
  __device__ __forceinline__ LoraLoader slice(int64_t) const { return *this; }     // grouped slices are not combined with LoRA
};


// ---------------------------------------------------------------------------------------------
// tensor amax
// ---------------------------------------------------------------------------------------------

template <typename Loader>
__global__ void __launch_bounds__(kThreads) amax_kernel(Loader src, int64_t nchunks,
                                                        const __nv_bfloat16* __restrict__ tail, int ntail,
                                                        uint32_t* __restrict__ amax_bits) {
  // gridDim.y > 1: one tensor per y-slice (the experts of a grouped layer), nchunks chunks each
  const Loader in = src.slice(static_cast<int64_t>(blockIdx.y) * nchunks);
  amax_bits += blockIdx.y;
  uint32_t m = 0;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  for (; i + 3 * stride < nchunks; i += 4 * stride) {
    uint4 a = in.chunk(i), b = in.chunk(i + stride), c = in.chunk(i + 2 * stride), d = in.chunk(i + 3 * stride);
    m = max(m, max(max(chunk_amax_bits(a), chunk_amax_bits(b)), max(chunk_amax_bits(c), chunk_amax_bits(d))));
  }
  for (; i < nchunks; i += stride) m = max(m, chunk_amax_bits(in.chunk(i)));
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

// s = amax / (6 * 448), 1.0 for an all-zero tensor: the NVFP4 tensor scale that goes with an absolute maximum
__global__ void amax_to_scale_kernel(const uint32_t* amax_bits, float* scale) {
  const float a = __uint_as_float(*amax_bits);
  *scale = a == 0.0f ? 1.0f : __fdiv_rn(a, 2688.0f);
}

// the same for an array of maxima, converted where they stand (one tensor scale per expert)
__global__ void amax_to_scale_inplace_kernel(uint32_t* bits, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const float a = __uint_as_float(bits[i]);
    bits[i] = __float_as_uint(a == 0.0f ? 1.0f : __fdiv_rn(a, 2688.0f));
  }
}

// The NVFP4 tensor scale a block works with, from whichever source the call uses: `amax_bits` (derive it; the scale is
// also stored to *tscale_out by the slice's first thread) or `tscale_in` (supplied, or a guess in the speculative
// first pass, whose bits are then recorded in *guess_out). Returns false when the block has nothing to do: the
// speculative second pass found the derived scale equal to the guess the first pass quantized with.
__device__ __forceinline__ bool nvfp4_resolve_scale(const float* tscale_in, const uint32_t* amax_bits, float* tscale_out,
                                                    uint32_t* guess_out, const uint32_t* skip_guess, float& s_t) {
  if (amax_bits) {
    const float amax_t = __uint_as_float(*amax_bits);
    s_t = amax_t == 0.0f ? 1.0f : __fdiv_rn(amax_t, 2688.0f);            // 2688 = 6 * 448
    // the first pass already quantized with exactly this scale: nothing to redo (every CTA decides alike)
    if (skip_guess && __float_as_uint(s_t) == *skip_guess) return false;
    if (tscale_out && blockIdx.x == 0 && threadIdx.x == 0) *tscale_out = s_t;
  } else {
    s_t = *tscale_in;
    if (guess_out && blockIdx.x == 0 && threadIdx.x == 0) *guess_out = __float_as_uint(s_t);
  }
  return true;
}

template <int FMT, typename Loader>
__global__ void __launch_bounds__(kThreads) qdq_fp4_kernel(Loader src, int64_t nunits,
                                                           uint4* __restrict__ out, uint2* __restrict__ codes,
                                                           uint8_t* __restrict__ scales,
                                                           const float* __restrict__ tscale_in,
                                                           const uint32_t* __restrict__ amax_bits,
                                                           float* __restrict__ tscale_out, int opts, Nvfp4Speculation spec) {
  const bool reverse = (opts & 1) != 0;       // walk back to front
  const bool noclip = (opts & 2) != 0;        // MXFP4 scale rule without saturation
  // gridDim.y > 1: one tensor of nunits units per y-slice, each with its own tensor scale (NVFP4 experts)
  const int64_t goff = static_cast<int64_t>(blockIdx.y) * nunits;
  const Loader in = src.slice(2 * goff);
  {
    if (out) out += 2 * goff;
    if (codes) codes += goff;
    if (scales) scales += FMT == QF_FMT_NVFP4 ? goff : goff / 2;
  }
  float s_t = 1.0f;
  if (FMT == QF_FMT_NVFP4) {
    if (!nvfp4_resolve_scale(tscale_in ? tscale_in + blockIdx.y : nullptr, amax_bits ? amax_bits + blockIdx.y : nullptr,
                             tscale_out ? tscale_out + blockIdx.y : nullptr, spec.guess_out, spec.skip_guess, s_t))
      return;
  }
  qdq_fp4_body<FMT, Loader>(in, nunits, out, codes, scales, nvfp4_tensor(s_t), reverse, noclip, spec.amax_accum,
                            static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x, static_cast<int64_t>(gridDim.x) * kThreads);
}

// ---- batched form: many tensors, each with its own pointers and size, in one launch -----------------------
// The table travels as a kernel parameter (no device-side table to allocate or copy). blockIdx.y selects the tensor;
// blocks beyond a short tensor's need leave at once.
constexpr int kMaxBatch = 64;
struct QdqBatch {
  const uint4* in[kMaxBatch];
  uint4* out[kMaxBatch];
  void* codes[kMaxBatch];
  void* scales[kMaxBatch];
  int64_t nunits[kMaxBatch];       // FP4: 16-element units; Q4_K: 32-weight sub-blocks
};

// role split of one launch: y-slices [0, n_qdq) quantize tensors of `q`, y-slices [n_qdq, n_qdq + n_amax) take the
// absolute maximum of the tensors of `a` (the NEXT sub-batch): its reads overlap the writes of this one and leave those
// tensors in L2 for the launch that quantizes them.
struct AmaxBatch {
  const uint4* in[kMaxBatch];
  int64_t nchunks[kMaxBatch];
};

__device__ __forceinline__ void amax_block(const uint4* __restrict__ in, int64_t nchunks, uint32_t* __restrict__ amax_bits,
                                           int64_t first, int64_t stride) {
  uint32_t m = 0;
  int64_t i = first;
  for (; i + 3 * stride < nchunks; i += 4 * stride) {
    const uint4 a = __ldg(in + i), b = __ldg(in + i + stride), c = __ldg(in + i + 2 * stride), d = __ldg(in + i + 3 * stride);
    m = max(m, max(max(chunk_amax_bits(a), chunk_amax_bits(b)), max(chunk_amax_bits(c), chunk_amax_bits(d))));
  }
  for (; i < nchunks; i += stride) m = max(m, chunk_amax_bits(__ldg(in + i)));
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

template <int FMT>
__global__ void __launch_bounds__(kThreads) qdq_fp4_batched_kernel(const __grid_constant__ QdqBatch q, int n_qdq,
                                                                   const __grid_constant__ AmaxBatch a,
                                                                   const float* __restrict__ tscale_in,
                                                                   const uint32_t* __restrict__ amax_bits,
                                                                   float* __restrict__ tscale_out, int opts,
                                                                   uint32_t* __restrict__ amax_accum, uint32_t* __restrict__ guess_out,
                                                                   const uint32_t* __restrict__ skip_guess,
                                                                   uint32_t* __restrict__ next_amax_bits) {
  const int64_t first = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  const int t = blockIdx.y;
  if (t >= n_qdq) {
    const int u = t - n_qdq;
    if (static_cast<int64_t>(blockIdx.x) * kThreads >= a.nchunks[u]) return;
    amax_block(a.in[u], a.nchunks[u], next_amax_bits + u, first, stride);
    return;
  }
  const int64_t nunits = q.nunits[t];
  // (block-uniform; block 0 stays even for an empty tensor: it stores the tensor scale, 1.0)
  if (blockIdx.x > 0 && static_cast<int64_t>(blockIdx.x) * kThreads >= nunits) return;
  float s_t = 1.0f;
  if (FMT == QF_FMT_NVFP4) {
    if (!nvfp4_resolve_scale(tscale_in ? tscale_in + t : nullptr, amax_bits ? amax_bits + t : nullptr,
                             tscale_out ? tscale_out + t : nullptr, guess_out ? guess_out + t : nullptr,
                             skip_guess ? skip_guess + t : nullptr, s_t))
      return;
  }
  qdq_fp4_body<FMT, PlainLoader>(PlainLoader{q.in[t]}, nunits, q.out[t], static_cast<uint2*>(q.codes[t]),
                                 static_cast<uint8_t*>(q.scales[t]), nvfp4_tensor(s_t), (opts & 1) != 0, (opts & 2) != 0,
                                 amax_accum ? amax_accum + t : nullptr, first, stride);
}

// ---------------------------------------------------------------------------------------------
// Q4_K: one lane owns a 32-weight sub-block (four 16-byte loads), eight lanes a 256-weight
// super-block, a warp four super-blocks.
// x_hat = (d * s6) * C - (dmin * m6)  (Eq. q4k-dequant); min/max affine rule for the quantizer.
// ---------------------------------------------------------------------------------------------

#ifndef QF_Q4K_MINBLOCKS
#define QF_Q4K_MINBLOCKS 4      // 64 registers, no spills; five blocks (48 registers) measured the same within 1%
#endif
constexpr float kRcp15 = 1.0f / 15.0f;        // correctly rounded reciprocals of the two constant divisors
constexpr float kRcp63 = 1.0f / 63.0f;
constexpr float kRound = 12582912.0f;      // 1.5 * 2^23: adding it rounds to the nearest integer, ties to even

template <bool FAST>
__device__ __forceinline__ float div_by(float x, float y, float rc) { return FAST ? div1_fast(x, y, rc) : __fdiv_rn(x, y); }

// Where the four 16-byte groups of a sub-block's dequantized values go: straight to global memory, or into a
// shared-memory staging tile (slot c of the lane holds chunk c ^ perm, see the staged kernel).
struct GlobalSink {
  uint4* out_ptr;                          // nullable: no dequantized copy wanted
  __device__ __forceinline__ void put(int c, uint4 v) const { if (out_ptr) out_ptr[c] = v; }
};
struct SmemSink {
  uint32_t base;                           // shared address of this lane's 64-byte record
  uint32_t perm;
  bool on;
  __device__ __forceinline__ void put(int c, uint4 v) const {
    if (on) st_shared_v4(base + ((static_cast<uint32_t>(c) ^ perm) << 4), v.x, v.y, v.z, v.w);
  }
};

// The 32 elements of one sub-block given its effective scale and offset: codes (one per byte in cbytes) and dequantized
// values. CLAMP = false leaves out the clamp of the quotient to [0, 15]: the caller has checked that no quotient of the
// sub-block can round outside that range.
template <bool FAST, bool CLAMP, typename Sink>
__device__ __forceinline__ void q4k_elements(const uint32_t (&w)[16], float es, float em, float rc, bool live, const Sink sink,
                                             uint32_t (&cbytes)[8]) {
  uint32_t xhat[4];
  const float2 em2 = splat(em), nem2 = splat(-em), es2 = splat(es), magic = splat(kRound), nmagic = splat(-kRound);
  uint32_t ybits[2][2];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float2 x = unpack2(w[j]);
    float2 y = magic;                                // code 0 when the sub-block has no scale
    if (FAST || live) {                              // FAST: rc = 0 makes the reciprocal-based quotient 0, no branch needed
      const float2 num = __fadd2_rn(x, em2);
      float2 t = FAST ? div2_fast(num, es, rc) : make_float2(__fdiv_rn(num.x, es), __fdiv_rn(num.y, es));
      if (CLAMP) {
        t.x = fminf(fmaxf(t.x, 0.0f), 15.0f);        // clamp first: rounding is monotone and 0, 15 are integers
        t.y = fminf(fmaxf(t.y, 0.0f), 15.0f);
      }
      y = __fadd2_rn(t, magic);                      // integer code now sits in the low mantissa bits
    }
    const float2 c = __fadd2_rn(y, nmagic);
    const float2 o = __ffma2_rn(es2, c, nem2);        // product exact: one rounding, as es*c - em
    xhat[j & 3] = pack_bf16x2(o.x, o.y);
    if ((j & 3) == 3) sink.put(j >> 2, make_uint4(xhat[0], xhat[1], xhat[2], xhat[3]));               // stored as soon as complete
    // the low byte of y's bit pattern is the code (the low byte of the rounding constant is zero)
    ybits[j & 1][0] = __float_as_uint(y.x);
    ybits[j & 1][1] = __float_as_uint(y.y);
    if (j & 1) {
      const uint32_t p01 = __byte_perm(ybits[0][0], ybits[0][1], 0x0040);
      const uint32_t p23 = __byte_perm(ybits[1][0], ybits[1][1], 0x0040);
      cbytes[j >> 1] = __byte_perm(p01, p23, 0x5410);             // codes 4k..4k+3, one per byte
    }
  }
}

template <bool FAST, typename Sink>
__device__ __forceinline__ void q4k_subblock(const uint32_t (&w)[16], float lo_raw, float hi, const Sink sink,
                                             uint32_t (&cbytes)[8], __half& d_h, __half& dmin_h, uint32_t& s6, uint32_t& m6) {
  const float lo = fminf(lo_raw, 0.0f);
  const float sc = div_by<FAST>(__fsub_rn(hi, lo), 15.0f, kRcp15);
  const float off = __fsub_rn(0.0f, lo);            // >= +0: a sub-block with no negative value has offset +0
  float max_sc = sc, max_off = off;
#pragma unroll
  for (int s = 1; s < 8; s <<= 1) {
    max_sc = fmaxf(max_sc, __shfl_xor_sync(0xFFFFFFFFu, max_sc, s));
    max_off = fmaxf(max_off, __shfl_xor_sync(0xFFFFFFFFu, max_off, s));
  }
  d_h = __float2half_rn(fminf(div_by<FAST>(max_sc, 63.0f, kRcp63), 65504.0f));
  dmin_h = __float2half_rn(fminf(div_by<FAST>(max_off, 63.0f, kRcp63), 65504.0f));
  const float d = __half2float(d_h), dmin = __half2float(dmin_h);
  // FP16 values are at least 2^-24, well inside the safe divisor range
  const float s6f = d == 0.0f ? 0.0f : fminf(fmaxf(rintf(div_by<FAST>(sc, d, __frcp_rn(d))), 0.0f), 63.0f);
  const float m6f = dmin == 0.0f ? 0.0f : fminf(fmaxf(rintf(div_by<FAST>(off, dmin, __frcp_rn(dmin))), 0.0f), 63.0f);
  s6 = static_cast<uint32_t>(s6f);
  m6 = static_cast<uint32_t>(m6f);
  const float es = __fmul_rn(d, s6f), em = __fmul_rn(dmin, m6f);
  const bool live = es > 0.0f;
  const float rc = live ? __frcp_rn(es) : 0.0f;
  if (FAST) {
    // The quotient (x + em) / es is monotone in x, so the sub-block's smallest and largest element bound every quotient;
    // when both ends round into [0, 15] (the usual case: the 6-bit rounding of scale and offset moves them by a few
    // percent of a step) the per-element clamp is left out. Same arithmetic as the loop, so the bound is exact.
    const float t_lo = div1_fast(__fadd_rn(lo_raw, em), es, rc), t_hi = div1_fast(__fadd_rn(hi, em), es, rc);
    const bool inside = t_lo >= -0.5f && t_hi < 15.5f;           // (a sub-block without a scale has rc = 0: both are 0)
    if (__all_sync(0xFFFFFFFFu, inside)) {
      q4k_elements<true, false>(w, es, em, rc, live, sink, cbytes);
      return;
    }
  }
  q4k_elements<FAST, true>(w, es, em, rc, live, sink, cbytes);
}

// Everything after the load of one sub-block (16 words in w, slot c holding chunk c ^ perm of the sub-block; perm = 0
// in the plain kernels): statistics, metadata, codes, dequantized values. `i` is the sub-block's index in the tensor.
template <typename Sink>
__device__ __forceinline__ void q4k_lane(const uint32_t (&w)[16], bool ok, int lane, const Sink sink, uint32_t perm,
                                         uint4* __restrict__ codes, uint4* __restrict__ scales, int64_t i, uint32_t codes_smem = 0) {
  __nv_bfloat162 mn = bits_bf2(w[0]), mx = bits_bf2(w[0]);
#pragma unroll
  for (int j = 1; j < 16; ++j) {
    mn = __hmin2(mn, bits_bf2(w[j]));
    mx = __hmax2(mx, bits_bf2(w[j]));
  }
  const float lo = fminf(bf16_lo(bf2_bits(mn)), bf16_hi(bf2_bits(mn)));
  const float hi = fmaxf(bf16_lo(bf2_bits(mx)), bf16_hi(bf2_bits(mx)));
  // the reciprocal-based division is exact away from the bottom of the FP32 range; a warp with a
  // tiny but non-zero range or offset takes the IEEE divide instead
  const float range = __fsub_rn(hi, fminf(lo, 0.0f)), offv = -fminf(lo, 0.0f);
  const bool fast_ok = (range == 0.0f || (range >= 0x1p-60f && range <= 0x1p60f)) && (offv == 0.0f || (offv >= 0x1p-60f && offv <= 0x1p60f));
  uint32_t cb[8], s6, m6;
  __half d_h, dmin_h;
  if (__all_sync(0xFFFFFFFFu, fast_ok)) q4k_subblock<true>(w, lo, hi, sink, cb, d_h, dmin_h, s6, m6);
  else q4k_subblock<false>(w, lo, hi, sink, cb, d_h, dmin_h, s6, m6);
  // cb[2c], cb[2c+1] hold the codes of slot c; put them back in chunk order (both lanes of a pair share perm)
  if (perm & 1u) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      uint32_t t = cb[k]; cb[k] = cb[2 + k]; cb[2 + k] = t;
      t = cb[4 + k]; cb[4 + k] = cb[6 + k]; cb[6 + k] = t;
    }
  }
  if (perm & 2u) {
#pragma unroll
    for (int k = 0; k < 4; ++k) { const uint32_t t = cb[k]; cb[k] = cb[4 + k]; cb[4 + k] = t; }
  }
  // code bytes: a 64-element chunk is the lane pair (2j, 2j+1); byte l = code[2j][l] | code[2j+1][l] << 4.
  // cb[k] holds codes 4k..4k+3 one per byte. The even lane forms bytes 0-15, the odd lane bytes 16-31.
  const bool odd = lane & 1;
  uint32_t mine[4], theirs[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint32_t send = odd ? cb[k] : cb[4 + k];            // what the partner needs from this lane
    theirs[k] = __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    mine[k] = odd ? cb[4 + k] : cb[k];
  }
  if (ok && codes) {
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) o[k] = odd ? (theirs[k] | (mine[k] << 4)) : (mine[k] | (theirs[k] << 4));
    // super-block = 8 lanes x 16 bytes = 128 bytes; chunk (lane/2 mod 4) owns 32 of them
    if (codes_smem) st_shared_v4(codes_smem, o[0], o[1], o[2], o[3]);      // staged: leaves with the warp's bulk store
    else codes[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  if (scales) {
    const int b = lane & 7;                                       // sub-block within its super-block
    uint32_t w0 = 0, w1 = 0, w2 = 0;                              // the 12 packed bytes as three words
    if (b < 4) {
      w0 = (s6 & 63u) << (8 * b);
      w1 = (m6 & 63u) << (8 * b);
    } else {
      w0 = ((s6 >> 4) << 6) << (8 * (b - 4));
      w1 = ((m6 >> 4) << 6) << (8 * (b - 4));
      w2 = ((s6 & 15u) | ((m6 & 15u) << 4)) << (8 * (b - 4));
    }
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) {
      w0 |= __shfl_xor_sync(0xFFFFFFFFu, w0, s);
      w1 |= __shfl_xor_sync(0xFFFFFFFFu, w1, s);
      w2 |= __shfl_xor_sync(0xFFFFFFFFu, w2, s);
    }
    if (ok && b == 0) {
      const uint32_t hdr = static_cast<uint32_t>(__half_as_ushort(d_h)) | (static_cast<uint32_t>(__half_as_ushort(dmin_h)) << 16);
      scales[i >> 3] = make_uint4(hdr, w0, w1, w2);
    }
  }
}

// grid-stride loop shared by the single-tensor and the batched Q4_K kernels: sub-blocks first, first + stride, ...
template <typename Loader>
__device__ __forceinline__ void qdq_q4k_body(const Loader& in, int64_t nsub, uint4* __restrict__ out, uint4* __restrict__ codes,
                                             uint4* __restrict__ scales, int64_t first, int64_t stride) {
  const int lane = threadIdx.x & 31;
  // nsub (sub-blocks) is a multiple of 8; a warp covers 32 of them, so the last warp may be partly idle
  for (int64_t i = first; i - lane < nsub; i += stride) {
    const bool ok = i < nsub;
    uint32_t w[16];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 v = ok ? in.chunk(4 * i + k) : make_uint4(0, 0, 0, 0);
      w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
    }
    q4k_lane(w, ok, lane, GlobalSink{(ok && out) ? out + 4 * i : nullptr}, 0u, codes, scales, i);
  }
}

// ---- staged form --------------------------------------------------------------------------------------------------
// The kernels above address global memory with a 64-byte stride between lanes (a lane owns a whole sub-block), which
// costs the load/store data pipe several wavefronts per access: it is that pipe, at 76% of its peak, that holds the
// plain kernel at 0.90 of the copy rate. Here the input travels global -> shared and the dequantized output shared ->
// global as bulk asynchronous copies (a producer warp, a ring of mbarrier-guarded stages), and the lanes read and write
// their 64-byte records in shared memory in a lane-dependent chunk order (slot c = chunk c ^ ((lane >> 1) & 3)) that
// makes every 16-byte access bank-conflict free. Codes and metadata are already written with unit stride.
constexpr int kQ4kTile = 256;                               // sub-blocks per tile: one per consumer thread, 16 KB of input
constexpr int kQ4kStagesIn = 2, kQ4kStagesOut = 2;
constexpr int kQ4kStagedThreads = kQ4kTile + 32;            // + the producer warp
constexpr int kQ4kTileBytes = kQ4kTile * 64;
constexpr int kQ4kCodeBytes = kQ4kTile * 16;                 // packed codes of one tile
constexpr int kQ4kStagedSmem = (kQ4kStagesIn + kQ4kStagesOut) * kQ4kTileBytes + kQ4kStagesOut * kQ4kCodeBytes + 1024;

__global__ void __launch_bounds__(kQ4kStagedThreads, 3) qdq_q4k_staged_kernel(const uint8_t* __restrict__ in, int64_t nsub,
                                                                               uint8_t* __restrict__ out, uint4* __restrict__ codes,
                                                                               uint4* __restrict__ scales, uint32_t* __restrict__ status) {
  extern __shared__ uint8_t q4k_smem_raw[];
  __shared__ uint64_t full[kQ4kStagesIn], empty[kQ4kStagesIn];
  __shared__ int abort_flag;
  const uint32_t base = (smem_u32(q4k_smem_raw) + 127u) & ~127u;
  const uint32_t out_base = base + kQ4kStagesIn * kQ4kTileBytes;
  const uint32_t code_base = out_base + kQ4kStagesOut * kQ4kTileBytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < kQ4kStagesIn; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), kQ4kTile / 32);          // one arrival per consumer warp
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  const int64_t ntiles = (nsub + kQ4kTile - 1) / kQ4kTile;
  if (warp == kQ4kTile / 32) {
    // ===== producer: one lane feeds the ring =====
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        if (!mbar_wait(smem_u32(&empty[stage]), phase ^ 1u, &abort_flag, status)) break;
        const int64_t first = t * kQ4kTile;
        const uint32_t bytes = static_cast<uint32_t>(min(static_cast<int64_t>(kQ4kTile), nsub - first)) * 64u;
        mbar_expect_tx(smem_u32(&full[stage]), bytes);
        bulk_load(base + stage * kQ4kTileBytes, in + first * 64, bytes, smem_u32(&full[stage]));
        if (++stage == kQ4kStagesIn) { stage = 0; phase ^= 1u; }
      }
    }
    return;
  }
  // ===== consumers: thread tid owns sub-block tid of each tile =====
  const uint32_t perm = (static_cast<uint32_t>(lane) >> 1) & 3u;
  uint32_t stage = 0, phase = 0, local = 0;
  for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++local) {
    const int64_t i = t * kQ4kTile + tid;
    const bool ok = i < nsub;
    int got = 1;
    if (lane == 0) got = mbar_wait(smem_u32(&full[stage]), phase, &abort_flag, status) ? 1 : 0;
    got = __shfl_sync(0xFFFFFFFFu, got, 0);
    if (!got) break;
    uint32_t w[16];
    const uint32_t rec = base + stage * kQ4kTileBytes + static_cast<uint32_t>(tid) * 64u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 v = ok ? ld_shared_v4(rec + ((static_cast<uint32_t>(k) ^ perm) << 4)) : make_uint4(0, 0, 0, 0);
      w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&empty[stage]));       // the record is in registers: the stage can be refilled
    if (++stage == kQ4kStagesIn) { stage = 0; phase ^= 1u; }
    // each warp stages and stores its own 32 records (2 KB of values, 512 bytes of codes): no block-wide synchronisation
    // on the output side
    const uint32_t obuf = out_base + (local & 1u) * kQ4kTileBytes + static_cast<uint32_t>(warp) * 2048u;
    const uint32_t cbuf = code_base + (local & 1u) * kQ4kCodeBytes + static_cast<uint32_t>(warp) * 512u;
    // the staging buffers about to be rewritten were the sources of the bulk stores this warp issued two tiles ago
    if (lane == 0) bulk_wait_group_read<1>();
    __syncwarp();
    q4k_lane(w, ok, lane, SmemSink{obuf + static_cast<uint32_t>(lane) * 64u, perm, out != nullptr && ok}, perm, codes, scales, i,
             cbuf + static_cast<uint32_t>(lane) * 16u);
    fence_proxy_async_smem();                                  // generic-proxy writes -> visible to the bulk copies
    __syncwarp();
    if (lane == 0) {
      const int64_t first = t * kQ4kTile + warp * 32;
      const int64_t left = nsub - first;
      if (left > 0) {
        const uint32_t n = static_cast<uint32_t>(left < 32 ? left : 32);
        if (out) bulk_store(out + first * 64, obuf, n * 64u);
        if (codes) bulk_store(codes + first, cbuf, n * 16u);
      }
      bulk_commit_group();
    }
  }
  if (lane == 0) bulk_wait_group_all();                        // every store of this warp has left shared memory and landed
}

template <typename Loader>
__global__ void __launch_bounds__(kThreads, QF_Q4K_MINBLOCKS) qdq_q4k_kernel(Loader in, int64_t nsub,
                                                           uint4* __restrict__ out, uint4* __restrict__ codes,
                                                           uint4* __restrict__ scales) {
  qdq_q4k_body<Loader>(in, nsub, out, codes, scales, static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x,
                       static_cast<int64_t>(gridDim.x) * kThreads);
}

__global__ void __launch_bounds__(kThreads, QF_Q4K_MINBLOCKS) qdq_q4k_batched_kernel(const __grid_constant__ QdqBatch q) {
  const int t = blockIdx.y;
  const int64_t nsub = q.nunits[t];
  if (static_cast<int64_t>(blockIdx.x) * kThreads >= nsub) return;
  qdq_q4k_body<PlainLoader>(PlainLoader{q.in[t]}, nsub, q.out[t], static_cast<uint4*>(q.codes[t]), static_cast<uint4*>(q.scales[t]),
                            static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x, static_cast<int64_t>(gridDim.x) * kThreads);
}

// exhaustive comparison of the reciprocal-based division with the IEEE divide: every x in xs against
// every y in ys (and, with bf16_sweep, every non-negative BF16 bit pattern as x)
__global__ void selftest_div_kernel(const float* __restrict__ xs, int64_t nx, const float* __restrict__ ys, int64_t ny,
                                    unsigned long long* __restrict__ mismatches) {
  const int64_t total = nx * ny;
  unsigned long long bad = 0;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const float x = xs[i % nx], y = ys[i / nx];
    if (!div_safe(y)) continue;
    const float rc = __frcp_rn(y);
    const float ref = __fdiv_rn(x, y);
    // Domain in which the kernels rely on exactness: a numerator that is zero or not tiny, or a
    // quotient large enough to sit near a rounding threshold (those start at 0.25). A tiny quotient
    // of a tiny numerator may differ in its last bit (the residual underflows) but rounds to code 0
    // either way. Quotients beyond 2^100 never occur (the callers bound the numerator by 8 * divisor).
    if (!(x == 0.0f || fabsf(x) >= 0x1p-60f || fabsf(ref) >= 0x1p-8f) || fabsf(ref) > 0x1p100f) continue;
    const float2 q = div2_fast(make_float2(x, -x), y, rc);
    const float q1 = div1_fast(x, y, rc);
    if (__float_as_uint(q.x) != __float_as_uint(ref)) ++bad;             // bit patterns: the sign of a zero counts
    if (__float_as_uint(q.y) != __float_as_uint(-ref)) ++bad;
    if (__float_as_uint(q1) != __float_as_uint(ref)) ++bad;
  }
  if (bad) atomicAdd(mismatches, bad);
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

// every BF16 bit pattern x against every scale code the packed-BF16 MXFP4 rounding is used for:
// it must give the same BF16 result as the conversion-instruction route
__global__ void selftest_mxfp4_bf16_kernel(unsigned long long* __restrict__ mismatches) {
  const uint32_t code = 8u + blockIdx.x;                    // grid = 233 blocks: codes 8 .. 240
  const float2 inv = splat(e8m0_inv_scale(code)), sc = splat(e8m0_scale(code));
  const uint32_t one2 = mxfp4_one2(code), six2 = mxfp4_six2(code);
  const uint32_t amax_hi = ((code + 2u) << 7) | 0x7Fu;      // the largest |x| a block with this scale can hold
  unsigned long long bad = 0;
  for (uint32_t x = threadIdx.x; x < 0x10000u; x += blockDim.x) {
    if ((x & 0x7FFFu) > amax_hi) continue;
    const uint32_t w = x | (((x * 40503u) & 0xFFFFu) << 16);  // pair it with another pattern in the high half
    const uint32_t hi = (w >> 16) & 0x7FFFu;
    const uint32_t w2 = hi > amax_hi ? (w & 0xFFFFu) : w;
    if (mxfp4_qdq_pair(w2, inv, sc, 0xFFu) != mxfp4_qdq_pair_bf16(w2, one2, six2)) ++bad;
  }
  if (bad) atomicAdd(mismatches, bad);
}

int grid_for(int64_t nchunks, int per_thread) {
  int64_t blocks = (nchunks + static_cast<int64_t>(kThreads) * per_thread - 1) / (static_cast<int64_t>(kThreads) * per_thread);
  const int64_t cap = static_cast<int64_t>(kNumSMs) * 8;       // 8 resident blocks of 256 threads per SM
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

// Grid for the grid-stride QDQ kernels: enough blocks for the work, capped at `blocks_per_sm` x SM
// count. Measured on B200 (235 MB tensor): MXFP4 is fastest with no cap at all (one pass per thread:
// 6.4 TB/s against 5.0 TB/s with exactly one resident wave), NVFP4 and Q4_K level off at 16-32 per SM.
int capped_grid(int64_t items, int per_thread, int blocks_per_sm) {
  int64_t blocks = (items + static_cast<int64_t>(kThreads) * per_thread - 1) / (static_cast<int64_t>(kThreads) * per_thread);
  if (blocks_per_sm > 0) {
    const int64_t cap = static_cast<int64_t>(kNumSMs) * blocks_per_sm;
    if (blocks > cap) blocks = cap;
  }
  if (blocks > 0x7FFFFFFF) blocks = 0x7FFFFFFF;
  if (blocks < 1) blocks = 1;
  return static_cast<int>(blocks);
}

}  // namespace

// G tensors of n elements each, stored back to back (n a multiple of 8): amax_bits[g] = max |x| of tensor g
cudaError_t launch_amax_grouped(const void* in, int64_t n, int G, uint32_t* amax_bits, cudaStream_t st) {
  const int64_t nchunks = n / 8;
  if (G <= 0 || nchunks == 0) return cudaSuccess;
  int gx = grid_for(nchunks, 4);
  const int cap = (kNumSMs * 8 + G - 1) / G;
  if (gx > cap) gx = cap < 1 ? 1 : cap;
  amax_kernel<PlainLoader><<<dim3(gx, G), kThreads, 0, st>>>(PlainLoader{static_cast<const uint4*>(in)}, nchunks, nullptr, 0, amax_bits);
  return cudaGetLastError();
}

cudaError_t launch_amax(const void* in, int64_t n, uint32_t* amax_bits, cudaStream_t st) {
  const int64_t nchunks = n / 8;
  const int ntail = static_cast<int>(n % 8);
  amax_kernel<PlainLoader><<<grid_for(nchunks, 4), kThreads, 0, st>>>(PlainLoader{static_cast<const uint4*>(in)}, nchunks,
                                                                      static_cast<const __nv_bfloat16*>(in) + nchunks * 8, ntail,
                                                                      amax_bits);
  return cudaGetLastError();
}

// ---- batched launches --------------------------------------------------------------------------------
// Many tensors per call (every linear weight of a model is quantized each step for weight synchronisation, Section 3.4):
// MXFP4, Q4_K and NVFP4 with supplied scales take one launch per 64 tensors. NVFP4 with derived scales needs every
// tensor's maximum before its blocks can be scaled; the batch is cut into sub-batches of kSubBatchBytes of input, and
// launch j quantizes sub-batch j-1 while its spare y-slices take the maxima of sub-batch j: S + 1 launches for S
// sub-batches instead of three per tensor, with part of the second read of every tensor served from L2. With speculated scales (the previous step's) one launch quantizes with the guesses and gathers the
// true maxima, a second one derives the scales and requantizes only the tensors whose guess was wrong.
// Measured on B200 with 32 tensors of 8 MB: the rate climbs with the sub-batch size up to about 40 MB (fewer launches) and is
// flat from there to 128 MB (3.9-4.2 TB/s); six resident blocks per SM beat four and sixteen.
constexpr int64_t kSubBatchBytes = 56ll << 20;
constexpr int kBatchBlocksPerSm = 6;

static int batched_grid_x(int64_t max_items, int per_thread, int ny, int blocks_per_sm) {
  int64_t gx = (max_items + static_cast<int64_t>(kThreads) * per_thread - 1) / (static_cast<int64_t>(kThreads) * per_thread);
  if (blocks_per_sm > 0) {
    const int64_t cap = (static_cast<int64_t>(kNumSMs) * blocks_per_sm + ny - 1) / ny;
    if (gx > cap) gx = cap;
  }
  if (gx > 0x7FFFFFFF) gx = 0x7FFFFFFF;
  return static_cast<int>(gx < 1 ? 1 : gx);
}

cudaError_t launch_qdq_batched(const QdqBatchArgs& a, cudaStream_t st) {
  const int unit = a.fmt == QF_FMT_Q4_K ? 32 : 16;
  auto fill = [&](QdqBatch& q, int t0, int cnt, int64_t& max_units) {
    max_units = 0;
    for (int i = 0; i < cnt; ++i) {
      const int t = t0 + i;
      q.in[i] = static_cast<const uint4*>(a.in[t]);
      q.out[i] = a.out ? static_cast<uint4*>(a.out[t]) : nullptr;
      q.codes[i] = a.codes ? a.codes[t] : nullptr;
      q.scales[i] = a.scales ? a.scales[t] : nullptr;
      q.nunits[i] = a.rows[t] * a.cols[t] / unit;
      if (q.nunits[i] > max_units) max_units = q.nunits[i];
    }
  };
  const int opts = a.noclip ? 2 : 0;
  static const AmaxBatch no_amax{};
  if (a.fmt != QF_FMT_NVFP4 || a.given || a.speculative) {
    for (int t0 = 0; t0 < a.n; t0 += kMaxBatch) {
      const int cnt = a.n - t0 < kMaxBatch ? a.n - t0 : kMaxBatch;
      QdqBatch q{};
      int64_t mx;
      fill(q, t0, cnt, mx);
      if (a.fmt == QF_FMT_Q4_K) {
        qdq_q4k_batched_kernel<<<dim3(batched_grid_x(mx, 1, cnt, 32), cnt), kThreads, 0, st>>>(q);
      } else if (a.fmt == QF_FMT_MXFP4) {
        qdq_fp4_batched_kernel<QF_FMT_MXFP4><<<dim3(batched_grid_x(mx, kUnitsPerThread, cnt, 0), cnt), kThreads, 0, st>>>(
            q, cnt, no_amax, nullptr, nullptr, nullptr, opts, nullptr, nullptr, nullptr, nullptr);
      } else if (a.given) {
        qdq_fp4_batched_kernel<QF_FMT_NVFP4><<<dim3(batched_grid_x(mx, kUnitsPerThread, cnt, 16), cnt), kThreads, 0, st>>>(
            q, cnt, no_amax, a.tscales + t0, nullptr, nullptr, 0, nullptr, nullptr, nullptr, nullptr);
      } else {
        uint32_t* amax = a.ws_words + t0;
        uint32_t* guess = a.ws_words + a.n + t0;
        const dim3 grid(batched_grid_x(mx, kUnitsPerThread, cnt, 16), cnt);
        qdq_fp4_batched_kernel<QF_FMT_NVFP4><<<grid, kThreads, 0, st>>>(q, cnt, no_amax, a.tscales + t0, nullptr, nullptr, 0, amax,
                                                                        guess, nullptr, nullptr);
        if (cudaError_t e = cudaGetLastError()) return e;
        qdq_fp4_batched_kernel<QF_FMT_NVFP4><<<grid, kThreads, 0, st>>>(q, cnt, no_amax, nullptr, amax, a.tscales + t0, 0, nullptr,
                                                                        nullptr, guess, nullptr);
      }
      if (cudaError_t e = cudaGetLastError()) return e;
    }
    return cudaSuccess;
  }
  // NVFP4, derived scales: software pipeline over L2-sized sub-batches
  int prev0 = 0, prev_cnt = 0;             // the sub-batch whose maxima are already being gathered / are complete
  int t = 0;
  while (t < a.n || prev_cnt > 0) {
    int cnt = 0;
    int64_t bytes = 0;
    while (t + cnt < a.n && cnt < kMaxBatch) {
      const int64_t b = a.rows[t + cnt] * a.cols[t + cnt] * 2;
      if (cnt > 0 && bytes + b > kSubBatchBytes) break;
      bytes += b;
      ++cnt;
    }
    QdqBatch q{};
    AmaxBatch am{};
    int64_t mq = 0, ma = 0;
    if (prev_cnt > 0) fill(q, prev0, prev_cnt, mq);
    for (int i = 0; i < cnt; ++i) {
      am.in[i] = static_cast<const uint4*>(a.in[t + i]);
      am.nchunks[i] = a.rows[t + i] * a.cols[t + i] / 8;
      if (am.nchunks[i] > ma) ma = am.nchunks[i];
    }
    const int ny = prev_cnt + cnt;
    const int64_t gq = batched_grid_x(mq, kUnitsPerThread, ny, kBatchBlocksPerSm), ga = batched_grid_x(ma, 4, ny, kBatchBlocksPerSm);
    qdq_fp4_batched_kernel<QF_FMT_NVFP4><<<dim3(static_cast<unsigned>(gq > ga ? gq : ga), ny), kThreads, 0, st>>>(
        q, prev_cnt, am, nullptr, a.ws_words + prev0, a.tscales + prev0, 0, nullptr, nullptr, nullptr, a.ws_words + t);
    if (cudaError_t e = cudaGetLastError()) return e;
    prev0 = t;
    prev_cnt = cnt;
    t += cnt;
  }
  return cudaSuccess;
}

static LoraLoader lora_loader(const QdqArgs& a) {
  return LoraLoader{static_cast<const uint4*>(a.in), static_cast<const __nv_bfloat16*>(a.lora_B), static_cast<const uint4*>(a.lora_A),
                    a.lora_rank, a.lora_scale, a.cols / 8};
}

cudaError_t launch_amax_to_scale(const uint32_t* amax_bits, float* scale, cudaStream_t st) {
  amax_to_scale_kernel<<<1, 1, 0, st>>>(amax_bits, scale);
  return cudaGetLastError();
}

cudaError_t launch_amax_to_float(const uint32_t* amax_bits, float* out, cudaStream_t st) {
  amax_to_float_kernel<<<1, 1, 0, st>>>(amax_bits, out);
  return cudaGetLastError();
}

// The staged Q4_K kernel serves plain tensors of 2^25 elements and more: at 2^24 (4096 x 4096: under five tiles per CTA) its
// ramp-up and tail still cost more than the plain kernel's addressing (17.0 against 15.4 us); at 14336 x 4096 it wins
// (51.5 against 54.6 us, sustained).
template <typename Loader> static bool q4k_staged_applies(int64_t) { return false; }
template <> bool q4k_staged_applies<PlainLoader>(int64_t nsub) { return nsub >= (1ll << 20); }

static cudaError_t launch_q4k_staged(const QdqArgs& a, int64_t nsub, cudaStream_t st) {
  static bool configured[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    if (cudaError_t e = cudaFuncSetAttribute(qdq_q4k_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kQ4kStagedSmem)) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  const int64_t ntiles = (nsub + kQ4kTile - 1) / kQ4kTile;
  const int grid = static_cast<int>(ntiles < 3ll * kNumSMs ? ntiles : 3ll * kNumSMs);
  qdq_q4k_staged_kernel<<<grid, kQ4kStagedThreads, kQ4kStagedSmem, st>>>(static_cast<const uint8_t*>(a.in), nsub, static_cast<uint8_t*>(a.out),
                                                                          static_cast<uint4*>(a.codes), static_cast<uint4*>(a.scales), nullptr);
  return cudaGetLastError();
}

template <typename Loader>
static cudaError_t launch_qdq_with(const QdqArgs& a, const Loader& in, cudaStream_t st) {
  const int64_t nelem = a.rows * a.cols;
  uint4* out = static_cast<uint4*>(a.out);
  if (a.fmt == QF_FMT_NVFP4) {
    const int slices = a.groups > 1 ? a.groups : 1;
    const int64_t nunits = nelem / 16 / slices;
    int gx = capped_grid(nunits, kUnitsPerThread, 16);
    if (slices > 1 && gx > (kNumSMs * 16 + slices - 1) / slices) gx = (kNumSMs * 16 + slices - 1) / slices;
    qdq_fp4_kernel<QF_FMT_NVFP4, Loader><<<dim3(gx, slices), kThreads, 0, st>>>(
        in, nunits, out, static_cast<uint2*>(a.codes), static_cast<uint8_t*>(a.scales), a.tscale_in, a.amax_bits, a.tscale_out,
        a.reverse ? 1 : 0, a.spec);
  } else if (a.fmt == QF_FMT_MXFP4) {
    const int64_t nunits = nelem / 16;
    qdq_fp4_kernel<QF_FMT_MXFP4, Loader><<<capped_grid(nunits, kUnitsPerThread, 0), kThreads, 0, st>>>(
        in, nunits, out, static_cast<uint2*>(a.codes), static_cast<uint8_t*>(a.scales), nullptr, nullptr, nullptr,
        a.mxfp4_noclip ? 2 : 0, Nvfp4Speculation{a.spec.amax_accum, nullptr, nullptr});
  } else {
    const int64_t nsub = nelem / 32;
    if (q4k_staged_applies<Loader>(nsub)) return launch_q4k_staged(a, nsub, st);
    qdq_q4k_kernel<Loader><<<capped_grid(nsub, 1, 32), kThreads, 0, st>>>(in, nsub, out, static_cast<uint4*>(a.codes),
                                                                          static_cast<uint4*>(a.scales));
  }
  return cudaGetLastError();
}

cudaError_t launch_qdq(const QdqArgs& a, cudaStream_t st) {
  const int64_t nelem = a.rows * a.cols;
  // an empty NVFP4 tensor still has a tensor scale to report (1.0): let one block write it
  if (nelem == 0 && !(a.fmt == QF_FMT_NVFP4 && a.tscale_out)) return cudaSuccess;
  if (a.lora_rank > 0) return launch_qdq_with(a, lora_loader(a), st);
  return launch_qdq_with(a, PlainLoader{static_cast<const uint4*>(a.in)}, st);
}

// NVFP4 with a derived tensor scale: tensor amax, then quantize. The second pass walks the tensor
// from the END: the amax pass has just streamed it front to back, so its tail is what the 126 MB L2 still
// holds, and reading that first turns most of the re-read into L2 hits (all of it for tensors well
// below the L2 size). A single cooperative pass that kept the tensor in registers across a grid
// barrier was tried for tensors under 10 MB and measured no faster (12.3 us against 12.3 us for
// 2048 x 2048), because at that size L2 already serves the second read; it was dropped.
cudaError_t launch_qdq_nvfp4_derive(const QdqArgs& a, uint32_t* header, int amax_word, cudaStream_t st) {
  QdqArgs q = a;
  q.tscale_in = nullptr;
  if (a.groups > 1) {
    // per-expert tensor scales: the caller's scale array first accumulates the maxima (FP32 bits of a
    // non-negative value) and is then converted to the derived scales
    uint32_t* bits = reinterpret_cast<uint32_t*>(a.tscale_out);
    if (cudaError_t e = cudaMemsetAsync(bits, 0, sizeof(uint32_t) * a.groups, st)) return e;
    if (cudaError_t e = launch_amax_grouped(a.in, a.rows * a.cols / a.groups, a.groups, bits, st)) return e;
    // The maxima become scales in place before the quantize pass starts: that pass must find finished scales,
    // not words that one of its own CTAs is still turning from a maximum into a scale.
    amax_to_scale_inplace_kernel<<<(a.groups + kThreads - 1) / kThreads, kThreads, 0, st>>>(bits, a.groups);
    if (cudaError_t e = cudaGetLastError()) return e;
    q.tscale_in = a.tscale_out;
    q.tscale_out = nullptr;
    q.amax_bits = nullptr;
    return launch_qdq(q, st);
  }
  uint32_t* amax_bits = header + amax_word;
  if (a.lora_rank > 0) {
    // the absolute maximum is that of the merged weight, so the amax pass merges on the fly as well
    const int64_t nchunks = a.rows * a.cols / 8;
    if (nchunks > 0) amax_kernel<LoraLoader><<<grid_for(nchunks, 4), kThreads, 0, st>>>(lora_loader(a), nchunks, nullptr, 0, amax_bits);
    if (cudaError_t e = cudaGetLastError()) return e;
  } else {
    if (cudaError_t e = launch_amax(a.in, a.rows * a.cols, amax_bits, st)) return e;
    q.reverse = true;
  }
  q.amax_bits = amax_bits;
  return launch_qdq(q, st);
}

// Tensor scale(s) alone, for a caller that quantizes the tensor somewhere else (inside the matmul kernel): the maxima,
// then amax / (6 * 448) into a.tscale_out[0 .. groups-1]. `header` must have been zeroed on the stream beforehand.
cudaError_t launch_nvfp4_scales_only(const QdqArgs& a, uint32_t* header, int amax_word, cudaStream_t st) {
  if (a.groups > 1) {
    uint32_t* bits = reinterpret_cast<uint32_t*>(a.tscale_out);
    if (cudaError_t e = cudaMemsetAsync(bits, 0, sizeof(uint32_t) * a.groups, st)) return e;
    if (cudaError_t e = launch_amax_grouped(a.in, a.rows * a.cols / a.groups, a.groups, bits, st)) return e;
    amax_to_scale_inplace_kernel<<<(a.groups + kThreads - 1) / kThreads, kThreads, 0, st>>>(bits, a.groups);
    return cudaGetLastError();
  }
  if (cudaError_t e = launch_amax(a.in, a.rows * a.cols, header + amax_word, st)) return e;
  return launch_amax_to_scale(header + amax_word, a.tscale_out, st);
}

// NVFP4 with a guessed tensor scale in *a.tscale_out (say, the scale of the previous training step). Pass one quantizes
// with the guess and accumulates the true maximum on the way; pass two derives the scale from that maximum, writes it
// to *a.tscale_out and requantizes, unless it equals the guess bit for bit, in which case its CTAs return at once.
// The results are those of deriving the scale first, always; a right guess saves the separate read of the tensor.
// `header` must have been zeroed on the stream beforehand.
cudaError_t launch_qdq_nvfp4_speculative(const QdqArgs& a, uint32_t* header, int amax_word, int guess_word, cudaStream_t st) {
  // (in place, the first pass would destroy the input the second one may need: derive the scale first then)
  if (a.groups > 1 || a.lora_rank > 0 || !a.tscale_out || a.out == a.in) return launch_qdq_nvfp4_derive(a, header, amax_word, st);
  QdqArgs first = a;
  first.tscale_in = a.tscale_out;
  first.tscale_out = nullptr;
  first.amax_bits = nullptr;
  first.reverse = false;
  first.spec = Nvfp4Speculation{header + amax_word, header + guess_word, nullptr};
  if (cudaError_t e = launch_qdq(first, st)) return e;
  QdqArgs second = a;
  second.tscale_in = nullptr;
  second.amax_bits = header + amax_word;
  second.reverse = true;
  second.spec = Nvfp4Speculation{nullptr, nullptr, header + guess_word};
  return launch_qdq(second, st);
}

cudaError_t launch_selftest_mxfp4_bf16(unsigned long long* mismatches, cudaStream_t st) {
  selftest_mxfp4_bf16_kernel<<<233, 256, 0, st>>>(mismatches);
  return cudaGetLastError();
}

cudaError_t launch_selftest_div(const float* xs, int64_t nx, const float* ys, int64_t ny, unsigned long long* mismatches,
                                cudaStream_t st) {
  if (nx == 0 || ny == 0) return cudaSuccess;
  selftest_div_kernel<<<kNumSMs * 8, 256, 0, st>>>(xs, nx, ys, ny, mismatches);
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
