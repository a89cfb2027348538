// C ABI of libqf.so: argument validation, workspace carving, and the launch sequences of the
// quantizer and of the quantization-aware linear layer (forward and straight-through backward).
// Nothing here computes; every step of the path runs in the kernels of qf_qdq.cu / qf_gemm.cu.
// The only state kept between calls is per-device caches of facts that never change (compute capability,
// kernel attributes already set, the device address of the allocation-free entry point's built-in buffer).
#include <stdio.h>

#include "qf_common.cuh"

namespace qf {
namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round256(size_t b) { return (b + 255) & ~static_cast<size_t>(255); }

inline int block_of(int fmt) {
  switch (fmt) {
    case QF_FMT_NVFP4: return 16;
    case QF_FMT_MXFP4: return 32;
    case QF_FMT_Q4_K: return 256;
    default: return 0;
  }
}
inline bool valid_fmt(int fmt, bool allow_none) { return (fmt >= (allow_none ? 0 : 1)) && fmt <= 3; }

// The device must be a compute-capability 10.x part: the kernels are built for sm_100a only.
qf_status_t check_arch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return QF_ERR_CUDA; }
  static int cached_major[64] = {0};
  int major = dev < 64 ? cached_major[dev] : 0;
  if (major == 0) {
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) { cudaGetLastError(); return QF_ERR_CUDA; }
    if (dev < 64) cached_major[dev] = major;
  }
  return major == 10 ? QF_OK : QF_ERR_ARCH;
}

inline qf_status_t cu(cudaError_t e) {
  if (e == cudaSuccess) return QF_OK;
  cudaGetLastError();
  return QF_ERR_CUDA;
}

struct Workspace {
  uint32_t* header;     // 64 words
  uint8_t* w_hat;       // fake-quantized weights
  uint8_t* x_hat;       // fake-quantized activations
};

size_t linear_ws_bytes(int64_t M, int64_t N, int64_t K, int64_t groups) {
  return kWsHeader + round256(static_cast<size_t>(groups) * N * K * 2) + round256(static_cast<size_t>(M) * K * 2);
}

Workspace carve(void* ws, int64_t N, int64_t K, int64_t groups) {
  Workspace w;
  uint8_t* base = static_cast<uint8_t*>(ws);
  w.header = reinterpret_cast<uint32_t*>(base);
  w.w_hat = base + kWsHeader;
  w.x_hat = w.w_hat + round256(static_cast<size_t>(groups) * N * K * 2);
  return w;
}

// Fake-quantize one operand into `dst` (BF16, same shape). NVFP4 derives or reads its tensor scale.
// `groups` > 1 (NVFP4 weights of a grouped layer): every expert has its own tensor scale, tscale_user is an
// array of `groups` floats (required).
qf_status_t quantize_operand(int fmt, const void* src, int64_t rows, int64_t cols, void* dst, float* tscale_user,
                             bool tscale_given, uint32_t* header, int amax_word, int scale_word, cudaStream_t st,
                             int groups = 1, bool mxfp4_noclip = false, bool speculative = false, uint32_t* amax_accum = nullptr) {
  QdqArgs q{};
  q.mxfp4_noclip = mxfp4_noclip;
  q.spec.amax_accum = amax_accum;       // FP4 formats, single pass: also accumulate max|src| there (zeroed beforehand)
  q.fmt = fmt;
  q.in = src;
  q.rows = rows;
  q.cols = cols;
  q.out = dst;
  q.groups = fmt == QF_FMT_NVFP4 ? groups : 1;
  if (fmt == QF_FMT_NVFP4) {
    if (tscale_given) {
      q.tscale_in = tscale_user;
    } else {
      q.tscale_out = tscale_user ? tscale_user : reinterpret_cast<float*>(header + scale_word);
      if (speculative && tscale_user && groups == 1) return cu(launch_qdq_nvfp4_speculative(q, header, amax_word, kWsGuessW, st));
      return cu(launch_qdq_nvfp4_derive(q, header, amax_word, st));
    }
  }
  return cu(launch_qdq(q, st));
}

// Tensor scale(s) of an NVFP4 operand that the matmul kernel quantizes itself (QF_FUSED_QDQ): *out receives a device
// pointer to the final scale(s) - the caller's when given, otherwise derived now from the operand's maximum (and written
// back to the caller's array when there is one), with the maximum left in header[amax_word] for single tensors.
qf_status_t fused_nvfp4_scale(const void* src, int64_t rows, int64_t cols, float* tscale_user, bool given, uint32_t* header,
                              int amax_word, int scale_word, int groups, cudaStream_t st, const float** out) {
  if (given) { *out = tscale_user; return QF_OK; }
  QdqArgs q{};
  q.fmt = QF_FMT_NVFP4;
  q.in = src;
  q.rows = rows;
  q.cols = cols;
  q.groups = groups;
  q.tscale_out = tscale_user ? tscale_user : reinterpret_cast<float*>(header + scale_word);
  *out = q.tscale_out;
  return cu(launch_nvfp4_scales_only(q, header, amax_word, st));
}

constexpr int64_t kWgradChunkRows = 16384;     // contraction rows per dW launch when the contraction is cut (a multiple of 64)

inline bool fusable_fmt(int fmt) { return fmt == QF_FMT_MXFP4 || fmt == QF_FMT_NVFP4; }

// Checks shared by the forward and backward calls. W may be NULL only when the caller does not need it
// (a backward call that asks for dW alone): need_w says whether it is required.
qf_status_t check_linear_common(const void* W, bool need_w, int64_t M, int64_t N, int64_t K, int wq, int aq, const float* w_ts,
                                const float* a_ts, uint32_t flags, void* ws, size_t ws_bytes, int64_t groups) {
  if (need_w && !W) return QF_ERR_NULL;
  if (!ws) return QF_ERR_WORKSPACE;
  if (M < 0 || N < 0 || K < 0) return QF_ERR_SHAPE;
  if (!valid_fmt(wq, true) || !valid_fmt(aq, true)) return QF_ERR_FORMAT;
  if (aq == QF_FMT_Q4_K) return QF_ERR_FORMAT;                    // Q4_K is a weight-only format
  if (K % 8 || N % 8) return QF_ERR_SHAPE;
  if (wq != QF_FMT_NONE && K % block_of(wq)) return QF_ERR_SHAPE;
  if (aq != QF_FMT_NONE && K % block_of(aq)) return QF_ERR_SHAPE;
  if (wq == QF_FMT_NVFP4 && (flags & QF_W_TSCALE_GIVEN) && !w_ts) return QF_ERR_NULL;
  if (wq == QF_FMT_NVFP4 && groups > 1 && !w_ts) return QF_ERR_NULL;       // one tensor scale per expert: the array is required
  if (aq == QF_FMT_NVFP4 && (flags & QF_A_TSCALE_GIVEN) && !a_ts) return QF_ERR_NULL;
  if ((W && !aligned16(W)) || !aligned16(ws)) return QF_ERR_ALIGN;
  if (ws_bytes < linear_ws_bytes(M, N, K, groups)) return QF_ERR_WORKSPACE;
  return QF_OK;
}

inline bool valid_dtype(int d) { return d == QF_DT_BF16 || d == QF_DT_F32; }

// Shared by the plain and the grouped calls (groups == 1 and offs == nullptr for the plain ones).
qf_status_t linear_fwd_impl(const void* X, const void* W, void* Y, int y_dtype, const int32_t* offs, int G, int64_t M,
                            int64_t N, int64_t K, int wq, int aq, float* w_ts, float* a_ts, float* a_amax_out,
                            uint32_t flags, void* ws, size_t ws_bytes, cudaStream_t st) {
  const bool grouped = offs != nullptr;
  const int64_t groups = grouped ? G : 1;
  const bool has_operands = M != 0 && N != 0 && K != 0;      // empty operands have no storage to point at
  if ((has_operands && !X) || (M != 0 && N != 0 && !Y)) return QF_ERR_NULL;
  if (!valid_dtype(y_dtype)) return QF_ERR_DTYPE;
  if (qf_status_t s = check_linear_common(W, has_operands, M, N, K, wq, aq, w_ts, a_ts, flags, ws, ws_bytes, groups)) return s;
  if (!aligned16(X) || !aligned16(Y)) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  if (M == 0 || N == 0) return QF_OK;
  if (K == 0)        // an empty contraction still defines the output: zeros
    return cu(cudaMemsetAsync(Y, 0, static_cast<size_t>(M) * N * (y_dtype == QF_DT_F32 ? 4 : 2), st));
  Workspace w = carve(ws, N, K, groups);
  if (cudaError_t e = cudaMemsetAsync(w.header, 0, kWsHeader, st)) return cu(e);
  GemmArgs g{};
  g.C = Y;
  g.Mo = M; g.No = N; g.Kc = K;
  g.lda = K; g.ldb = K; g.ldc = N;
  g.a_mn_major = false; g.b_mn_major = false;
  g.c_dtype = y_dtype;
  g.status_word = w.header + kWsStatus;
  g.mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
  if (grouped) {
    g.group_mode = 1; g.group_offsets = offs; g.G = G; g.rows_padded = M;
  }
  const bool may_fuse = (flags & QF_FUSED_QDQ) && gemm_can_fuse(g);
  const bool fuse_b = may_fuse && fusable_fmt(wq) && !(flags & QF_REUSE_W_HAT);
  const bool fuse_a = may_fuse && fusable_fmt(aq) && !(flags & QF_REUSE_X_HAT);
  const void* Wh = W;
  const void* Xh = X;
  if (fuse_b) {
    g.fuse_b_fmt = wq;
    g.fuse_b_tscale_per_group = groups > 1;
    if (wq == QF_FMT_NVFP4)
      if (qf_status_t s = fused_nvfp4_scale(W, groups * N, K, w_ts, flags & QF_W_TSCALE_GIVEN, w.header, kWsAmaxW, kWsScaleW, static_cast<int>(groups), st, &g.fuse_b_tscale)) return s;
  } else if (wq != QF_FMT_NONE) {
    if (!(flags & QF_REUSE_W_HAT))
      if (qf_status_t s = quantize_operand(wq, W, groups * N, K, w.w_hat, w_ts, flags & QF_W_TSCALE_GIVEN, w.header, kWsAmaxW, kWsScaleW, st, static_cast<int>(groups), (flags & QF_MXFP4_NO_CLIP) != 0, (flags & QF_W_TSCALE_SPECULATIVE) != 0)) return s;
    Wh = w.w_hat;
  }
  // max|X| for the caller's running maximum: taken from the pass that derives X's NVFP4 scale (its maximum word) or from
  // the single-pass FP4 quantizer over X (its own accumulator) where there is one, otherwise from a pass of its own
  const bool x_pass = aq != QF_FMT_NONE && !fuse_a && !(flags & QF_REUSE_X_HAT);
  const bool x_derives = aq == QF_FMT_NVFP4 && !(flags & QF_A_TSCALE_GIVEN) && (x_pass || fuse_a);
  const bool x_accumulates = x_pass && !x_derives && (aq == QF_FMT_NVFP4 || aq == QF_FMT_MXFP4);
  uint32_t* amax_word = a_amax_out ? (x_derives ? w.header + kWsAmaxA : w.header + kWsAmaxReport) : nullptr;
  if (a_amax_out && !x_derives && !x_accumulates)
    if (cudaError_t e = launch_amax(X, M * K, amax_word, st)) return cu(e);
  if (fuse_a) {
    g.fuse_a_fmt = aq;
    if (aq == QF_FMT_NVFP4)
      if (qf_status_t s = fused_nvfp4_scale(X, M, K, a_ts, flags & QF_A_TSCALE_GIVEN, w.header, kWsAmaxA, kWsScaleA, 1, st, &g.fuse_a_tscale)) return s;
  } else if (aq != QF_FMT_NONE) {
    if (!(flags & QF_REUSE_X_HAT))
      if (qf_status_t s = quantize_operand(aq, X, M, K, w.x_hat, a_ts, flags & QF_A_TSCALE_GIVEN, w.header, kWsAmaxA, kWsScaleA, st, 1, (flags & QF_MXFP4_NO_CLIP) != 0, false, (a_amax_out && x_accumulates) ? amax_word : nullptr)) return s;
    Xh = w.x_hat;
  }
  if (a_amax_out)
    if (cudaError_t e = launch_amax_to_float(amax_word, a_amax_out, st)) return cu(e);
  g.A = Xh; g.B = Wh;
  g.tile_sync_word = w.header + kWsTileSync;
  return cu(launch_gemm(g, st));
}

qf_status_t linear_bwd_impl(const void* dY, const void* X, const void* W, void* dX, int dx_dtype, void* dW, int dw_dtype,
                            const int32_t* offs, int G, int64_t M, int64_t N, int64_t K, int wq, int aq, float* w_ts,
                            float* a_ts, uint32_t flags, void* ws, size_t ws_bytes, cudaStream_t st) {
  const bool grouped = offs != nullptr;
  const int64_t groups = grouped ? G : 1;
  if (!dY) return QF_ERR_NULL;
  if (!dX && !dW) return QF_ERR_NULL;
  if (dW && !X) return QF_ERR_NULL;
  if ((dX && !valid_dtype(dx_dtype)) || (dW && !valid_dtype(dw_dtype))) return QF_ERR_DTYPE;
  if (qf_status_t s = check_linear_common(W, dX != nullptr, M, N, K, wq, aq, w_ts, a_ts, flags, ws, ws_bytes, groups)) return s;
  if (!aligned16(dY) || (X && !aligned16(X)) || (dX && !aligned16(dX)) || (dW && !aligned16(dW))) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  if (M == 0 || N == 0 || K == 0) {
    // an empty contraction still defines the outputs: they are zero (unless accumulating)
    if (dW && M == 0 && N > 0 && K > 0 && !(flags & QF_ACCUMULATE_DW))
      if (cudaError_t e = cudaMemsetAsync(dW, 0, static_cast<size_t>(groups) * N * K * (dw_dtype == QF_DT_F32 ? 4 : 2), st)) return cu(e);
    if (dX && N == 0 && M > 0 && K > 0)
      if (cudaError_t e = cudaMemsetAsync(dX, 0, static_cast<size_t>(M) * K * (dx_dtype == QF_DT_F32 ? 4 : 2), st)) return cu(e);
    return QF_OK;
  }
  Workspace w = carve(ws, N, K, groups);
  if (cudaError_t e = cudaMemsetAsync(w.header, 0, kWsHeader, st)) return cu(e);
  bool x_hat_done = false;          // X_hat already produced by a side job of the dX launch
  if (dX) {
    // dX[M,K] = dY[M,N] . W_hat[N,K]: A = dY contraction-major, B = W_hat stored [contraction N, K]
    GemmArgs g{};
    g.A = dY; g.C = dX;
    g.Mo = M; g.No = K; g.Kc = N;
    g.lda = N; g.ldb = K; g.ldc = K;
    g.a_mn_major = false; g.b_mn_major = true;
    g.c_dtype = dx_dtype;
    g.status_word = w.header + kWsStatus;
  g.mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
    if (grouped) { g.group_mode = 1; g.group_offsets = offs; g.G = G; g.rows_padded = M; }
    const bool fuse_b = (flags & QF_FUSED_QDQ) && fusable_fmt(wq) && !(flags & QF_REUSE_W_HAT) && gemm_can_fuse(g);
    const void* Wh = W;
    if (fuse_b) {
      g.fuse_b_fmt = wq;
      g.fuse_b_tscale_per_group = groups > 1;
      if (wq == QF_FMT_NVFP4)
        if (qf_status_t s = fused_nvfp4_scale(W, groups * N, K, w_ts, flags & QF_W_TSCALE_GIVEN, w.header, kWsAmaxW, kWsScaleW, static_cast<int>(groups), st, &g.fuse_b_tscale)) return s;
    } else if (wq != QF_FMT_NONE) {
      if (!(flags & QF_REUSE_W_HAT))
        if (qf_status_t s = quantize_operand(wq, W, groups * N, K, w.w_hat, w_ts, flags & QF_W_TSCALE_GIVEN, w.header, kWsAmaxW, kWsScaleW, st, static_cast<int>(groups), (flags & QF_MXFP4_NO_CLIP) != 0, (flags & QF_W_TSCALE_SPECULATIVE) != 0)) return s;
      Wh = w.w_hat;
    }
    g.B = Wh;
    // The activations' quantize pass belongs to the next product (dW). It is HBM-bound and this product is tensor-bound,
    // so where the kernel can carry it (MXFP4, or NVFP4 with a supplied scale) it runs as a side job of this launch.
    if (dW && (aq == QF_FMT_MXFP4 || (aq == QF_FMT_NVFP4 && (flags & QF_A_TSCALE_GIVEN))) && !(flags & (QF_REUSE_X_HAT | QF_FUSED_QDQ)) &&
        M * K > 0 && (M * K) % 32 == 0 && gemm_side_supported(g)) {
      g.side[0].in = X;
      g.side[0].out = w.x_hat;
      g.side[0].nelem = M * K;
      g.side[0].fmt = aq;
      g.side[0].tscale = a_ts;
      g.side[0].mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
      x_hat_done = true;
    }
    g.tile_sync_word = w.header + kWsTileSync;
    if (cudaError_t e = launch_gemm(g, st)) return cu(e);
  }
  if (dW) {
    // dW[N,K] = dY[M,N]^T . X_hat[M,K]: both operands stored [contraction M, rows]
    GemmArgs g{};
    g.A = dY; g.C = dW;
    g.Mo = N; g.No = K; g.Kc = M;
    g.lda = N; g.ldb = K; g.ldc = K;
    g.a_mn_major = true; g.b_mn_major = true;
    g.c_dtype = dw_dtype;
    g.accumulate = (flags & QF_ACCUMULATE_DW) != 0;
    g.status_word = w.header + kWsStatus;
  g.mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
    if (grouped) { g.group_mode = 2; g.group_offsets = offs; g.G = G; g.rows_padded = M; g.c_group_stride = N * K; }
    const bool fuse_b = (flags & QF_FUSED_QDQ) && fusable_fmt(aq) && !(flags & QF_REUSE_X_HAT) && gemm_can_fuse(g);
    const void* Xh = X;
    if (fuse_b) {
      g.fuse_b_fmt = aq;                 // the activations are this product's B operand; one scale for all of X
      if (aq == QF_FMT_NVFP4)
        if (qf_status_t s = fused_nvfp4_scale(X, M, K, a_ts, flags & QF_A_TSCALE_GIVEN, w.header, kWsAmaxA, kWsScaleA, 1, st, &g.fuse_b_tscale)) return s;
    } else if (aq != QF_FMT_NONE) {
      if (!(flags & QF_REUSE_X_HAT) && !x_hat_done)
        if (qf_status_t s = quantize_operand(aq, X, M, K, w.x_hat, a_ts, flags & QF_A_TSCALE_GIVEN, w.header, kWsAmaxA, kWsScaleA, st, 1, (flags & QF_MXFP4_NO_CLIP) != 0)) return s;
      Xh = w.x_hat;
    }
    g.B = Xh;
    // A very long contraction (M tokens) makes the operand panels of a tile too long to be shared through L2 by the CTAs
    // that need them (measured at M = 32768: 8-10 GB of DRAM reads per launch against 1.2 GB of operands). With an FP32
    // output the contraction is cut into chunks of kWgradChunkRows tokens, one launch each, the later ones adding into dW
    // through the epilogue's TMA add-reduce: 5.1 GB and 6% less time at M = 32768.
    const int64_t chunks = (!grouped && dw_dtype == QF_DT_F32 && !fuse_b && M >= 2 * kWgradChunkRows) ? (M + kWgradChunkRows - 1) / kWgradChunkRows : 1;
    for (int64_t c = 0; c < chunks; ++c) {
      const int64_t r0 = c * kWgradChunkRows;
      GemmArgs gc = g;
      gc.tile_sync_word = c + 1 < kWsTileSyncCount ? w.header + kWsTileSync + 1 + c : nullptr;
      if (chunks > 1) {
        gc.A = static_cast<const uint8_t*>(g.A) + static_cast<size_t>(r0) * N * 2;
        gc.B = static_cast<const uint8_t*>(g.B) + static_cast<size_t>(r0) * K * 2;
        gc.Kc = (M - r0 < kWgradChunkRows) ? M - r0 : kWgradChunkRows;
        gc.accumulate = g.accumulate || c > 0;
      }
      if (cudaError_t e = launch_gemm(gc, st)) return cu(e);
    }
  }
  return QF_OK;
}

}  // namespace
}  // namespace qf

using namespace qf;

extern "C" {

const char* qf_status_string(qf_status_t s) {
  switch (s) {
    case QF_OK: return "ok";
    case QF_ERR_NULL: return "a required pointer is NULL";
    case QF_ERR_SHAPE: return "bad shape (negative, or not a multiple of the block / vector width)";
    case QF_ERR_ALIGN: return "pointer not 16-byte aligned";
    case QF_ERR_FORMAT: return "unknown format, or format not allowed for this operand";
    case QF_ERR_WORKSPACE: return "workspace missing or too small";
    case QF_ERR_CUDA: return "CUDA call failed";
    case QF_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case QF_ERR_ARCH: return "device is not compute capability 10.x";
    case QF_ERR_DTYPE: return "unknown output dtype";
    case QF_ERR_TOO_LARGE: return "problem needs more scratch than the built-in buffer of the allocation-free entry point";
  }
  return "unknown status";
}

int qf_version(void) { return 100; }

size_t qf_workspace_bytes(qf_op_t op, int64_t M, int64_t N, int64_t K, int groups) {
  if (M < 0) M = 0;
  if (N < 0) N = 0;
  if (K < 0) K = 0;
  if (op == QF_OP_QDQ) return kWsHeader;
  if (op == QF_OP_QDQ_BATCHED) return kWsHeader + round256(8 * static_cast<size_t>(groups > 0 ? groups : 0));
  const int64_t g = (op == QF_OP_GROUPED_FWD || op == QF_OP_GROUPED_BWD) ? (groups > 0 ? groups : 1) : 1;
  return linear_ws_bytes(M, N, K, g);
}

qf_status_t qf_read_status(const void* workspace, void* stream, int* host_status_out) {
  if (!workspace || !host_status_out) return QF_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaError_t e = cudaStreamSynchronize(st)) return cu(e);
  uint32_t v = 0;
  if (cudaError_t e = cudaMemcpy(&v, workspace, 4, cudaMemcpyDeviceToHost)) return cu(e);
  *host_status_out = static_cast<int>(v);
  return QF_OK;
}

qf_status_t qf_qdq(qf_format_t fmt, const void* in, int64_t rows, int64_t cols, void* out_bf16, void* codes,
                   void* scales, float* tensor_scale, uint32_t flags, void* workspace, size_t workspace_bytes,
                   void* stream) {
  if (!valid_fmt(fmt, false)) return QF_ERR_FORMAT;
  if (rows < 0 || cols < 0 || cols % block_of(fmt)) return QF_ERR_SHAPE;
  const bool empty = rows == 0 || cols == 0;            // an empty tensor has no data pointers to check
  if (!empty && !in) return QF_ERR_NULL;
  if (!empty && !out_bf16 && !codes && !scales) return QF_ERR_NULL;
  if (fmt == QF_FMT_NVFP4 && !tensor_scale) return QF_ERR_NULL;
  if (!aligned16(in) || (out_bf16 && !aligned16(out_bf16)) || (codes && !aligned16(codes)) || (scales && !aligned16(scales)))
    return QF_ERR_ALIGN;
  const bool need_amax = fmt == QF_FMT_NVFP4 && !(flags & QF_TENSOR_SCALE_GIVEN);
  if (need_amax) {
    if (!workspace || workspace_bytes < kWsHeader) return QF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QF_ERR_ALIGN;
  }
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  QdqArgs q{};
  q.fmt = fmt;
  q.in = in;
  q.rows = rows;
  q.cols = cols;
  q.out = out_bf16;
  q.codes = codes;
  q.scales = scales;
  q.mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
  if (fmt == QF_FMT_NVFP4) {
    if (need_amax) {
      uint32_t* header = static_cast<uint32_t*>(workspace);
      if (cudaError_t e = cudaMemsetAsync(header, 0, kWsHeader, st)) return cu(e);
      q.tscale_out = tensor_scale;
      if ((flags & QF_TENSOR_SCALE_SPECULATIVE) && tensor_scale) return cu(launch_qdq_nvfp4_speculative(q, header, kWsAmaxW, kWsGuessW, st));
      return cu(launch_qdq_nvfp4_derive(q, header, kWsAmaxW, st));
    } else {
      q.tscale_in = tensor_scale;
    }
  }
  return cu(launch_qdq(q, st));
}

qf_status_t qf_qdq_batched(qf_format_t fmt, int n, const void* const* in, const int64_t* rows, const int64_t* cols,
                           void* const* out_bf16, void* const* codes, void* const* scales, float* tensor_scales, uint32_t flags,
                           void* workspace, size_t workspace_bytes, void* stream) {
  if (!valid_fmt(fmt, false)) return QF_ERR_FORMAT;
  if (n < 0) return QF_ERR_SHAPE;
  if (n == 0) return QF_OK;
  if (!in || !rows || !cols) return QF_ERR_NULL;
  if (fmt == QF_FMT_NVFP4 && !tensor_scales) return QF_ERR_NULL;
  bool in_place = false;
  for (int i = 0; i < n; ++i) {
    if (rows[i] < 0 || cols[i] < 0 || cols[i] % block_of(fmt)) return QF_ERR_SHAPE;
    const bool empty = rows[i] == 0 || cols[i] == 0;
    void* o = out_bf16 ? out_bf16[i] : nullptr;
    void* c = codes ? codes[i] : nullptr;
    void* sc = scales ? scales[i] : nullptr;
    if (!empty && (!in[i] || (!o && !c && !sc))) return QF_ERR_NULL;
    if (!aligned16(in[i]) || !aligned16(o) || !aligned16(c) || !aligned16(sc)) return QF_ERR_ALIGN;
    if (!empty && o == in[i]) in_place = true;
  }
  const bool given = fmt == QF_FMT_NVFP4 && (flags & QF_TENSOR_SCALE_GIVEN);
  const bool need_ws = fmt == QF_FMT_NVFP4 && !given;
  const size_t ws_need = kWsHeader + round256(8 * static_cast<size_t>(n));
  if (need_ws) {
    if (!workspace || workspace_bytes < ws_need) return QF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QF_ERR_ALIGN;
  }
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  QdqBatchArgs a{};
  a.fmt = fmt;
  a.n = n;
  a.in = in; a.rows = rows; a.cols = cols;
  a.out = out_bf16; a.codes = codes; a.scales = scales;
  a.tscales = tensor_scales;
  a.given = given;
  // a first pass with a guessed scale would overwrite an input that the second pass may still need
  a.speculative = need_ws && (flags & QF_TENSOR_SCALE_SPECULATIVE) && !in_place;
  a.noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
  if (need_ws) {
    if (cudaError_t e = cudaMemsetAsync(workspace, 0, ws_need, st)) return cu(e);
    a.ws_words = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(workspace) + kWsHeader);
  }
  return cu(launch_qdq_batched(a, st));
}

qf_status_t qf_qdq_lora(qf_format_t fmt, const void* W, const void* B, const void* A, int rank, float lora_scale, int64_t rows,
                        int64_t cols, void* out_bf16, void* codes, void* scales, float* tensor_scale, uint32_t flags,
                        void* workspace, size_t workspace_bytes, void* stream) {
  if (!valid_fmt(fmt, false)) return QF_ERR_FORMAT;
  if (rows < 0 || cols < 0 || cols % block_of(fmt) || rank < 0 || rank > 1024) return QF_ERR_SHAPE;
  const bool empty = rows == 0 || cols == 0;
  if (!empty && (!W || (rank > 0 && (!B || !A)))) return QF_ERR_NULL;
  if (!empty && !out_bf16 && !codes && !scales) return QF_ERR_NULL;
  if (fmt == QF_FMT_NVFP4 && !tensor_scale) return QF_ERR_NULL;
  if (!aligned16(W) || !aligned16(A) || (out_bf16 && !aligned16(out_bf16)) || (codes && !aligned16(codes)) ||
      (scales && !aligned16(scales)))
    return QF_ERR_ALIGN;
  if (B && (reinterpret_cast<uintptr_t>(B) & 1u)) return QF_ERR_ALIGN;
  const bool need_amax = fmt == QF_FMT_NVFP4 && !(flags & QF_TENSOR_SCALE_GIVEN);
  if (need_amax) {
    if (!workspace || workspace_bytes < kWsHeader) return QF_ERR_WORKSPACE;
    if (!aligned16(workspace)) return QF_ERR_ALIGN;
  }
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  QdqArgs q{};
  q.fmt = fmt;
  q.in = W;
  q.rows = rows;
  q.cols = cols;
  q.out = out_bf16;
  q.codes = codes;
  q.scales = scales;
  q.mxfp4_noclip = (flags & QF_MXFP4_NO_CLIP) != 0;
  q.lora_B = B;
  q.lora_A = A;
  q.lora_rank = empty ? 0 : rank;
  q.lora_scale = lora_scale;
  if (fmt == QF_FMT_NVFP4) {
    if (need_amax) {
      uint32_t* header = static_cast<uint32_t*>(workspace);
      if (cudaError_t e = cudaMemsetAsync(header, 0, kWsHeader, st)) return cu(e);
      q.tscale_out = tensor_scale;
      return cu(launch_qdq_nvfp4_derive(q, header, kWsAmaxW, st));
    }
    q.tscale_in = tensor_scale;
  }
  return cu(launch_qdq(q, st));
}

qf_status_t qf_dequant(qf_format_t fmt, const void* codes, const void* scales, const float* tensor_scale, int64_t rows,
                       int64_t cols, void* out_bf16, void* stream) {
  if (!valid_fmt(fmt, false)) return QF_ERR_FORMAT;
  if (!codes || !scales || !out_bf16) return QF_ERR_NULL;
  if (fmt == QF_FMT_NVFP4 && !tensor_scale) return QF_ERR_NULL;
  if (rows < 0 || cols < 0 || cols % block_of(fmt)) return QF_ERR_SHAPE;
  if (!aligned16(codes) || !aligned16(out_bf16) || (fmt == QF_FMT_Q4_K && !aligned16(scales))) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  return cu(launch_dequant(fmt, codes, scales, tensor_scale, rows, cols, out_bf16, static_cast<cudaStream_t>(stream)));
}

qf_status_t qf_amax(const void* in, int64_t n, float* amax_out, void* stream) {
  if (!in || !amax_out) return QF_ERR_NULL;
  if (n < 0) return QF_ERR_SHAPE;
  if (!aligned16(in)) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the result word doubles as the accumulator: FP32 bits of a non-negative value
  if (cudaError_t e = cudaMemsetAsync(amax_out, 0, 4, st)) return cu(e);
  if (n == 0) return QF_OK;
  return cu(launch_amax(in, n, reinterpret_cast<uint32_t*>(amax_out), st));
}

qf_status_t qf_nvfp4_tensor_scale(const void* const* tensors, const int64_t* sizes, int n, float* amax_state, float* scale_out,
                                  uint32_t flags, void* stream) {
  if (n < 0) return QF_ERR_SHAPE;
  if (!amax_state || (n > 0 && (!tensors || !sizes))) return QF_ERR_NULL;
  for (int i = 0; i < n; ++i) {
    if (sizes[i] < 0) return QF_ERR_SHAPE;
    if (sizes[i] > 0 && !tensors[i]) return QF_ERR_NULL;
    if (!aligned16(tensors[i])) return QF_ERR_ALIGN;
  }
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the state word is the accumulator: FP32 bits of a non-negative value order like unsigned integers
  if (!(flags & QF_AMAX_RUNNING))
    if (cudaError_t e = cudaMemsetAsync(amax_state, 0, 4, st)) return cu(e);
  for (int i = 0; i < n; ++i)
    if (sizes[i] > 0)
      if (cudaError_t e = launch_amax(tensors[i], sizes[i], reinterpret_cast<uint32_t*>(amax_state), st)) return cu(e);
  if (scale_out) return cu(launch_amax_to_scale(reinterpret_cast<const uint32_t*>(amax_state), scale_out, st));
  return QF_OK;
}

qf_status_t qf_fq_linear_fwd(const void* X, const void* W, void* Y, qf_dtype_t y_dtype, int64_t M, int64_t N, int64_t K,
                             qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale, float* a_tscale, float* a_amax_out,
                             uint32_t flags, void* workspace, size_t workspace_bytes, void* stream) {
  return linear_fwd_impl(X, W, Y, y_dtype, nullptr, 1, M, N, K, wq_fmt, aq_fmt, w_tscale, a_tscale, a_amax_out, flags,
                         workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

qf_status_t qf_fq_linear_bwd(const void* dY, const void* X, const void* W, void* dX, qf_dtype_t dx_dtype, void* dW,
                             qf_dtype_t dw_dtype, int64_t M, int64_t N, int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt,
                             float* w_tscale, float* a_tscale, uint32_t flags, void* workspace, size_t workspace_bytes,
                             void* stream) {
  return linear_bwd_impl(dY, X, W, dX, dx_dtype, dW, dw_dtype, nullptr, 1, M, N, K, wq_fmt, aq_fmt, w_tscale, a_tscale,
                         flags, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

static qf_status_t check_groups(const int32_t* offs, int G, int64_t rows_padded) {
  if (!offs) return QF_ERR_NULL;
  if (G <= 0 || rows_padded < 0 || rows_padded % 128) return QF_ERR_SHAPE;
  return QF_OK;
}

qf_status_t qf_fq_grouped_linear_fwd(const void* X, const void* W, void* Y, qf_dtype_t y_dtype, const int32_t* group_offsets,
                                     int G, int64_t rows_padded, int64_t N, int64_t K, qf_format_t wq_fmt,
                                     qf_format_t aq_fmt, float* w_tscale, float* a_tscale, uint32_t flags, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  if (qf_status_t s = check_groups(group_offsets, G, rows_padded)) return s;
  return linear_fwd_impl(X, W, Y, y_dtype, group_offsets, G, rows_padded, N, K, wq_fmt, aq_fmt, w_tscale, a_tscale, nullptr,
                         flags, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

qf_status_t qf_fq_grouped_linear_bwd(const void* dY, const void* X, const void* W, void* dX, qf_dtype_t dx_dtype, void* dW,
                                     qf_dtype_t dw_dtype, const int32_t* group_offsets, int G, int64_t rows_padded, int64_t N,
                                     int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale, float* a_tscale,
                                     uint32_t flags, void* workspace, size_t workspace_bytes, void* stream) {
  if (qf_status_t s = check_groups(group_offsets, G, rows_padded)) return s;
  return linear_bwd_impl(dY, X, W, dX, dx_dtype, dW, dw_dtype, group_offsets, G, rows_padded, N, K, wq_fmt, aq_fmt, w_tscale,
                         a_tscale, flags, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

qf_status_t qf_selftest_cvt(const float* in, int64_t n, uint8_t* e2m1_out, uint8_t* e4m3_out, void* stream) {
  if (!in || (!e2m1_out && !e4m3_out)) return QF_ERR_NULL;
  if (n < 0) return QF_ERR_SHAPE;
  if (qf_status_t s = check_arch()) return s;
  return cu(launch_selftest_cvt(in, n, e2m1_out, e4m3_out, static_cast<cudaStream_t>(stream)));
}

// ---- allocation-free variant -----------------------------------------------------------------------
// Scratch for qf_fq_linear_fwd_noalloc lives in the library image itself. In host code the name of a
// __device__ array is only a handle, not an address a kernel can use: the device address is
// obtained per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) unsigned char g_noalloc_scratch[QF_NOALLOC_SCRATCH_BYTES];

static qf_status_t noalloc_scratch_ptr(void** out) {
  static void* cached[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return QF_ERR_CUDA; }
  if (dev < 0 || dev >= 64) return QF_ERR_CUDA;
  void* p = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    // once per device, with that device current; racing first calls resolve to the same address
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return QF_ERR_CUDA; }
    __atomic_store_n(&cached[dev], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return QF_OK;
}

qf_status_t qf_fq_linear_fwd_noalloc(const void* X, const void* W, void* Y, qf_dtype_t y_dtype, int64_t M, int64_t N,
                                     int64_t K, qf_format_t wq_fmt, qf_format_t aq_fmt, float* w_tscale, float* a_tscale,
                                     uint32_t flags, void* stream) {
  if (M < 0 || N < 0 || K < 0) return QF_ERR_SHAPE;
  // size check in a form that cannot overflow: each operand copy must fit on its own first
  const unsigned long long cap = QF_NOALLOC_SCRATCH_BYTES;
  const unsigned long long n = static_cast<unsigned long long>(N), k = static_cast<unsigned long long>(K),
                           m = static_cast<unsigned long long>(M);
  if ((k != 0 && (n > cap / 2 / k || m > cap / 2 / k)) || linear_ws_bytes(M, N, K, 1) > cap) return QF_ERR_TOO_LARGE;
  if (qf_status_t s = check_arch()) return s;
  void* scratch = nullptr;
  if (qf_status_t s = noalloc_scratch_ptr(&scratch)) return s;
  // the buffer is shared by every caller: copies left there by an earlier call are never trusted
  flags &= ~static_cast<uint32_t>(QF_REUSE_W_HAT | QF_REUSE_X_HAT);
  return linear_fwd_impl(X, W, Y, y_dtype, nullptr, 1, M, N, K, wq_fmt, aq_fmt, w_tscale, a_tscale, nullptr, flags, scratch,
                         QF_NOALLOC_SCRATCH_BYTES, static_cast<cudaStream_t>(stream));
}

static qf_status_t check_pack(int layout, int fmt, int64_t rows, int64_t cols) {
  if (layout == QF_LAYOUT_GGUF_Q4_K) { if (fmt != QF_FMT_Q4_K) return QF_ERR_FORMAT; }
  else if (layout == QF_LAYOUT_FP4_SWIZZLED_SCALES) { if (fmt != QF_FMT_NVFP4 && fmt != QF_FMT_MXFP4) return QF_ERR_FORMAT; }
  else return QF_ERR_FORMAT;
  if (rows < 0 || cols < 0 || cols % block_of(fmt)) return QF_ERR_SHAPE;
  return QF_OK;
}

size_t qf_pack_bytes(qf_layout_t layout, qf_format_t fmt, int64_t rows, int64_t cols) {
  if (check_pack(layout, fmt, rows, cols) != QF_OK) return 0;
  if (layout == QF_LAYOUT_GGUF_Q4_K) return static_cast<size_t>(rows) * (cols / 256) * 144;
  const int64_t nblk = cols / block_of(fmt);
  return static_cast<size_t>((rows + 127) / 128) * ((nblk + 3) / 4) * 512;
}

qf_status_t qf_pack(qf_layout_t layout, qf_format_t fmt, const void* codes, const void* scales, int64_t rows, int64_t cols,
                    void* packed, void* stream) {
  if (qf_status_t s = check_pack(layout, fmt, rows, cols)) return s;
  const bool empty = rows == 0 || cols == 0;
  if (!empty && (!scales || !packed || (layout == QF_LAYOUT_GGUF_Q4_K && !codes))) return QF_ERR_NULL;
  if (!aligned16(scales) || !aligned16(packed) || (layout == QF_LAYOUT_GGUF_Q4_K && !aligned16(codes))) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (layout == QF_LAYOUT_GGUF_Q4_K) return cu(launch_pack_q4k(codes, scales, rows * (cols / 256), packed, false, nullptr, nullptr, st));
  return cu(launch_swizzle_scales(scales, rows, cols / block_of(fmt), packed, false, st));
}

qf_status_t qf_unpack(qf_layout_t layout, qf_format_t fmt, const void* packed, int64_t rows, int64_t cols, void* codes,
                      void* scales, void* stream) {
  if (qf_status_t s = check_pack(layout, fmt, rows, cols)) return s;
  const bool empty = rows == 0 || cols == 0;
  if (!empty && (!scales || !packed || (layout == QF_LAYOUT_GGUF_Q4_K && !codes))) return QF_ERR_NULL;
  if (!aligned16(scales) || !aligned16(packed) || (layout == QF_LAYOUT_GGUF_Q4_K && !aligned16(codes))) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (layout == QF_LAYOUT_GGUF_Q4_K) return cu(launch_pack_q4k(nullptr, nullptr, rows * (cols / 256), const_cast<void*>(packed), true, codes, scales, st));
  return cu(launch_swizzle_scales(packed, rows, cols / block_of(fmt), scales, true, st));
}

qf_status_t qf_fp4_matmul_native(qf_format_t fmt, const void* a_codes, const void* a_scales, const float* a_tscale,
                                 const void* b_codes, const void* b_scales, const float* b_tscale, int64_t M, int64_t N,
                                 int64_t K, float* Y, uint32_t flags, void* workspace, size_t workspace_bytes, void* stream) {
  if (fmt != QF_FMT_MXFP4 && fmt != QF_FMT_NVFP4) return QF_ERR_FORMAT;
  if (M < 0 || N < 0 || K < 0 || K % 32) return QF_ERR_SHAPE;
  if (M > INT32_MAX - 128 || N > INT32_MAX - 128) return QF_ERR_SHAPE;             // tile coordinates are 32-bit
  if (!workspace || workspace_bytes < kWsHeader) return QF_ERR_WORKSPACE;
  if (M == 0 || N == 0) return QF_OK;
  if (!Y) return QF_ERR_NULL;
  if (K > 0 && (!a_codes || !a_scales || !b_codes || !b_scales)) return QF_ERR_NULL;
  if (fmt == QF_FMT_NVFP4 && K > 0 && (!a_tscale || !b_tscale)) return QF_ERR_NULL;
  if (!aligned16(a_codes) || !aligned16(b_codes) || !aligned16(Y) || !aligned16(workspace)) return QF_ERR_ALIGN;
  if ((flags & QF_SCALES_TILED) && (!aligned16(a_scales) || !aligned16(b_scales))) return QF_ERR_ALIGN;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* header = static_cast<uint32_t*>(workspace);
  if (cudaError_t e = cudaMemsetAsync(header, 0, kWsHeader, st)) return cu(e);
  Fp4GemmArgs g{};
  g.scales_tiled = (flags & QF_SCALES_TILED) != 0;
  g.fmt = fmt;
  g.a_codes = a_codes; g.a_scales = a_scales; g.a_tscale = a_tscale;
  g.b_codes = b_codes; g.b_scales = b_scales; g.b_tscale = b_tscale;
  g.Y = Y;
  g.M = M; g.N = N; g.K = K;
  g.status_word = header + kWsStatus;
  return cu(launch_fp4_native(g, st));
}

qf_status_t qf_selftest_timeout(void* workspace, size_t workspace_bytes, int64_t limit_cycles, void* stream) {
  if (!workspace) return QF_ERR_WORKSPACE;
  if (workspace_bytes < kWsHeader) return QF_ERR_WORKSPACE;
  if (limit_cycles < 1 || limit_cycles > (1ll << 28)) return QF_ERR_SHAPE;      // a fraction of a second at most
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* header = static_cast<uint32_t*>(workspace);
  if (cudaError_t e = cudaMemsetAsync(header, 0, kWsHeader, st)) return cu(e);
  return cu(launch_selftest_timeout(header + kWsStatus, limit_cycles, reinterpret_cast<int*>(header + 16), st));
}

qf_status_t qf_selftest_mxfp4_bf16(uint64_t* mismatches, void* stream) {
  if (!mismatches) return QF_ERR_NULL;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaError_t e = cudaMemsetAsync(mismatches, 0, 8, st)) return cu(e);
  return cu(launch_selftest_mxfp4_bf16(reinterpret_cast<unsigned long long*>(mismatches), st));
}

qf_status_t qf_selftest_div(const float* xs, int64_t nx, const float* ys, int64_t ny, uint64_t* mismatches, void* stream) {
  if (!xs || !ys || !mismatches) return QF_ERR_NULL;
  if (nx < 0 || ny < 0) return QF_ERR_SHAPE;
  if (qf_status_t s = check_arch()) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaError_t e = cudaMemsetAsync(mismatches, 0, 8, st)) return cu(e);
  return cu(launch_selftest_div(xs, nx, ys, ny, reinterpret_cast<unsigned long long*>(mismatches), st));
}

}  // extern "C"
