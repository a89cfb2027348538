// BF16 x BF16 -> FP32 matmul on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory), operands staged by TMA into 128-byte-swizzled shared memory. Two persistent kernels share
// one pipeline design (a TMA ring feeding a single MMA-issuing thread; the 512 TMEM columns hold two
// accumulators, so the epilogue of one tile overlaps the main loop of the next):
//   gemm_pair_kernel  the main one: a cluster of two CTAs per 256 x 256 output tile, cta_group::2 MMAs, 6 stages,
//                     optional in-kernel MXFP4 quantization of the staged tiles;
//   gemm_kernel       one CTA per 128 x 256 tile, 4 stages: outputs with fewer than 256 rows, and grouped layers
//                     with more experts than the pair kernel's shared-memory tile table holds.
//
// The three products of the quantization-aware layer (Eq. fakequant, Eq. ste, Eq. activation-ste)
// differ only in which operand dimension is contiguous in memory:
//   forward  Y  = X_hat . W_hat^T : both operands contraction-major ("K-major")
//   dgrad    dX = dY . W_hat      : A contraction-major, B row-major over the contraction ("MN-major")
//   wgrad    dW = dY^T . X_hat    : both MN-major
// so one kernel, templated on the two majors, serves all of them; the shared-memory descriptor and
// the TMA box shape change, the pipeline does not.
//
// Every wait on an mbarrier is bounded. A wait that gives up raises a CTA-wide abort flag and
// records QF_ERR_TIMEOUT in the caller's status word; all roles then fall through to the common
// teardown (the producer first gives its outstanding copies a bounded chance to land), tensor
// memory is released and the kernel returns.
#include <cuda.h>

#include "qf_common.cuh"
#include "qf_ptx.cuh"
#include "qf_qdq_body.cuh"

namespace qf {
namespace {

constexpr int BM = 128;                 // output rows per tile   (UMMA M)
constexpr int BN = 256;                 // output cols per tile   (UMMA N)
constexpr int BK = 64;                  // contraction per stage  (one 128-byte swizzle row of BF16)
constexpr int UMMA_K = 16;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;    // 16 KB
constexpr int B_BYTES = BN * BK * 2;    // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int ACC_COLS = BN;            // FP32 accumulator columns per tile
constexpr int TMEM_COLS = 2 * ACC_COLS; // 512: two accumulators
constexpr int NUM_THREADS = 192;        // warp 0 TMA, warp 1 MMA + TMEM owner, warps 2-5 epilogue
constexpr int EPI_THREADS = 128;

struct alignas(8) Barriers {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

constexpr int STAGING_BYTES = 4 * 2 * 4096;    // epilogue: per warp two 32-row x 128-byte staging buffers for TMA stores
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /* alignment slack */ + 256 /* Barriers */;

struct KParams {
  void* C;
  int64_t Mo, No, Kc, ldc;
  int c_dtype, accumulate;
  int tiles_m, tiles_n, num_tiles;
  int band;                  // tiles per rasterization band along the banded dimension (see choose_raster())
  int raster;                // 0: bands of row tiles, rows fastest inside a band (the band's A panels stay in L2, B streams);
                             // 1: bands of column tiles, columns fastest (the band's B panels stay, A streams)
  int group_mode, G;
  const int32_t* offs;
  int64_t b_group_rows;      // mode 1: rows one group occupies in B's 2-D tensor map
  int64_t c_group_stride;    // mode 2: elements between per-group outputs
  uint32_t* status;
  uint32_t* tile_sync;       // plain problems: global arrival counter that keeps the CTA pairs' tile starts together (nullable)
  long long tile_sync_limit; // SM clocks a pair waits for the others at a tile start before it goes on alone
  int mxfp4_noclip;          // scale rule of the in-kernel MXFP4 quantizer
  int fuse_a_fmt, fuse_b_fmt;        // format of the in-kernel quantizer per operand (QF_FMT_MXFP4 / QF_FMT_NVFP4)
  const float* a_tscale;             // NVFP4 in-kernel quantizer: tensor scale of A
  const float* b_tscale;             // ... of B: one value, or one per group (grouped mode 1)
  int b_tscale_per_group;
  struct Side {                      // side jobs of the SIDE variant (see GemmArgs::Side)
    const uint4* in;
    uint4* out;
    int64_t nunits;                  // 16-element units
    const float* tscale;
    int fmt, noclip;
  } side[2];
};

// ---- descriptors ------------------------------------------------------------------------------

// Shared-memory matrix descriptor, 128-byte swizzle. Offsets are in 16-byte units.
//   contraction-major tile: rows of 128 bytes, 8-row groups 1024 bytes apart (stride offset);
//     the leading offset is not used by the hardware for this layout.
//   MN-major tile: TMA boxes of 64 (MN) x 64 (contraction) elements = 8 KB each; inside a box the
//     8-row contraction groups are 1024 bytes apart (stride offset) and successive 64-element MN
//     groups are one box = 8192 bytes apart (leading offset).
template <bool MN_MAJOR>
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  const uint64_t lbo = MN_MAJOR ? (8192u >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}
// 16-byte units to advance the start address by for the next 16 contraction elements
template <bool MN_MAJOR>
__device__ __forceinline__ uint32_t desc_k_step() { return MN_MAJOR ? (UMMA_K * 128u) >> 4 : (UMMA_K * 2u) >> 4; }

template <bool A_MN, bool B_MN>
__device__ __forceinline__ uint32_t instr_desc() {
  return (1u << 4)                      // D = FP32
         | (1u << 7) | (1u << 10)       // A, B = BF16
         | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16)
         | (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
}

// ---- tile bookkeeping ---------------------------------------------------------------------------

// Segment start i of a grouped call. The table lives in device memory, so the host cannot check it: whatever it holds is
// forced into the form the interface requires (a multiple of 128 inside [0, rows]), so that a bad table can give
// wrong numbers but never a negative store coordinate or a contraction loop of unbounded length.
__device__ __forceinline__ int group_off(const KParams& p, int i) {
  const int bound = static_cast<int>(p.group_mode == 2 ? p.Kc : p.Mo);
  return min(max(__ldg(p.offs + i), 0), bound) & ~127;
}

struct Tile {
  int m0, n0;          // output coordinates (rows of A, rows of B)
  int k_begin, k_end;  // contraction range
  int b_row_off;       // mode 1: row offset of this tile's group in B's tensor map
  int64_t c_off;       // mode 2: element offset of this tile's group in C
  int m_limit;         // rows of C that exist for this tile's matrix
  int group;           // mode 2: which per-group output matrix
};

__device__ __forceinline__ Tile decode_tile(const KParams& p, int t, bool need_group) {
  Tile r;
  r.b_row_off = 0;
  r.c_off = 0;
  r.k_begin = 0;
  r.k_end = static_cast<int>(p.Kc);
  r.m_limit = static_cast<int>(p.Mo);
  r.group = 0;
  int g = 0;
  if (p.group_mode == 2) {
    const int per = p.tiles_m * p.tiles_n;
    g = t / per;
    t -= g * per;
  }
  // m fastest inside bands of p.band row-tiles: concurrently running CTAs share A and B tiles in L2
  const int band = p.band * p.tiles_n;
  const int bidx = t / band;
  const int first_m = bidx * p.band;
  const int rows_in_band = min(p.band, p.tiles_m - first_m);
  const int within = t - bidx * band;
  r.m0 = (first_m + within % rows_in_band) * BM;
  r.n0 = (within / rows_in_band) * BN;
  if (p.group_mode == 1 && need_group) {
    // segments start on multiples of BM, so a row tile lies in exactly one group: find it
    int lo = 0, hi = p.G;                   // invariant: offs[lo] <= m0 < offs[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(p.offs + mid) <= r.m0) lo = mid; else hi = mid;
    }
    r.b_row_off = lo * static_cast<int>(p.b_group_rows);
  } else if (p.group_mode == 2) {
    r.k_begin = group_off(p, g);
    r.k_end = group_off(p, g + 1);
    r.c_off = static_cast<int64_t>(g) * p.c_group_stride;
    r.group = g;
  }
  return r;
}

// ---- epilogue stores ------------------------------------------------------------------------------

template <typename OutT>
__device__ __forceinline__ void store_chunk32(OutT* row_ptr, int col0, int n_limit, const uint32_t (&acc)[32], bool accumulate);

template <>
__device__ __forceinline__ void store_chunk32<__nv_bfloat16>(__nv_bfloat16* row_ptr, int col0, int n_limit,
                                                             const uint32_t (&acc)[32], bool accumulate) {
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int col = col0 + 8 * g;
    if (col + 8 <= n_limit) {
      uint4* dst = reinterpret_cast<uint4*>(row_ptr + col);
      float v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(acc[8 * g + j]);
      if (accumulate) {
        const uint4 old = *dst;
        const uint32_t w[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[2 * j] += bf16_lo(w[j]);
          v[2 * j + 1] += bf16_hi(w[j]);
        }
      }
      *dst = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
    }
  }
}

template <>
__device__ __forceinline__ void store_chunk32<float>(float* row_ptr, int col0, int n_limit, const uint32_t (&acc)[32],
                                                     bool accumulate) {
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    const int col = col0 + 4 * g;
    if (col + 4 <= n_limit) {
      float4* dst = reinterpret_cast<float4*>(row_ptr + col);
      float4 v = make_float4(__uint_as_float(acc[4 * g]), __uint_as_float(acc[4 * g + 1]), __uint_as_float(acc[4 * g + 2]),
                             __uint_as_float(acc[4 * g + 3]));
      if (accumulate) {
        const float4 old = *dst;
        v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
      }
      *dst = v;
    }
  }
}

// ---- epilogue through shared memory and TMA stores ------------------------------------------------------
// Each epilogue warp owns 32 accumulator rows (its quarter of the TMEM lanes). Per column chunk of
// 128 bytes of output (64 BF16 or 32 FP32 values) a lane reads its row from TMEM, converts it, and writes
// it into a 32 x 128-byte staging buffer with the 128-byte swizzle (16-byte chunk j of row r goes to
// chunk j ^ (r & 7): conflict-free), then one lane issues a TMA store (or a TMA add-reduce when
// accumulating in FP32) of the 32-row box. The tensor map clips rows and columns past the matrix edge.
// Two staging buffers per warp let the next chunk be converted while the previous store drains.

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y), "r"(z)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <typename OutT>
struct EpiChunk {
  static constexpr int COLS = 128 / static_cast<int>(sizeof(OutT));   // output columns per 128-byte staging row
  static constexpr int NCHUNK = BN / COLS;
};

// One tile's worth of TMA-store epilogue for one warp. `release` is called once, right after the last
// TMEM read, so the accumulator can be handed back before the remaining stores are issued.
template <typename OutT, typename Release>
__device__ __forceinline__ void epilogue_tile_tma(const CUtensorMap* tmC, uint32_t warp_staging, uint32_t& which, uint32_t taddr,
                                                  int row0, int n0, int z, int rows_limit, int n_limit, bool accumulate,
                                                  bool empty_k, int lane, Release release) {
  constexpr int COLS = EpiChunk<OutT>::COLS;
  constexpr int NCHUNK = EpiChunk<OutT>::NCHUNK;
#pragma unroll 1
  for (int c = 0; c < NCHUNK; ++c) {
    uint32_t acc[COLS];
#pragma unroll
    for (int h = 0; h < COLS / 32; ++h) tmem_ld32(taddr + c * COLS + h * 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[32 * h]));
    tmem_ld_wait();
    if (c == NCHUNK - 1) release();
    if (empty_k) {
#pragma unroll
      for (int j = 0; j < COLS; ++j) acc[j] = 0u;
    }
    // the buffer about to be overwritten was the source of the store issued two chunks ago
    if (lane == 0) bulk_wait_read_1();
    __syncwarp();
    const uint32_t buf = warp_staging + which * 4096u;
    const uint32_t row_addr = buf + static_cast<uint32_t>(lane) * 128u;
    const uint32_t sw = static_cast<uint32_t>(lane & 7);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      uint32_t v0, v1, v2, v3;
      if constexpr (sizeof(OutT) == 2) {
        v0 = pack_bf16x2(__uint_as_float(acc[8 * j]), __uint_as_float(acc[8 * j + 1]));
        v1 = pack_bf16x2(__uint_as_float(acc[8 * j + 2]), __uint_as_float(acc[8 * j + 3]));
        v2 = pack_bf16x2(__uint_as_float(acc[8 * j + 4]), __uint_as_float(acc[8 * j + 5]));
        v3 = pack_bf16x2(__uint_as_float(acc[8 * j + 6]), __uint_as_float(acc[8 * j + 7]));
      } else {
        v0 = acc[4 * j]; v1 = acc[4 * j + 1]; v2 = acc[4 * j + 2]; v3 = acc[4 * j + 3];
      }
      st_shared_v4(row_addr + ((static_cast<uint32_t>(j) ^ sw) << 4), v0, v1, v2, v3);
    }
    fence_async_smem();
    __syncwarp();
    const int col0 = n0 + c * COLS;
    if (lane == 0) {
      if (row0 < rows_limit && col0 < n_limit) {
        if (accumulate) tma_reduce_add_3d(tmC, buf, col0, row0, z);
        else tma_store_3d(tmC, buf, col0, row0, z);
      }
      bulk_commit();
    }
    which ^= 1u;
  }
}

// ---- the kernel -----------------------------------------------------------------------------------

template <bool A_MN, bool B_MN, typename OutT>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, const KParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;                   // swizzled tiles need 1024-byte alignment
  uint8_t* tiles_ptr = smem_raw + (tiles_base - raw);
  const uint32_t staging_base = tiles_base + STAGES * STAGE_BYTES;
  Barriers* bars = reinterpret_cast<Barriers*>(tiles_ptr + STAGES * STAGE_BYTES + STAGING_BYTES);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  KernelClock kclock;
  const bool clocked = blockIdx.x == 0 && threadIdx.x == 0;
  if (clocked) kclock.start();

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);
      mbar_init(smem_u32(&bars->acc_empty[b]), EPI_THREADS);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&bars->tmem_base), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ===== TMA producer =====
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool alive = true;
      for (int t = blockIdx.x; t < p.num_tiles && alive; t += gridDim.x) {
        const Tile tile = decode_tile(p, t, true);
        for (int k = tile.k_begin; k < tile.k_end; k += BK) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, p.status)) { alive = false; break; }
          const uint32_t full = smem_u32(&bars->full[stage]);
          const uint32_t a_dst = tiles_base + stage * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          mbar_expect_tx(full, STAGE_BYTES);
          if (A_MN) {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d(a_dst + i * 8192, &tmA, tile.m0 + 64 * i, k, full);
          } else {
            tma_load_2d(a_dst, &tmA, k, tile.m0, full);
          }
          if (B_MN) {
#pragma unroll
            for (int i = 0; i < BN / 64; ++i) tma_load_2d(b_dst + i * 8192, &tmB, tile.n0 + 64 * i, tile.b_row_off + k, full);
          } else {
            tma_load_2d(b_dst, &tmB, k, tile.b_row_off + tile.n0, full);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!alive) {
        // give copies already in flight a bounded chance to land before the CTA retires
        uint32_t s = stage, ph = phase;
        for (uint32_t n = 0; n < min(issued, static_cast<uint32_t>(STAGES)); ++n) {
          if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (mbar_try_wait(smem_u32(&bars->full[s]), ph)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer =====
    if (lane == 0) {
      const uint32_t idesc = instr_desc<A_MN, B_MN>();
      uint32_t stage = 0, phase = 0;
      uint32_t local = 0;
      bool alive = true;
      for (int t = blockIdx.x; t < p.num_tiles && alive; t += gridDim.x, ++local) {
        const Tile tile = decode_tile(p, t, false);
        const uint32_t buf = local & 1u;
        const uint32_t use = local >> 1;                      // how many times this accumulator was used before
        if (!mbar_wait(smem_u32(&bars->acc_empty[buf]), (use & 1u) ^ 1u, abort_flag, p.status)) { alive = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * ACC_COLS;
        uint32_t accumulate = 0;
        for (int k = tile.k_begin; k < tile.k_end; k += BK) {
          if (!mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, p.status)) { alive = false; break; }
          tc_fence_after();
          const uint32_t a_addr = tiles_base + stage * STAGE_BYTES;
          const uint64_t a_desc = smem_desc<A_MN>(a_addr);
          const uint64_t b_desc = smem_desc<B_MN>(a_addr + A_BYTES);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            umma_bf16(d_tmem, a_desc + kk * desc_k_step<A_MN>(), b_desc + kk * desc_k_step<B_MN>(), idesc, accumulate);
            accumulate = 1;
          }
          umma_commit(smem_u32(&bars->empty[stage]));           // frees the stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        if (tile.k_end <= tile.k_begin) {
          // empty contraction (an expert with no rows): nothing was accumulated; the epilogue writes zeros
        }
        umma_commit(smem_u32(&bars->acc_full[buf]));
      }
    }
  } else {
    // ===== epilogue: TMEM -> registers -> global =====
    const int quarter = warp & 3;                               // TMEM lanes 32*quarter .. +31 belong to this warp
    uint32_t local = 0, which = 0;
    bool alive = true;
    const bool use_tma = !(p.accumulate != 0 && sizeof(OutT) == 2);
    for (int t = blockIdx.x; t < p.num_tiles && alive; t += gridDim.x, ++local) {
      const Tile tile = decode_tile(p, t, false);
      const uint32_t buf = local & 1u;
      const uint32_t use = local >> 1;
      const bool got = mbar_wait(smem_u32(&bars->acc_full[buf]), use & 1u, abort_flag, p.status);
      if (!__all_sync(0xFFFFFFFFu, got)) { alive = false; break; }        // keep the warp converged for tcgen05.ld
      tc_fence_after();
      const uint32_t taddr = tmem_base + buf * ACC_COLS + (static_cast<uint32_t>(quarter * 32) << 16);
      const bool empty_k = tile.k_end <= tile.k_begin;
      if (use_tma) {
        epilogue_tile_tma<OutT>(&tmC, staging_base + static_cast<uint32_t>(warp - 2) * 8192u, which, taddr,
                                tile.m0 + quarter * 32, tile.n0, tile.group, tile.m_limit, static_cast<int>(p.No),
                                p.accumulate != 0, empty_k, lane, [&]() {
                                  tc_fence_before();
                                  mbar_arrive(smem_u32(&bars->acc_empty[buf]));
                                });
      } else {
        // BF16 output with accumulation: add in FP32 and round once (a TMA add-reduce would round twice)
        const int row = tile.m0 + quarter * 32 + lane;
        const bool row_ok = row < tile.m_limit;
        OutT* row_ptr = static_cast<OutT*>(p.C) + tile.c_off + static_cast<int64_t>(row) * p.ldc;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          if (c == BN / 32 - 1) {
            tc_fence_before();
            mbar_arrive(smem_u32(&bars->acc_empty[buf]));
          }
          if (empty_k) {
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[j] = 0u;
          }
          const int col0 = tile.n0 + c * 32;
          if (row_ok && col0 < p.No) store_chunk32<OutT>(row_ptr, col0, static_cast<int>(p.No), acc, true);
        }
      }
    }
    if (lane == 0) bulk_wait_all();          // every TMA store of this warp has completed before the CTA retires
  }

  // ===== teardown =====
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (clocked) kclock.stop(p.status);
}

// =====================================================================================================
// Two-CTA variant (cta_group::2): a cluster of two CTAs on neighbouring SMs computes a 256 x 256 output
// tile with one M=256 MMA stream issued by the leader CTA. Each CTA stages only its own 128 rows of A
// and its own 128 rows (half) of B, so the shared-memory operand traffic per SM is 64 B/clk instead of
// the 96 B/clk of the one-CTA tile, and each holds its 128 accumulator rows in its own tensor memory.
//   * both producers' TMA copies complete on the LEADER's full barrier (each CTA fetches its own tiles);
//   * the leader frees a stage / publishes an accumulator with a tcgen05.commit multicast to the same
//     barrier offset in both CTAs;
//   * both CTAs' epilogue warps release the accumulator on the leader's barrier (remote arrive).
// Plain (non-grouped) problems only.
// =====================================================================================================

constexpr int STAGES2 = 6;
constexpr int MAX_PAIR_GROUPS = 256;     // experts the two-CTA kernel's shared-memory tile table holds
constexpr int A2_BYTES = BM * BK * 2;           // 16 KB: this CTA's 128 rows of A
constexpr int B2_BYTES = (BN / 2) * BK * 2;     // 16 KB: this CTA's 128 rows of B
constexpr int STAGE2_BYTES = A2_BYTES + B2_BYTES;
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + STAGING_BYTES + 1024 + 256 + 4 * (MAX_PAIR_GROUPS + 4);

constexpr int TRANSFORM_WARPS = 16;                      // fused variant: warps that quantize-dequantize staged tiles
constexpr int TRANSFORM_GROUPS = 4;                      // group g takes k-blocks g, g + 4, ... (must not exceed STAGES2)
constexpr int WARPS_PER_GROUP = TRANSFORM_WARPS / TRANSFORM_GROUPS;
constexpr int NUM_THREADS_FUSED = NUM_THREADS + 32 * TRANSFORM_WARPS;
constexpr int SIDE_WARPS = 8;                           // SIDE variant: warps that run the side jobs
constexpr int NUM_THREADS_SIDE = NUM_THREADS + 32 * SIDE_WARPS;
static_assert(TRANSFORM_GROUPS <= 6, "more groups than pipeline stages would let a group wait on a stage two uses ahead");

struct alignas(8) Barriers2 {
  uint64_t ready[STAGES2];      // fused variant, leader's copy: both CTAs' tiles have been quantized in place
  uint64_t full[STAGES2];       // leader's copy is the live one (fused variant: each CTA's own copy)
  uint64_t empty[STAGES2];      // one per CTA, released by the leader's commit multicast
  uint64_t acc_full[2];         // one per CTA, published by the leader's commit multicast
  uint64_t acc_empty[2];        // leader's copy is the live one: 8 arrivals (4 epilogue warps x 2 CTAs)
  uint32_t tmem_base;
  int abort_flag;
  int cum[MAX_PAIR_GROUPS + 1];  // grouped mode 1: pair row-tiles before each expert (prefix sum)
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA copy into this CTA's shared memory whose completion is counted on a barrier that may live in the
// other CTA of the pair (cluster address). Each CTA fetches its own tiles; nothing is broadcast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_gpu_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this offset in both CTAs of the pair once all MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}

template <bool A_MN, bool B_MN>
__device__ __forceinline__ uint32_t instr_desc_pair() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
         (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>((2 * BM) >> 4) << 24);
}

struct PairTile {
  int m0, n0;            // first output row / column of the 256 x 256 pair tile
  int k_begin, k_end;    // contraction range
  int b_row_off;         // mode 1: row offset of this tile's expert in B's 2-D tensor map
  int z;                 // mode 2: which per-expert output matrix
  int rows_limit;        // output rows at or beyond this index do not belong to this tile's matrix / segment
  int group;             // mode 1: the expert whose weights this tile multiplies by (0 otherwise)
};

// Pair tiles are walked row-tile fastest inside bands (see band_rows()). Grouped mode 1: the row-tile
// index counts 256-row tiles expert by expert (cum[] = tiles before each expert, built at kernel start);
// a segment with an odd number of 128-row blocks ends in a tile whose second half lies in the next
// expert's rows: that half is computed and thrown away (rows_limit = end of the segment).
__device__ __forceinline__ PairTile decode_pair(const KParams& p, const int* cum, int tiles_m, int t) {
  PairTile r;
  r.k_begin = 0;
  r.k_end = static_cast<int>(p.Kc);
  r.b_row_off = 0;
  r.z = 0;
  r.group = 0;
  r.rows_limit = static_cast<int>(p.Mo);
  int g = 0;
  if (p.group_mode == 2) {
    const int per = tiles_m * p.tiles_n;
    g = t / per;
    t -= g * per;
  }
  int mt;
  if (p.raster == 0) {
    const int band = p.band * p.tiles_n;
    const int bidx = t / band;
    const int first_m = bidx * p.band;
    const int rows_in_band = min(p.band, tiles_m - first_m);
    const int within = t - bidx * band;
    mt = first_m + within % rows_in_band;
    r.n0 = (within / rows_in_band) * BN;
  } else {
    const int band = p.band * tiles_m;
    const int bidx = t / band;
    const int first_n = bidx * p.band;
    const int cols_in_band = min(p.band, p.tiles_n - first_n);
    const int within = t - bidx * band;
    mt = within / cols_in_band;
    r.n0 = (first_n + within % cols_in_band) * BN;
  }
  r.m0 = mt * (2 * BM);
  if (p.group_mode == 1) {
    int lo = 0, hi = p.G;                     // invariant: cum[lo] <= mt < cum[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cum[mid] <= mt) lo = mid; else hi = mid;
    }
    r.m0 = group_off(p, lo) + (mt - cum[lo]) * (2 * BM);
    r.rows_limit = group_off(p, lo + 1);
    r.b_row_off = lo * static_cast<int>(p.b_group_rows);
    r.group = lo;
  } else if (p.group_mode == 2) {
    r.k_begin = group_off(p, g);
    r.k_end = group_off(p, g + 1);
    r.z = g;
  }
  return r;
}

// In-place MXFP4 quantize-dequantize of `nchunks` 16-byte chunks of a staged operand tile by the 256
// transform threads. A tile is a stack of 128-byte rows holding 64 consecutive elements of the
// tensor's last (block) dimension, whatever the operand's majorness, so a 32-element block is an aligned
// group of four chunks; the 128-byte swizzle permutes chunks only inside aligned groups of eight by
// an XOR, which maps aligned groups of four onto aligned groups of four. Lane l takes chunk l of each
// 512-byte span (bank-conflict free); the four lanes of a block combine their maxima by shuffles.
// One batch: PER chunks per lane, loads first, then shuffles, then independent arithmetic chains, then stores.
template <int PER>
__device__ __forceinline__ void mxfp4_transform_batch(uint32_t slab, bool noclip) {
  uint4 v[PER];
  uint32_t m[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) v[i] = ld_shared_v4(slab + static_cast<uint32_t>(i) * 512u);
#pragma unroll
  for (int i = 0; i < PER; ++i) m[i] = chunk8_amax_bits(v[i].x, v[i].y, v[i].z, v[i].w);
#pragma unroll
  for (int i = 0; i < PER; ++i) m[i] = max(m[i], __shfl_xor_sync(0xFFFFFFFFu, m[i], 1));
#pragma unroll
  for (int i = 0; i < PER; ++i) m[i] = max(m[i], __shfl_xor_sync(0xFFFFFFFFu, m[i], 2));
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const uint32_t code = mxfp4_scale_code(m[i], noclip);
    const uint32_t dst = slab + static_cast<uint32_t>(i) * 512u;
    if (mxfp4_bf16_path_ok(code)) {
      // conversion-free rounding in packed BF16 arithmetic (the common case)
      const uint32_t one2 = mxfp4_one2(code), six2 = mxfp4_six2(code);
      st_shared_v4(dst, mxfp4_qdq_pair_bf16(v[i].x, one2, six2), mxfp4_qdq_pair_bf16(v[i].y, one2, six2),
                   mxfp4_qdq_pair_bf16(v[i].z, one2, six2), mxfp4_qdq_pair_bf16(v[i].w, one2, six2));
    } else {
      // all-zero blocks (tile padding) and blocks at the very ends of the BF16 exponent range
      const float2 inv = splat(e8m0_inv_scale(code)), sc = splat(e8m0_scale(code));
      const uint32_t keep = m[i] == 0 ? 0u : 0xFFu;
      st_shared_v4(dst, mxfp4_qdq_pair(v[i].x, inv, sc, keep), mxfp4_qdq_pair(v[i].y, inv, sc, keep),
                   mxfp4_qdq_pair(v[i].z, inv, sc, keep), mxfp4_qdq_pair(v[i].w, inv, sc, keep));
    }
  }
}

// A staged tile of NCHUNKS 16-byte chunks, split between the WARPS_PER_GROUP warps of one transform group:
// each warp owns a contiguous slab and walks it in batches of four chunks per lane (512 bytes per warp
// per load instruction: bank-conflict free, and every aligned group of four lanes holds one 32-element block).
template <int NCHUNKS>
__device__ __forceinline__ void mxfp4_transform_tile(uint32_t base, int warp_in_group, int lane, bool noclip) {
  constexpr int PER_WARP = NCHUNKS / WARPS_PER_GROUP;          // chunks per warp
  constexpr int BATCH = 4;
  static_assert(PER_WARP % (32 * BATCH) == 0, "tile must split evenly");
  const uint32_t slab = base + static_cast<uint32_t>(warp_in_group * PER_WARP + lane) * 16u;
#pragma unroll 1
  for (int b = 0; b < PER_WARP / (32 * BATCH); ++b) mxfp4_transform_batch<BATCH>(slab + static_cast<uint32_t>(b) * (32u * BATCH * 16u), noclip);
}

// The same for NVFP4 (Eq. nvfp4 with the tensor scale already final): a 16-element block is an aligned PAIR of 16-byte
// chunks, which the swizzle also maps onto an aligned pair, so lanes l and l ^ 1 hold one block and combine their maxima
// with one shuffle. Arithmetic identical to the stand-alone quantizer (nvfp4_block_words): same bits.
template <int PER>
__device__ __forceinline__ void nvfp4_transform_batch(uint32_t slab, const Nvfp4Tensor nt) {
  uint4 v[PER];
  uint32_t m[PER];
#pragma unroll
  for (int i = 0; i < PER; ++i) v[i] = ld_shared_v4(slab + static_cast<uint32_t>(i) * 512u);
#pragma unroll
  for (int i = 0; i < PER; ++i) m[i] = chunk8_amax_bits(v[i].x, v[i].y, v[i].z, v[i].w);
#pragma unroll
  for (int i = 0; i < PER; ++i) m[i] = max(m[i], __shfl_xor_sync(0xFFFFFFFFu, m[i], 1));
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
    uint32_t o[4], codes[4], scale_code;
    nvfp4_block_words<4>(w, __uint_as_float(m[i] << 16), nt, o, codes, scale_code);
    st_shared_v4(slab + static_cast<uint32_t>(i) * 512u, o[0], o[1], o[2], o[3]);
  }
}

template <int NCHUNKS>
__device__ __forceinline__ void nvfp4_transform_tile(uint32_t base, int warp_in_group, int lane, const Nvfp4Tensor nt) {
  constexpr int PER_WARP = NCHUNKS / WARPS_PER_GROUP;
  constexpr int BATCH = 2;
  static_assert(PER_WARP % (32 * BATCH) == 0, "tile must split evenly");
  const uint32_t slab = base + static_cast<uint32_t>(warp_in_group * PER_WARP + lane) * 16u;
#pragma unroll 1
  for (int b = 0; b < PER_WARP / (32 * BATCH); ++b) nvfp4_transform_batch<BATCH>(slab + static_cast<uint32_t>(b) * (32u * BATCH * 16u), nt);
}

// FUSE: bit 0 = quantize-dequantize the staged A tile, bit 1 = the staged B tile (format per operand at run time:
// MXFP4 or NVFP4). With FUSE != 0
// TRANSFORM_WARPS extra warps (sixteen, in four groups that take alternate k-blocks) transform each stage in
// shared memory between the TMA arrival and the MMA issue, so the fake-quantized operand never exists in
// global memory.
// SIDE: eight more warps run up to two flat FP4 quantize-dequantize passes over other tensors (the operand of the next
// product) from global to global memory while the tensor cores work: an HBM-bound pass hidden under a tensor-bound one.
template <bool A_MN, bool B_MN, typename OutT, int FUSE, bool SIDE = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FUSE ? NUM_THREADS_FUSED : (SIDE ? NUM_THREADS_SIDE : NUM_THREADS), 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmC, const KParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles_base - raw);
  const uint32_t staging_base = tiles_base + STAGES2 * STAGE2_BYTES;
  Barriers2* bars = reinterpret_cast<Barriers2*>(tiles_ptr + STAGES2 * STAGE2_BYTES + STAGING_BYTES);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  KernelClock kclock;
  const bool clocked = blockIdx.x == 0 && threadIdx.x == 0;
  if (clocked) kclock.start();

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(smem_u32(&bars->ready[s]), 2 * WARPS_PER_GROUP);
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->acc_full[b]), 1);
      mbar_init(smem_u32(&bars->acc_empty[b]), 8);
    }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(&bars->tmem_base), TMEM_COLS);
  if (warp == 2 && p.group_mode == 1) {
    // prefix sum of pair row-tiles per expert (G <= MAX_PAIR_GROUPS): lane l takes experts 8l .. 8l+7
    int cnt[8], sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int g = lane * 8 + j;
      cnt[j] = g < p.G ? max(group_off(p, g + 1) - group_off(p, g) + 2 * BM - 1, 0) / (2 * BM) : 0;
      sum += cnt[j];
    }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += up;
    }
    int run = incl - sum;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int g = lane * 8 + j;
      if (g <= p.G) bars->cum[g] = run;
      run += cnt[j];
    }
    if (lane * 8 + 8 == p.G) bars->cum[p.G] = run;      // G a multiple of 8: the total has no lane of its own when G = 256
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // both CTAs' barriers exist before any remote access
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const int* cum = bars->cum;
  const int tiles_m = p.group_mode == 1 ? cum[p.G] : p.tiles_m;
  const int num_tiles = p.group_mode == 1 ? tiles_m * p.tiles_n : p.num_tiles;

  if (warp == 0) {
    // ===== TMA producer (both CTAs): own rows of A, own half of B, counted on the leader's barrier =====
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool alive = true;
      uint32_t local = 0, sync_misses = 0;
      for (int t = cluster_id; t < num_tiles && alive; t += num_clusters, ++local) {
        const PairTile tile = decode_pair(p, cum, tiles_m, t);
        const int m0 = tile.m0 + static_cast<int>(rank) * BM;
        const int n0 = tile.n0 + static_cast<int>(rank) * (BN / 2);
        if (p.tile_sync) {
          // Rendezvous of all CTA pairs at the start of their local-th tile. Pairs that share an operand panel only find
          // each other's loads in L2 while they walk the contraction together; left alone they drift apart by a few
          // percent per tile (measured: 2.5 us per 80 us tile) and the sharing is gone after a few waves. Best effort:
          // a pair waits a fraction of a tile time at most, then goes on alone; after two such misses it stops waiting
          // (the grid may not be co-resident, e.g. next to another stream's kernel), so nothing can hang or fail.
          if (leader) atomicAdd(p.tile_sync, 1u);
          if (local > 0 && sync_misses < 2) {
            const uint32_t target = static_cast<uint32_t>(min(static_cast<long long>(local + 1) * num_clusters, static_cast<long long>(num_tiles)));
            const long long t0 = clock64();
            bool met = true;
            while (ld_acquire_gpu_u32(p.tile_sync) < target) {
              if (clock64() - t0 > p.tile_sync_limit) { met = false; break; }
              __nanosleep(64);
            }
            sync_misses = met ? 0u : sync_misses + 1u;
          }
        }
        for (int k = tile.k_begin; k < tile.k_end; k += BK) {
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, p.status)) { alive = false; break; }
          const uint32_t full_local = smem_u32(&bars->full[stage]);
          // plain variant: both CTAs' bytes are counted on the leader's barrier, which the MMA thread watches;
          // fused variant: each CTA counts its own bytes, its transform warps watch its own barrier
          const uint32_t full_leader = FUSE ? full_local : mapa_shared(full_local, 0);
          const uint32_t a_dst = tiles_base + stage * STAGE2_BYTES;
          const uint32_t b_dst = a_dst + A2_BYTES;
          if (FUSE) mbar_expect_tx(full_local, STAGE2_BYTES);
          else if (leader) mbar_expect_tx(full_local, 2 * STAGE2_BYTES);
          if (A_MN) {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(a_dst + i * 8192, &tmA, m0 + 64 * i, k, full_leader);
          } else {
            tma_load_2d_pair(a_dst, &tmA, k, m0, full_leader);
          }
          if (B_MN) {
#pragma unroll
            for (int i = 0; i < BN / 2 / 64; ++i) tma_load_2d_pair(b_dst + i * 8192, &tmB, n0 + 64 * i, tile.b_row_off + k, full_leader);
          } else {
            tma_load_2d_pair(b_dst, &tmB, k, tile.b_row_off + n0, full_leader);
          }
          ++issued;
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
      }
      (void)issued;
    }
  } else if (warp == 1) {
    // ===== MMA issuer (leader CTA only) =====
    if (leader && lane == 0) {
      const uint32_t idesc = instr_desc_pair<A_MN, B_MN>();
      uint32_t stage = 0, phase = 0, local = 0;
      bool alive = true;
      for (int t = cluster_id; t < num_tiles && alive; t += num_clusters, ++local) {
        const PairTile tile = decode_pair(p, cum, tiles_m, t);
        const uint32_t buf = local & 1u;
        const uint32_t use = local >> 1;
        if (!mbar_wait(smem_u32(&bars->acc_empty[buf]), (use & 1u) ^ 1u, abort_flag, p.status)) { alive = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * ACC_COLS;
        uint32_t accumulate = 0;
        for (int k = tile.k_begin; k < tile.k_end; k += BK) {
          if (!mbar_wait(smem_u32(FUSE ? &bars->ready[stage] : &bars->full[stage]), phase, abort_flag, p.status)) { alive = false; break; }
          tc_fence_after();
          const uint32_t a_addr = tiles_base + stage * STAGE2_BYTES;
          const uint64_t a_desc = smem_desc<A_MN>(a_addr);
          const uint64_t b_desc = smem_desc<B_MN>(a_addr + A2_BYTES);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            umma_bf16_pair(d_tmem, a_desc + kk * desc_k_step<A_MN>(), b_desc + kk * desc_k_step<B_MN>(), idesc, accumulate);
            accumulate = 1;
          }
          umma_commit_pair(smem_u32(&bars->empty[stage]));
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
        if (!alive) break;
        umma_commit_pair(smem_u32(&bars->acc_full[buf]));
      }
    }
  } else if (FUSE && warp >= 6) {
    // ===== transform warps (both CTAs): MXFP4 quantize-dequantize of the staged tiles, in place =====
    // Group g handles k-blocks g, g + GROUPS, ...: the groups work on different stages at the same time,
    // so the wake-up / fence / signal latency of one stage overlaps the arithmetic of the others.
    const int twarp = warp - 6;
    const int group = twarp / WARPS_PER_GROUP, wig = twarp % WARPS_PER_GROUP;
    uint32_t it = 0;                                  // running k-block count over all of this CTA's tiles
    bool alive = true;
    const bool a_nv = (FUSE & 1) && p.fuse_a_fmt == QF_FMT_NVFP4, b_nv = (FUSE & 2) && p.fuse_b_fmt == QF_FMT_NVFP4;
    const Nvfp4Tensor nt_a = nvfp4_tensor(a_nv ? __ldg(p.a_tscale) : 1.0f);
    for (int t = cluster_id; t < num_tiles && alive; t += num_clusters) {
      const PairTile tile = decode_pair(p, cum, tiles_m, t);
      const Nvfp4Tensor nt_b = nvfp4_tensor(b_nv ? __ldg(p.b_tscale + (p.b_tscale_per_group ? tile.group : 0)) : 1.0f);
      for (int k = tile.k_begin; k < tile.k_end; k += BK, ++it) {
        if (static_cast<int>(it % TRANSFORM_GROUPS) != group) continue;
        const uint32_t stage = it % STAGES2, phase = (it / STAGES2) & 1u;
        // one lane polls the barrier; the warp then proceeds together (the shuffles need all lanes)
        int got = 1;
        if (lane == 0) {
          // A group may run ahead of the others. Before trusting full[stage] for its second and later uses,
          // make sure the previous use of this stage has been consumed (its MMAs committed to empty[stage]);
          // otherwise a parity wait could be satisfied by the phase of the previous use.
          if (it >= STAGES2) got = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, p.status) ? 1 : 0;
          if (got) got = mbar_wait(smem_u32(&bars->full[stage]), phase, abort_flag, p.status) ? 1 : 0;
        }
        got = __shfl_sync(0xFFFFFFFFu, got, 0);
        if (!got) { alive = false; break; }
        const uint32_t a_addr = tiles_base + stage * STAGE2_BYTES;
        if (FUSE & 1) {
          if (a_nv) nvfp4_transform_tile<A2_BYTES / 16>(a_addr, wig, lane, nt_a);
          else mxfp4_transform_tile<A2_BYTES / 16>(a_addr, wig, lane, p.mxfp4_noclip != 0);
        }
        if (FUSE & 2) {
          if (b_nv) nvfp4_transform_tile<B2_BYTES / 16>(a_addr + A2_BYTES, wig, lane, nt_b);
          else mxfp4_transform_tile<B2_BYTES / 16>(a_addr + A2_BYTES, wig, lane, p.mxfp4_noclip != 0);
        }
        fence_async_smem();                          // make the generic-proxy writes visible to the tensor core
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(mapa_shared(smem_u32(&bars->ready[stage]), 0));
      }
    }
  } else if (SIDE && warp >= 6) {
    // ===== side jobs (both CTAs): grid-stride over the units of each job; no synchronisation with the other roles =====
    const int64_t first = static_cast<int64_t>(blockIdx.x) * (32 * SIDE_WARPS) + (threadIdx.x - NUM_THREADS);
    const int64_t stride = static_cast<int64_t>(gridDim.x) * (32 * SIDE_WARPS);
#pragma unroll 1
    for (int j = 0; j < 2; ++j) {
      const auto& job = p.side[j];
      if (job.nunits <= 0) continue;
      if (job.fmt == QF_FMT_NVFP4)
        qdq_fp4_body<QF_FMT_NVFP4, PlainLoader, false>(PlainLoader{job.in}, job.nunits, job.out, nullptr, nullptr,
                                                       nvfp4_tensor(__ldg(job.tscale)), false, false, nullptr, first, stride);
      else
        qdq_fp4_body<QF_FMT_MXFP4, PlainLoader, false>(PlainLoader{job.in}, job.nunits, job.out, nullptr, nullptr,
                                                       nvfp4_tensor(1.0f), false, job.noclip != 0, nullptr, first, stride);
    }
  } else {
    // ===== epilogue (both CTAs): own 128 accumulator rows =====
    const int quarter = warp & 3;
    uint32_t local = 0, which = 0;
    bool alive = true;
    const bool use_tma = !(p.accumulate != 0 && sizeof(OutT) == 2);
    for (int t = cluster_id; t < num_tiles && alive; t += num_clusters, ++local) {
      const PairTile tile = decode_pair(p, cum, tiles_m, t);
      const int m0 = tile.m0 + static_cast<int>(rank) * BM;
      const int n0 = tile.n0;
      const uint32_t buf = local & 1u;
      const uint32_t use = local >> 1;
      const bool got = mbar_wait(smem_u32(&bars->acc_full[buf]), use & 1u, abort_flag, p.status);
      if (!__all_sync(0xFFFFFFFFu, got)) { alive = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + buf * ACC_COLS + (static_cast<uint32_t>(quarter * 32) << 16);
      const bool empty_k = tile.k_end <= tile.k_begin;
      auto release = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(mapa_shared(smem_u32(&bars->acc_empty[buf]), 0));
      };
      if (use_tma) {
        epilogue_tile_tma<OutT>(&tmC, staging_base + static_cast<uint32_t>(warp - 2) * 8192u, which, taddr, m0 + quarter * 32, n0, tile.z,
                                tile.rows_limit, static_cast<int>(p.No), p.accumulate != 0, empty_k, lane, release);
      } else {
        const int row = m0 + quarter * 32 + lane;
        const bool row_ok = row < tile.rows_limit;
        OutT* row_ptr = static_cast<OutT*>(p.C) + static_cast<int64_t>(tile.z) * p.c_group_stride + static_cast<int64_t>(row) * p.ldc;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t acc[32];
          tmem_ld32(taddr + c * 32, acc);
          tmem_ld_wait();
          if (c == BN / 32 - 1) release();
          if (empty_k) {
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[j] = 0u;
          }
          const int col0 = n0 + c * 32;
          if (row_ok && col0 < p.No) store_chunk32<OutT>(row_ptr, col0, static_cast<int>(p.No), acc, true);
        }
      }
    }
    if (lane == 0) bulk_wait_all();
  }

  // ===== teardown: nobody leaves while the partner may still touch this CTA's memory or barriers =====
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
  if (clocked) kclock.stop(p.status);
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing will ever arrive at, with a
// short limit. The wait must give up, raise the abort flag and record QF_ERR_TIMEOUT; the kernel then
// returns normally and the context stays usable.
__global__ void selftest_timeout_kernel(uint32_t* status, long long limit_cycles, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_cycles);
    *gave_up = (!ok && abort_flag == 1) ? 1 : 0;
  }
}

// ---- host side --------------------------------------------------------------------------------------

// 2-D BF16 tensor map over a row-major [rows, cols] matrix with pitch ld (elements); box = {box_cols, box_rows}.
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Row-tiles per rasterization band. Tiles are walked row-tile fastest inside a band, so the band's A
// panel (band * tile_rows * Kc BF16 values) is what must stay in the 126 MB L2 while B streams past once
// per band: the larger the band the fewer times B is re-read from HBM. The panel is kept near 40 MB.
int band_rows(int64_t tile_rows, int64_t Kc, int tiles_m) {
  const int64_t per_tile = tile_rows * (Kc > 0 ? Kc : 1) * 2;
  int64_t band = (40ll << 20) / per_tile;
  if (band < 4) band = 4;
  if (band > 32) band = 32;
  if (band > tiles_m) band = tiles_m;
  return static_cast<int>(band < 1 ? 1 : band);
}

// Rasterization of plain problems on the two-CTA kernel. Tiles are walked in bands along one output dimension, the
// banded dimension fastest: the band's operand panels are re-read by every wave and stay in L2, the other operand
// streams past once per band. DRAM traffic is then about  banded + other * (number of bands),  so the SMALLER operand is
// the one to band (the product term is the same either way, the additive term is the banded operand). A band of panels
// is kept near 50 MB (measured on B200 with ncu at 8192 x 12288 x 4096: beyond that the band no longer survives in
// the 126 MB L2 and traffic doubles; hints to evict the streaming operand first made things worse, since that operand
// is shared by the CTAs of a wave), and the bands are made equal. Measured DRAM bytes per launch with this choice against
// row bands of 40 MB for every product: forward 514 vs 526 MB, dgrad 912 vs 1131 MB, wgrad 978 vs 1158 MB.
void choose_raster(int64_t Mo, int64_t No, int64_t Kc, int tiles_m, int tiles_n, int* raster, int* band) {
  const bool band_cols = No < Mo;                                   // B (No x Kc) is the smaller operand
  const int tiles = band_cols ? tiles_n : tiles_m;
  const int64_t panel = 256 * (Kc > 0 ? Kc : 1) * 2;                // bytes of one 256-wide operand panel
  int64_t band_max = (52ll << 20) / panel;
  if (band_max < 4) band_max = 4;
  const int64_t nbands = (tiles + band_max - 1) / band_max;
  *raster = band_cols ? 1 : 0;
  *band = static_cast<int>((tiles + nbands - 1) / nbands);
}

// 3-D tensor map over the output for the epilogue's TMA stores: [groups, rows, cols] with a
// box of 32 rows x 128 bytes, 128-byte swizzle. Plain outputs use groups = 1.
bool make_map_c(CUtensorMap* map, void* base, int c_dtype, int64_t groups, int64_t rows, int64_t cols, int64_t ld,
                int64_t group_stride) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  const cuuint64_t es = c_dtype == QF_DT_F32 ? 4 : 2;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows), static_cast<cuuint64_t>(groups)};
  const cuuint64_t gs = groups > 1 ? static_cast<cuuint64_t>(group_stride) : static_cast<cuuint64_t>(rows) * static_cast<cuuint64_t>(ld);
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * es, gs * es};
  const cuuint32_t box[3] = {static_cast<cuuint32_t>(128 / es), 32, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, c_dtype == QF_DT_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides,
             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool A_MN, bool B_MN, typename OutT>
cudaError_t launch_t(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const KParams& kp, int grid,
                     cudaStream_t st) {
  auto kern = gemm_kernel<A_MN, B_MN, OutT>;
  static bool configured[64] = {false};           // per device: the attribute is a per-context property of the kernel
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  kern<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tmA, tmB, tmC, kp);
  return cudaGetLastError();
}

template <bool A_MN, bool B_MN, typename OutT, int FUSE, bool SIDE = false>
cudaError_t launch_pair_t(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, const KParams& kp, int grid,
                          cudaStream_t st) {
  auto kern = gemm_pair_kernel<A_MN, B_MN, OutT, FUSE, SIDE>;
  static bool configured[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return cudaGetLastError();
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  kern<<<grid, FUSE ? NUM_THREADS_FUSED : (SIDE ? NUM_THREADS_SIDE : NUM_THREADS), SMEM2_BYTES, st>>>(tmA, tmB, tmC, kp);   // cluster shape (2,1,1) is a kernel attribute
  return cudaGetLastError();
}

template <typename OutT>
cudaError_t launch_pair_majors(const GemmArgs& a, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                               const KParams& kp, int grid, cudaStream_t st) {
  const int fuse = (a.fuse_a_fmt ? 1 : 0) | (a.fuse_b_fmt ? 2 : 0);
  if (a.side[0].nelem > 0 || a.side[1].nelem > 0) {
    if (fuse != 0 || a.a_mn_major) return cudaErrorInvalidValue;          // see gemm_side_supported
    if (a.b_mn_major) return launch_pair_t<false, true, OutT, 0, true>(tmA, tmB, tmC, kp, grid, st);
    return launch_pair_t<false, false, OutT, 0, true>(tmA, tmB, tmC, kp, grid, st);
  }
  if (!a.a_mn_major && !a.b_mn_major) {
    if (fuse == 3) return launch_pair_t<false, false, OutT, 3>(tmA, tmB, tmC, kp, grid, st);
    if (fuse == 2) return launch_pair_t<false, false, OutT, 2>(tmA, tmB, tmC, kp, grid, st);
    if (fuse == 1) return launch_pair_t<false, false, OutT, 1>(tmA, tmB, tmC, kp, grid, st);
    return launch_pair_t<false, false, OutT, 0>(tmA, tmB, tmC, kp, grid, st);
  }
  if (!a.a_mn_major && a.b_mn_major) {
    if (fuse == 2) return launch_pair_t<false, true, OutT, 2>(tmA, tmB, tmC, kp, grid, st);
    if (fuse != 0) return cudaErrorInvalidValue;
    return launch_pair_t<false, true, OutT, 0>(tmA, tmB, tmC, kp, grid, st);
  }
  if (a.a_mn_major && a.b_mn_major) {
    if (fuse == 2) return launch_pair_t<true, true, OutT, 2>(tmA, tmB, tmC, kp, grid, st);
    if (fuse != 0) return cudaErrorInvalidValue;
    return launch_pair_t<true, true, OutT, 0>(tmA, tmB, tmC, kp, grid, st);
  }
  if (fuse != 0) return cudaErrorInvalidValue;
  return launch_pair_t<true, false, OutT, 0>(tmA, tmB, tmC, kp, grid, st);
}

template <typename OutT>
cudaError_t launch_majors(const GemmArgs& a, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                          const KParams& kp, int grid, cudaStream_t st) {
  if (!a.a_mn_major && !a.b_mn_major) return launch_t<false, false, OutT>(tmA, tmB, tmC, kp, grid, st);
  if (!a.a_mn_major && a.b_mn_major) return launch_t<false, true, OutT>(tmA, tmB, tmC, kp, grid, st);
  if (a.a_mn_major && a.b_mn_major) return launch_t<true, true, OutT>(tmA, tmB, tmC, kp, grid, st);
  return launch_t<true, false, OutT>(tmA, tmB, tmC, kp, grid, st);
}

}  // namespace

cudaError_t launch_selftest_timeout(uint32_t* status, long long limit_cycles, int* gave_up, cudaStream_t st) {
  selftest_timeout_kernel<<<1, 32, 0, st>>>(status, limit_cycles, gave_up);
  return cudaGetLastError();
}

// Two-CTA path: plain problems whose output has at least one full 256-row pair tile.
cudaError_t launch_gemm_pair(const GemmArgs& a, cudaStream_t st) {
  KParams kp{};
  kp.C = a.C;
  kp.Mo = a.group_mode == 1 ? a.rows_padded : a.Mo;
  kp.No = a.No;
  kp.Kc = a.Kc;
  kp.ldc = a.ldc;
  kp.c_dtype = a.c_dtype;
  kp.accumulate = a.accumulate ? 1 : 0;
  kp.status = a.status_word;
  // Tile-start rendezvous for plain problems with long contractions (measured at 32768 x 4096 x 14336: DRAM reads of the dX
  // launch 8.7 -> 4.1 GB, 2719 -> 2480 us; neutral from 8192 to 12288; a loss below, where a tile lasts 25 us).
  kp.tile_sync = (a.group_mode == 0 && a.Kc >= 8192) ? a.tile_sync_word : nullptr;
  kp.tile_sync_limit = a.Kc;                   // one eighth of a tile's main loop (Kc / 64 k-blocks of about 512 clocks)
  kp.mxfp4_noclip = a.mxfp4_noclip ? 1 : 0;
  kp.fuse_a_fmt = a.fuse_a_fmt;
  kp.fuse_b_fmt = a.fuse_b_fmt;
  kp.a_tscale = a.fuse_a_tscale;
  kp.b_tscale = a.fuse_b_tscale;
  kp.b_tscale_per_group = a.fuse_b_tscale_per_group ? 1 : 0;
  for (int j = 0; j < 2; ++j) {
    kp.side[j].in = static_cast<const uint4*>(a.side[j].in);
    kp.side[j].out = static_cast<uint4*>(a.side[j].out);
    kp.side[j].nunits = a.side[j].nelem / 16;
    kp.side[j].tscale = a.side[j].tscale;
    kp.side[j].fmt = a.side[j].fmt;
    kp.side[j].noclip = a.side[j].mxfp4_noclip ? 1 : 0;
  }
  kp.group_mode = a.group_mode;
  kp.G = a.G;
  kp.offs = a.group_offsets;
  kp.c_group_stride = a.c_group_stride;
  const int64_t a_rows_total = kp.Mo;
  // mode 1: the true number of pair row-tiles is only known on the device (it depends on the segment
  // lengths); this is an upper bound used for the grid size and the band width
  kp.tiles_m = static_cast<int>((a_rows_total + 2 * BM - 1) / (2 * BM)) + (a.group_mode == 1 ? a.G : 0);
  kp.tiles_n = static_cast<int>((a.No + BN - 1) / BN);
  kp.num_tiles = kp.tiles_m * kp.tiles_n * (a.group_mode == 2 ? a.G : 1);
  const int64_t contraction_rows = a.group_mode == 2 ? a.rows_padded : a.Kc;
  kp.band = band_rows(2 * BM, a.group_mode == 2 ? a.rows_padded / (a.G > 0 ? a.G : 1) : a.Kc, kp.tiles_m);
  if (a.group_mode == 0) choose_raster(a.Mo, a.No, a.Kc, kp.tiles_m, kp.tiles_n, &kp.raster, &kp.band);
  CUtensorMap tmA, tmB;
  bool ok;
  if (a.a_mn_major) ok = make_map(&tmA, a.A, contraction_rows, a.Mo, a.lda, 64, BK);
  else ok = make_map(&tmA, a.A, a_rows_total, a.Kc, a.lda, BK, BM);
  if (!ok) return cudaErrorInvalidValue;
  const int64_t groups_b = a.group_mode == 1 ? a.G : 1;
  if (a.b_mn_major) {
    ok = make_map(&tmB, a.B, a.group_mode == 1 ? groups_b * a.Kc : contraction_rows, a.No, a.ldb, 64, BK);
    kp.b_group_rows = a.Kc;
  } else {
    ok = make_map(&tmB, a.B, groups_b * a.No, a.Kc, a.ldb, BK, BN / 2);
    kp.b_group_rows = a.No;
  }
  if (!ok) return cudaErrorInvalidValue;
  CUtensorMap tmC;
  const bool per_group_c = a.group_mode == 2;
  if (!make_map_c(&tmC, a.C, a.c_dtype, per_group_c ? a.G : 1, kp.Mo, a.No, a.ldc, a.c_group_stride)) return cudaErrorInvalidValue;
  const int clusters = kp.num_tiles < kNumSMs / 2 ? kp.num_tiles : kNumSMs / 2;
  const int grid = 2 * clusters;
  if (a.c_dtype == QF_DT_F32) return launch_pair_majors<float>(a, tmA, tmB, tmC, kp, grid, st);
  return launch_pair_majors<__nv_bfloat16>(a, tmA, tmB, tmC, kp, grid, st);
}

// Problems the two-CTA kernel takes: plain ones with at least one full 256-row tile, and grouped ones
// whose expert count fits its shared-memory tile table (segments start on multiples of 128 rows).
static bool pair_applies(const GemmArgs& a) {
  if (a.Kc <= 0) return false;
  if (a.group_mode == 0) return a.Mo >= 2 * BM;
  if (a.G < 1 || a.G > MAX_PAIR_GROUPS) return false;
  if (a.group_mode == 1) return a.rows_padded >= 2 * BM;
  return a.Mo >= 2 * BM && a.rows_padded > 0;
}

// True if launch_gemm would run this problem on the kernel that can quantize-dequantize staged tiles itself
// (plain and grouped problems alike: the transform works on whatever tile the producer staged).
bool gemm_can_fuse(const GemmArgs& a) { return pair_applies(a); }

// True if this product runs on the two-CTA kernel in a variant that can carry side jobs (forward and dX products
// without the in-kernel quantizer). A launch with side jobs always uses every SM, however few tiles it has.
bool gemm_side_supported(const GemmArgs& a) { return pair_applies(a) && !a.a_mn_major && !a.fuse_a_fmt && !a.fuse_b_fmt; }

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st) {
  if (a.Mo <= 0 || a.No <= 0) return cudaSuccess;
  if (pair_applies(a)) return launch_gemm_pair(a, st);
  if (a.fuse_a_fmt || a.fuse_b_fmt || a.side[0].nelem > 0 || a.side[1].nelem > 0) return cudaErrorInvalidValue;   // only the two-CTA kernel fuses or carries side jobs
  KParams kp{};
  kp.C = a.C;
  kp.Mo = a.Mo;
  kp.No = a.No;
  kp.Kc = a.Kc;
  kp.ldc = a.ldc;
  kp.c_dtype = a.c_dtype;
  kp.accumulate = a.accumulate ? 1 : 0;
  kp.group_mode = a.group_mode;
  kp.G = a.G;
  kp.offs = a.group_offsets;
  kp.c_group_stride = a.c_group_stride;
  kp.status = a.status_word;
  kp.mxfp4_noclip = 0;
  const int64_t a_rows_total = a.group_mode == 1 ? a.rows_padded : a.Mo;   // rows of A (and of C) in mode 1
  kp.tiles_m = static_cast<int>((a_rows_total + BM - 1) / BM);
  kp.tiles_n = static_cast<int>((a.No + BN - 1) / BN);
  kp.num_tiles = kp.tiles_m * kp.tiles_n * (a.group_mode == 2 ? a.G : 1);
  kp.band = band_rows(BM, a.group_mode == 2 ? a.rows_padded / (a.G > 0 ? a.G : 1) : a.Kc, kp.tiles_m);
  if (a.group_mode == 1) kp.Mo = a.rows_padded;
  if (kp.num_tiles <= 0) return cudaSuccess;

  // Tensor maps. K-major operand: matrix [rows, contraction]; MN-major operand: matrix [contraction, rows].
  const int64_t contraction_rows = a.group_mode == 2 ? a.rows_padded : a.Kc;
  CUtensorMap tmA, tmB;
  bool ok;
  if (a.a_mn_major) ok = make_map(&tmA, a.A, contraction_rows, a.Mo, a.lda, 64, BK);
  else ok = make_map(&tmA, a.A, a_rows_total, a.Kc, a.lda, BK, BM);
  if (!ok) return cudaErrorInvalidValue;
  const int64_t groups_b = a.group_mode == 1 ? a.G : 1;
  if (a.b_mn_major) {
    // [groups * Kc, No] (mode 1) or [contraction_rows, No]
    const int64_t rows = a.group_mode == 1 ? groups_b * a.Kc : contraction_rows;
    ok = make_map(&tmB, a.B, rows, a.No, a.ldb, 64, BK);
    kp.b_group_rows = a.Kc;
  } else {
    ok = make_map(&tmB, a.B, groups_b * a.No, a.Kc, a.ldb, BK, BN);
    kp.b_group_rows = a.No;
  }
  if (!ok) return cudaErrorInvalidValue;

  CUtensorMap tmC;
  const bool per_group_c = a.group_mode == 2;
  if (!make_map_c(&tmC, a.C, a.c_dtype, per_group_c ? a.G : 1, kp.Mo, a.No, a.ldc, a.c_group_stride)) return cudaErrorInvalidValue;
  const int grid = kp.num_tiles < kNumSMs ? kp.num_tiles : kNumSMs;
  if (a.c_dtype == QF_DT_F32) return launch_majors<float>(a, tmA, tmB, tmC, kp, grid, st);
  return launch_majors<__nv_bfloat16>(a, tmA, tmB, tmC, kp, grid, st);
}

}  // namespace qf
