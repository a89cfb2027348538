// The deployment-side product: Y = deq(A) . deq(B)^T computed by the block-scaled FP4 tensor-core
// instruction (tcgen05.mma kind::mxf4 / kind::mxf4nvf4 with block scales in tensor memory) directly on the
// E2M1 codes and block scales the quantizer emits. The training path multiplies BF16 copies of the same
// dequantized values (Eq. fakequant); this kernel exists so that the two can be compared: for MXFP4 both
// sum the same exact products 2^(pA+pB) * C_A * C_B and may differ only in FP32 summation order.
//
// It is a checking tool, not a tuned matmul: one CTA per 128 x 128 output tile, one stage of shared memory,
// every step serialised. Per 256 contraction elements: TMA brings 128 rows x 128 bytes of packed codes per
// operand (128-byte swizzle, contraction-major); the CTA's threads gather the block scales of their row
// into the 512-byte scale atoms the copy-to-tensor-memory instruction expects; one thread copies the atoms
// to tensor memory and issues four MMAs of 64 contraction elements each.
//
// Scale atom (128 rows x 4 scales): byte (row % 32) * 16 + (row / 32) * 4 + j. `tcgen05.cp ... 32x128b.warpx4`
// copies its 32 x 16 bytes to 4 columns of every 32-lane quarter of tensor memory, which is where the MMA
// looks up the scales of row r: lane r % 32 of the quarter, column r / 32, byte j.
//
// Every mbarrier wait is bounded, as in the BF16 kernels.
#include <cuda.h>

#include "qf_common.cuh"
#include "qf_ptx.cuh"

namespace qf {
namespace {

constexpr int TM = 128, TN = 128;        // output tile
constexpr int TKB = 128;                 // bytes of packed codes per row per stage (256 elements)
constexpr int MMA_K_BYTES = 32;          // 64 FP4 elements per MMA
constexpr int TILE_BYTES = TM * TKB;     // 16 KB per operand
constexpr int ATOM_BYTES = 512;
constexpr int MAX_ATOMS = 4;             // per operand per stage: 256 / (4 * block) = 2 (block 32) or 4 (block 16)
constexpr int THREADS = 128;
constexpr int TMEM_COLS_FP4 = 256;       // 128 accumulator columns + 16 + 16 scale columns, rounded to a power of two
constexpr int SFA_COL = 128, SFB_COL = 144;
constexpr int SMEM_FP4 = 2 * TILE_BYTES + 2 * MAX_ATOMS * ATOM_BYTES + 1024 + 64;

struct alignas(8) Fp4Bars {
  uint64_t tma;
  uint64_t mma;
  uint32_t tmem_base;
  int abort_flag;
};

struct Fp4Params {
  const uint8_t* sfa;      // [M, K / block] scale bytes, row-major
  const uint8_t* sfb;      // [N, K / block]
  const float* tsa;        // NVFP4 tensor scales (device), else null
  const float* tsb;
  float* Y;                // [M, N] FP32
  int64_t M, N, K;
  int sf_tiled;            // scales come in the 512-byte tiles of QF_LAYOUT_FP4_SWIZZLED_SCALES instead of row-major
  uint32_t* status;
};

// shared-memory descriptor of a contraction-major, 128-byte-swizzled tile (8-row groups 1024 bytes apart)
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (1ull << 16) | (static_cast<uint64_t>(1024u >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// descriptor of one scale atom: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart
__device__ __forceinline__ uint64_t desc_atom(uint32_t addr) {
  return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (static_cast<uint64_t>(128u >> 4) << 32) | (1ull << 46);
}
__device__ __forceinline__ void tmem_cp_atom(uint32_t taddr, uint64_t desc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}

// Instruction descriptor of the block-scaled kinds: A, B = E2M1 (format 1), contraction-major, FP32 accumulate;
// scale type UE8M0 (bit 23) for block 32, UE4M3 for block 16; the byte of the 32-bit scale column an MMA
// starts at goes in bits 29-30 (A) and 4-5 (B).
template <bool NV>
__device__ __forceinline__ uint32_t instr_desc_fp4(uint32_t sf_byte) {
  return (sf_byte << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(TN >> 3) << 17) | ((NV ? 0u : 1u) << 23) |
         (static_cast<uint32_t>(TM >> 4) << 24) | (sf_byte << 29);
}

template <bool NV>
__device__ __forceinline__ void umma_fp4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa,
                                         uint32_t sfb, uint32_t accumulate) {
  if (NV) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%4], [%5], p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%4], [%5], p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate)
        : "memory");
  }
}

template <bool NV>
__global__ void __launch_bounds__(THREADS, 1)
fp4_native_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const Fp4Params p) {
  constexpr int BLOCK = NV ? 16 : 32;
  constexpr int SF_PER_STAGE = 2 * TKB / BLOCK;          // scales per row per stage: 8 or 16
  constexpr int ATOMS = SF_PER_STAGE / 4;
  constexpr uint32_t SF_FILL = NV ? 0u : 127u;           // past the edges: scale 0 (E4M3) / 1 (E8M0); the codes there are 0

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t a_tile = (raw + 1023u) & ~1023u;
  const uint32_t b_tile = a_tile + TILE_BYTES;
  const uint32_t sfa_smem = b_tile + TILE_BYTES;
  const uint32_t sfb_smem = sfa_smem + MAX_ATOMS * ATOM_BYTES;
  uint8_t* base_ptr = smem_raw + (a_tile - raw);
  uint32_t* sfa_ptr = reinterpret_cast<uint32_t*>(base_ptr + 2 * TILE_BYTES);
  uint32_t* sfb_ptr = sfa_ptr + MAX_ATOMS * ATOM_BYTES / 4;
  Fp4Bars* bars = reinterpret_cast<Fp4Bars*>(base_ptr + 2 * TILE_BYTES + 2 * MAX_ATOMS * ATOM_BYTES);
  volatile int* abort_flag = &bars->abort_flag;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM;
  const int64_t n0 = static_cast<int64_t>(blockIdx.x) * TN;
  const int64_t nsf = p.K / BLOCK;                        // scales per row

  if (tid == 0) {
    mbar_init(smem_u32(&bars->tma), 1);
    mbar_init(smem_u32(&bars->mma), 1);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&bars->tmem_base), TMEM_COLS_FP4);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  const int stages = static_cast<int>((p.K + 2 * TKB - 1) / (2 * TKB));
  bool alive = true;
  for (int kc = 0; kc < stages; ++kc) {
    const uint32_t phase = static_cast<uint32_t>(kc) & 1u;
    if (tid == 0) {
      mbar_expect_tx(smem_u32(&bars->tma), 2 * TILE_BYTES);
      tma_load_2d(a_tile, &tmA, kc * TKB, static_cast<int>(m0), smem_u32(&bars->tma));
      tma_load_2d(b_tile, &tmB, kc * TKB, static_cast<int>(n0), smem_u32(&bars->tma));
    }
    if (p.sf_tiled) {
      // already in atom order: tile (row tile, scale-column tile) is 512 contiguous bytes; copy word for word
      const int64_t tiles_c = (nsf + 3) / 4;
      const uint32_t* ga = reinterpret_cast<const uint32_t*>(p.sfa) + static_cast<int64_t>(blockIdx.y) * tiles_c * (ATOM_BYTES / 4);
      const uint32_t* gb = reinterpret_cast<const uint32_t*>(p.sfb) + static_cast<int64_t>(blockIdx.x) * tiles_c * (ATOM_BYTES / 4);
#pragma unroll
      for (int a = 0; a < ATOMS; ++a) {
        const int64_t ct = static_cast<int64_t>(kc) * ATOMS + a;
        const uint32_t fill = SF_FILL * 0x01010101u;
        sfa_ptr[a * (ATOM_BYTES / 4) + tid] = ct < tiles_c ? ga[ct * (ATOM_BYTES / 4) + tid] : fill;
        sfb_ptr[a * (ATOM_BYTES / 4) + tid] = ct < tiles_c ? gb[ct * (ATOM_BYTES / 4) + tid] : fill;
      }
    } else {
      // this thread's row of A and of B: SF_PER_STAGE scale bytes each, four to an atom
      const int64_t ra = m0 + tid, rb = n0 + tid;
      const int64_t sf0 = static_cast<int64_t>(kc) * SF_PER_STAGE;
      const int word = (tid & 31) * 4 + (tid >> 5);       // 32-bit word of this row inside an atom
#pragma unroll
      for (int a = 0; a < ATOMS; ++a) {
        uint32_t wa = 0, wb = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int64_t s = sf0 + 4 * a + j;
          const uint32_t va = (ra < p.M && s < nsf) ? p.sfa[ra * nsf + s] : SF_FILL;
          const uint32_t vb = (rb < p.N && s < nsf) ? p.sfb[rb * nsf + s] : SF_FILL;
          wa |= va << (8 * j);
          wb |= vb << (8 * j);
        }
        sfa_ptr[a * (ATOM_BYTES / 4) + word] = wa;
        sfb_ptr[a * (ATOM_BYTES / 4) + word] = wb;
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the copy to tensor memory reads through the async proxy
    __syncthreads();
    if (tid == 0) {
      if (mbar_wait(smem_u32(&bars->tma), phase, abort_flag, p.status)) {
        tc_fence_after();
#pragma unroll
        for (int a = 0; a < ATOMS; ++a) {
          tmem_cp_atom(tmem_base + SFA_COL + 4 * a, desc_atom(sfa_smem + a * ATOM_BYTES));
          tmem_cp_atom(tmem_base + SFB_COL + 4 * a, desc_atom(sfb_smem + a * ATOM_BYTES));
        }
#pragma unroll
        for (int j = 0; j < TKB / MMA_K_BYTES; ++j) {
          // block 16: one MMA uses the four scales of one 32-bit column; block 32: two MMAs share a column
          const uint32_t col = NV ? 4u * j : 4u * (j >> 1);
          const uint32_t sf_byte = NV ? 0u : 2u * (j & 1);
          const uint32_t sfa = tmem_base + SFA_COL + col;
          const uint32_t sfb = tmem_base + SFB_COL + col;
          umma_fp4<NV>(tmem_base, desc_sw128(a_tile) + static_cast<uint64_t>(j * (MMA_K_BYTES >> 4)),
                       desc_sw128(b_tile) + static_cast<uint64_t>(j * (MMA_K_BYTES >> 4)), instr_desc_fp4<NV>(sf_byte), sfa, sfb,
                       (kc > 0 || j > 0) ? 1u : 0u);
        }
        umma_commit(smem_u32(&bars->mma));
      }
    }
    // the MMAs read the tiles and the scale columns: nothing may be overwritten before they have completed
    mbar_wait(smem_u32(&bars->mma), phase, abort_flag, p.status);
    __syncthreads();                                   // every wait has ended: the abort flag is now the same for all
    if (*abort_flag) { alive = false; break; }
  }
  tc_fence_after();
  if (alive) {
    float scale = 1.0f;
    if (NV) scale = __fmul_rn(*p.tsa, *p.tsb);
    const int64_t row = m0 + warp * 32 + lane;
#pragma unroll 1
    for (int c = 0; c < TN / 32; ++c) {
      uint32_t acc[32];
      tmem_ld32(tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + c * 32, acc);
      tmem_ld_wait();
      if (row < p.M) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int64_t col = n0 + c * 32 + j;
          if (col < p.N) {
            const float v = __uint_as_float(acc[j]);
            p.Y[row * p.N + col] = NV ? __fmul_rn(v, scale) : v;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS_FP4);
}

// uint8 tensor map over packed codes [rows, K/2 bytes], box 128 bytes x 128 rows, 128-byte swizzle
bool make_map_codes(CUtensorMap* map, const void* base, int64_t rows, int64_t K) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K / 2), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K / 2)};
  const cuuint32_t box[2] = {TKB, TM};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool NV>
cudaError_t launch_fp4_t(const CUtensorMap& tmA, const CUtensorMap& tmB, const Fp4Params& p, dim3 grid, cudaStream_t st) {
  auto kern = fp4_native_kernel<NV>;
  static bool configured[64] = {false};
  int dev = 0;
  if (cudaError_t e = cudaGetDevice(&dev)) return e;
  if (dev < 0 || dev >= 64 || !configured[dev]) {
    if (cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_FP4)) return e;
    if (dev >= 0 && dev < 64) configured[dev] = true;
  }
  kern<<<grid, THREADS, SMEM_FP4, st>>>(tmA, tmB, p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fp4_native(const Fp4GemmArgs& a, cudaStream_t st) {
  if (a.M <= 0 || a.N <= 0) return cudaSuccess;
  if (a.K <= 0) return cudaMemsetAsync(a.Y, 0, static_cast<size_t>(a.M) * a.N * sizeof(float), st);
  CUtensorMap tmA, tmB;
  if (!make_map_codes(&tmA, a.a_codes, a.M, a.K) || !make_map_codes(&tmB, a.b_codes, a.N, a.K)) return cudaErrorInvalidValue;
  Fp4Params p{};
  p.sfa = static_cast<const uint8_t*>(a.a_scales);
  p.sfb = static_cast<const uint8_t*>(a.b_scales);
  p.tsa = a.a_tscale;
  p.tsb = a.b_tscale;
  p.Y = a.Y;
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.sf_tiled = a.scales_tiled ? 1 : 0;
  p.status = a.status_word;
  const dim3 grid(static_cast<unsigned>((a.N + TN - 1) / TN), static_cast<unsigned>((a.M + TM - 1) / TM));
  if (a.fmt == QF_FMT_NVFP4) return launch_fp4_t<true>(tmA, tmB, p, grid, st);
  return launch_fp4_t<false>(tmA, tmB, p, grid, st);
}

}  // namespace qf
