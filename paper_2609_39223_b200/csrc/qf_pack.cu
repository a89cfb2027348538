// Engine-native packing of quantized weights (the export / weight-synchronisation step of the paper,
// Section 3.4 "Low-precision weight synchronization" and Section 3.5 "Packing the checkpoint"): lossless
// re-layouts of the codes and metadata qf_qdq emits. Pure data movement, one pass, 16-byte accesses.
//   * GGUF Q4_K: 144-byte records {fp16 d, fp16 dmin, 12 packed 6-bit bytes, 128 code bytes} per 256 weights.
//   * FP4 block scales for block-scaled tensor-core GEMMs (the layout vLLM / SGLang hand to their FP4
//     kernels): scales padded to multiples of 128 rows x 4 scale columns and stored tile by tile, 512
//     bytes per tile, byte (r, c) of a tile at (r mod 32) * 16 + (r div 32) * 4 + c. The 4-bit codes need
//     no re-layout (two per byte, even element in the low nibble, row-major).
#include "qf_common.cuh"

namespace qf {
namespace {

__global__ void __launch_bounds__(256) pack_q4k_kernel(const uint4* __restrict__ codes, const uint4* __restrict__ scales,
                                                       int64_t nsb, uint4* __restrict__ records, int unpack,
                                                       uint4* __restrict__ codes_out, uint4* __restrict__ scales_out) {
  const int64_t total = nsb * 9;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < total; i += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t sb = i / 9;
    const int j = static_cast<int>(i - sb * 9);
    if (!unpack) {
      records[i] = j == 0 ? __ldg(scales + sb) : __ldg(codes + sb * 8 + (j - 1));
    } else {
      const uint4 v = __ldg(records + i);
      if (j == 0) scales_out[sb] = v; else codes_out[sb * 8 + (j - 1)] = v;
    }
  }
}

// one thread per 32-bit word of the swizzled buffer = the four scale columns of one row of one tile
__global__ void __launch_bounds__(256) swizzle_scales_kernel(const uint8_t* __restrict__ scales, int64_t rows, int64_t nblk,
                                                             int64_t row_tiles, int64_t col_tiles, uint32_t* __restrict__ out) {
  const int64_t total = row_tiles * col_tiles * 128;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < total; i += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t tile = i >> 7;
    const int w = static_cast<int>(i & 127);          // word within the tile: (r mod 32) * 4 + (r div 32)
    const int r_in = (w >> 2) + 32 * (w & 3);
    const int64_t r = (tile / col_tiles) * 128 + r_in;
    const int64_t c0 = (tile % col_tiles) * 4;
    uint32_t v = 0;
    if (r < rows) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (c0 + c < nblk) v |= static_cast<uint32_t>(scales[r * nblk + c0 + c]) << (8 * c);
    }
    out[i] = v;
  }
}

__global__ void __launch_bounds__(256) unswizzle_scales_kernel(const uint8_t* __restrict__ swz, int64_t rows, int64_t nblk,
                                                               int64_t col_tiles, uint8_t* __restrict__ scales) {
  const int64_t total = rows * nblk;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < total; i += static_cast<int64_t>(gridDim.x) * 256) {
    const int64_t r = i / nblk, c = i - r * nblk;
    const int64_t tile = (r >> 7) * col_tiles + (c >> 2);
    const int r_in = static_cast<int>(r & 127);
    scales[i] = swz[tile * 512 + (r_in & 31) * 16 + (r_in >> 5) * 4 + (c & 3)];
  }
}

int grid_of(int64_t items) {
  int64_t b = (items + 255) / 256;
  const int64_t cap = static_cast<int64_t>(kNumSMs) * 16;
  if (b > cap) b = cap;
  return static_cast<int>(b < 1 ? 1 : b);
}

}  // namespace

cudaError_t launch_pack_q4k(const void* codes, const void* scales, int64_t nsb, void* records, bool unpack, void* codes_out,
                            void* scales_out, cudaStream_t st) {
  if (nsb == 0) return cudaSuccess;
  pack_q4k_kernel<<<grid_of(nsb * 9), 256, 0, st>>>(static_cast<const uint4*>(codes), static_cast<const uint4*>(scales), nsb,
                                                    static_cast<uint4*>(records), unpack ? 1 : 0, static_cast<uint4*>(codes_out),
                                                    static_cast<uint4*>(scales_out));
  return cudaGetLastError();
}

cudaError_t launch_swizzle_scales(const void* scales, int64_t rows, int64_t nblk, void* out, bool unswizzle, cudaStream_t st) {
  const int64_t row_tiles = (rows + 127) / 128, col_tiles = (nblk + 3) / 4;
  if (row_tiles * col_tiles == 0) return cudaSuccess;
  if (!unswizzle)
    swizzle_scales_kernel<<<grid_of(row_tiles * col_tiles * 128), 256, 0, st>>>(static_cast<const uint8_t*>(scales), rows, nblk,
                                                                               row_tiles, col_tiles, static_cast<uint32_t*>(out));
  else
    unswizzle_scales_kernel<<<grid_of(rows * nblk), 256, 0, st>>>(static_cast<const uint8_t*>(scales), rows, nblk, col_tiles,
                                                                   static_cast<uint8_t*>(out));
  return cudaGetLastError();
}

}  // namespace qf
