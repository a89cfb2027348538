"""Engine-native packing (the export / weight-synchronisation step): oracle pins on CPU, and the CUDA
re-layout kernels against the oracle, byte for byte."""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from oracle import FMT_MXFP4, FMT_NVFP4, FMT_Q4_K
from paper_2609_39223_b200 import api, synth
from util import f32_to_bits, torch_to_bits

GOLDEN = Path(__file__).parent / "golden"


def _w(rows, cols, seed):
    rng = np.random.default_rng(seed)
    return f32_to_bits(rng.normal(0, 0.02, (rows, cols)))


def test_oracle_gguf_records_read_back_through_gguf():
    from gguf import GGMLQuantizationType as T, quants
    rows, cols = 5, 768
    r = oracle.qdq(FMT_Q4_K, _w(rows, cols, 1))
    rec = oracle.pack_gguf_q4k(r["codes"], r["scales"])
    assert rec.shape == (rows, cols // 256, 144)
    # llama.cpp's reader turns the records into exactly the quantizer's dequantized tensor (Eq. q4k-dequant)
    np.testing.assert_array_equal(f32_to_bits(quants.dequantize(rec.reshape(rows, -1), T.Q4_K)), r["out"])


def test_oracle_scale_swizzle_is_a_padded_bijection_with_the_documented_tile_layout():
    rows, nblk = 200, 10                               # pads to 256 rows x 12 scale columns = 2 x 3 tiles
    s = (np.arange(rows * nblk, dtype=np.int64) % 251 + 1).astype(np.uint8).reshape(rows, nblk)
    z = oracle.swizzle_block_scales(s)
    assert z.size == 2 * 3 * 512
    # hand-placed entries: first tile holds rows 0..127 x cols 0..3
    assert z[0] == s[0, 0] and z[1] == s[0, 1] and z[16] == s[1, 0] and z[4] == s[32, 0] and z[8 + 3] == s[64, 3]
    assert z[31 * 16 + 3 * 4 + 2] == s[127, 2]
    assert z[512] == s[0, 4]                            # second tile of the first tile row: scale columns 4..7
    assert z[3 * 512] == s[128, 0]                      # first tile of the second tile row
    # every source byte appears exactly where the inverse map says, everything else is padding (zero)
    seen = np.zeros(z.size, bool)
    for r in range(rows):
        for c in range(nblk):
            o = ((r // 128) * 3 + c // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + c % 4
            assert z[o] == s[r, c] and not seen[o]
            seen[o] = True
    assert not z[~seen].any()


def _tiled_scales_by_reshape(s: np.ndarray) -> np.ndarray:
    """The tiled scale-factor layout written a second way, from its description as nested blocks rather than as
    a byte-offset formula (NVIDIA's documentation of 1-D block-scaling factor layouts for block-scaled matmuls:
    128 x 4 scale tiles, each stored as 32 rows of 16 bytes in which row i holds the four scales of rows
    i, i + 32, i + 64, i + 96 one after another; tiles follow each other along the scale columns first)."""
    rows, nblk = s.shape
    rt, ct = -(-rows // 128), -(-nblk // 4)
    p = np.zeros((rt * 128, ct * 4), np.uint8)
    p[:rows, :nblk] = s
    # [row tile, quarter of the tile (rows 32q..32q+31), row in quarter, column tile, column in tile]
    return p.reshape(rt, 4, 32, ct, 4).transpose(0, 3, 2, 1, 4).reshape(-1)


@pytest.mark.parametrize("rows,nblk", [(1, 1), (128, 4), (130, 6), (200, 10), (257, 33), (384, 128)])
def test_oracle_scale_swizzle_equals_the_nested_block_description(rows, nblk):
    rng = np.random.default_rng(rows * 1000 + nblk)
    s = rng.integers(1, 256, (rows, nblk), dtype=np.uint8)
    np.testing.assert_array_equal(oracle.swizzle_block_scales(s), _tiled_scales_by_reshape(s))


def test_oracle_scale_swizzle_stored_offsets():
    """Byte offsets of every entry of a 130 x 6 scale matrix, stored by golden/make_fp4_scale_tiles.py; the
    first tile's first rows are also spelled out here by hand from the layout's description."""
    table = {}
    for line in (GOLDEN / "fp4_scale_tiles.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            r, offs = line.split("|")
            table[int(r)] = [int(v) for v in offs.split()]
    assert len(table) == 130
    # by hand: row 0 opens the tile; row 1 is the next 16-byte line; rows 32 / 64 / 96 share line 0 with row 0;
    # scale columns 4, 5 open the next tile (512 bytes on); row 128 opens the second row of tiles (2 tiles on)
    assert table[0] == [0, 1, 2, 3, 512, 513] and table[1][:4] == [16, 17, 18, 19]
    assert table[32][:4] == [4, 5, 6, 7] and table[64][:4] == [8, 9, 10, 11] and table[96][:4] == [12, 13, 14, 15]
    assert table[127][:4] == [508, 509, 510, 511] and table[128] == [1024, 1025, 1026, 1027, 1536, 1537]
    s = np.random.default_rng(5).integers(1, 256, (130, 6), dtype=np.uint8)
    z = oracle.swizzle_block_scales(s)
    used = np.zeros(z.size, bool)
    for r, offs in table.items():
        for c, o in enumerate(offs):
            assert z[o] == s[r, c]
            used[o] = True
    assert used.sum() == 130 * 6 and not z[~used].any()


@pytest.mark.gpu
@pytest.mark.parametrize("rows,cols", [(1, 256), (37, 1024), (300, 4096)])
def test_gpu_gguf_q4k_records(rows, cols):
    from gguf import GGMLQuantizationType as T, quants
    w = synth.randn_bf16((rows, cols), 0.02, rows)
    g = api.qf_qdq(api.FMT_Q4_K, w.cuda())
    packed = api.qf_pack(api.LAYOUT_GGUF_Q4_K, api.FMT_Q4_K, g["codes"], g["scales"], rows, cols)
    o = oracle.qdq(FMT_Q4_K, torch_to_bits(w))
    rec = oracle.pack_gguf_q4k(o["codes"], o["scales"])
    np.testing.assert_array_equal(packed.cpu().numpy(), rec.reshape(-1))
    # what an engine would load: the records alone reproduce the trained fake-quantized weights
    np.testing.assert_array_equal(f32_to_bits(quants.dequantize(packed.cpu().numpy().reshape(rows, -1), T.Q4_K)), torch_to_bits(g["out"]))
    codes, scales = api.qf_unpack(api.LAYOUT_GGUF_Q4_K, api.FMT_Q4_K, packed, rows, cols)     # lossless
    assert torch.equal(codes, g["codes"]) and torch.equal(scales, g["scales"])


@pytest.mark.gpu
@pytest.mark.parametrize("fmt", [api.FMT_NVFP4, api.FMT_MXFP4])
@pytest.mark.parametrize("rows,cols", [(1, 64), (200, 320), (129, 4096), (1024, 2048)])
def test_gpu_swizzled_fp4_scales(fmt, rows, cols):
    w = synth.randn_bf16((rows, cols), 0.02, rows + cols)
    g = api.qf_qdq(fmt, w.cuda())
    packed = api.qf_pack(api.LAYOUT_FP4_SWIZZLED_SCALES, fmt, None, g["scales"], rows, cols)
    want = oracle.swizzle_block_scales(oracle.qdq(fmt, torch_to_bits(w))["scales"])
    np.testing.assert_array_equal(packed.cpu().numpy(), want)
    _, scales = api.qf_unpack(api.LAYOUT_FP4_SWIZZLED_SCALES, fmt, packed, rows, cols)
    assert torch.equal(scales, g["scales"])


def test_pack_argument_errors_need_no_gpu():
    L = api.lib()
    P = 0x10000
    assert L.qf_pack(api.LAYOUT_GGUF_Q4_K, api.FMT_MXFP4, P, P, 4, 256, P, None) == 4       # layout/format mismatch
    assert L.qf_pack(api.LAYOUT_FP4_SWIZZLED_SCALES, api.FMT_Q4_K, P, P, 4, 256, P, None) == 4
    assert L.qf_pack(9, api.FMT_Q4_K, P, P, 4, 256, P, None) == 4
    assert L.qf_pack(api.LAYOUT_GGUF_Q4_K, api.FMT_Q4_K, P, P, 4, 128, P, None) == 2
    assert L.qf_pack(api.LAYOUT_GGUF_Q4_K, api.FMT_Q4_K, None, P, 4, 256, P, None) == 1
    assert api.qf_pack_bytes(api.LAYOUT_GGUF_Q4_K, api.FMT_Q4_K, 4, 512) == 4 * 2 * 144
    assert api.qf_pack_bytes(api.LAYOUT_FP4_SWIZZLED_SCALES, api.FMT_NVFP4, 200, 160) == 2 * 3 * 512
    assert api.qf_pack_bytes(api.LAYOUT_FP4_SWIZZLED_SCALES, api.FMT_MXFP4, 128, 128) == 512
