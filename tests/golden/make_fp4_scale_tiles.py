"""Writes tests/golden/fp4_scale_tiles.txt: where the oracle's tiled FP4 block-scale layout puts every
entry of a 130 x 6 scale matrix (pads to 256 rows x 8 scale columns = 2 x 2 tiles of 512 bytes).
Calls only the oracle. Run from the repository root: python tests/golden/make_fp4_scale_tiles.py"""
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))
import oracle  # noqa: E402

ROWS, NBLK = 130, 6


def main():
    lines = ["# Tiled FP4 block-scale layout (the form block-scaled tensor-core matmuls read; Section 3.5's",
             "# \"engine's native layout\"): byte offset of scale (row, block) of a 130 x 6 scale matrix in the",
             "# packed buffer of 2 x 2 tiles x 512 bytes. Written by make_fp4_scale_tiles.py from the oracle.",
             "# One line per row: row | offsets of blocks 0..5"]
    offs = np.zeros((ROWS, NBLK), np.int64)
    for c in range(NBLK):
        # one scale column at a time carries the row number (+1, so that padding stays distinguishable) in two passes
        for part, shift in ((0, 0), (1, 7)):
            s = np.zeros((ROWS, NBLK), np.uint8)
            s[:, c] = ((np.arange(ROWS) + 1) >> shift) & 127 | 128
            z = oracle.swizzle_block_scales(s)
            pos = np.flatnonzero(z)
            assert pos.size == ROWS
            vals = (z[pos] & 127).astype(np.int64)
            if part == 0:
                low = dict(zip(pos.tolist(), vals.tolist()))
            else:
                for p, hi in zip(pos.tolist(), vals.tolist()):
                    offs[(hi << 7 | low[p]) - 1, c] = p
    for r in range(ROWS):
        lines.append(f"{r} | " + " ".join(str(int(v)) for v in offs[r]))
    (Path(__file__).parent / "fp4_scale_tiles.txt").write_text("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
