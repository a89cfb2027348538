"""Small helpers shared by the tests: BF16 bit-pattern conversions (format conversions only)."""
import ml_dtypes
import numpy as np
import torch


def f32_to_bits(a) -> np.ndarray:
    """float array -> BF16 bit patterns (round to nearest even), as uint16."""
    return np.ascontiguousarray(np.asarray(a, np.float32).astype(ml_dtypes.bfloat16)).view(np.uint16)


def bits_to_f32(b) -> np.ndarray:
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def torch_to_bits(t: torch.Tensor) -> np.ndarray:
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_torch(b: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).view(torch.bfloat16).to(device)


def unpack_nibbles(codes: np.ndarray) -> np.ndarray:
    """[rows, cols/2] bytes -> [rows, cols] 4-bit codes, even element in the low nibble."""
    lo = codes & 15
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


E2M1_VALUES = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6], np.float32)
