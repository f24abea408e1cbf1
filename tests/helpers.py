"""Small numpy helpers shared by the tests (no method arithmetic lives here)."""
import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def alg1_python(W: int, N: int):
    """Algorithm 1 of the paper, literally, with Python list slices."""
    A, Q = [], []
    for t in range(N):
        if len(A) < 3 * W:
            A = A + [t]
        else:
            Q += A[1:2 * W:2]
            A = A[0:2 * W:2] + A[2 * W:3 * W]
            A = A + [t]
    return A, Q
