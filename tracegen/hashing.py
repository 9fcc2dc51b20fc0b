"""Counter-based 64-bit mixer used by every sampler (numpy and CUDA restate the same steps).

The finaliser is the well-known xor-shift-multiply avalanche (shift 30, multiply, shift 27,
multiply, shift 31); word ``k`` of record ``i`` is ``mix64(base + STREAM[k] + i * GOLD)``.
"""
import numpy as np

MASK = 0xFFFFFFFFFFFFFFFF
GOLD = np.uint64(0x9E3779B97F4A7C15)
M1 = 0xBF58476D1CE4E5B9
M2 = 0x94D049BB133111EB
# per-field stream offsets
STREAM = (0x0000000000000000, 0x6A09E667F3BCC909, 0xBB67AE8584CAA73B)


def mix64_scalar(x: int) -> int:
    x &= MASK
    x ^= x >> 30
    x = (x * M1) & MASK
    x ^= x >> 27
    x = (x * M2) & MASK
    x ^= x >> 31
    return x


def mix64(x: np.ndarray) -> np.ndarray:
    """Vectorised mixer over uint64 arrays (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        x = np.asarray(x, dtype=np.uint64).copy()
        x ^= x >> np.uint64(30)
        x *= np.uint64(M1)
        x ^= x >> np.uint64(27)
        x *= np.uint64(M2)
        x ^= x >> np.uint64(31)
    return x


def word(base: int, k: int, idx: np.ndarray) -> np.ndarray:
    """Random word ``k`` for record indices ``idx`` (uint64 array)."""
    with np.errstate(over="ignore"):
        return mix64(np.uint64((base + STREAM[k]) & MASK) + idx * GOLD)
