"""Counter-based seeded random tensors (numpy Philox).

Every tensor role gets its own (seed, stream) key, so a tensor's bytes do not
depend on which other tensors were drawn before it.
"""
import numpy as np


def _gen(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)]))


def normal(seed: int, stream: int, shape, std: float = 1.0, dtype=np.float32) -> np.ndarray:
    """N(0, std^2) samples of the given shape."""
    g = _gen(seed, stream)
    out = g.standard_normal(size=shape, dtype=np.float32 if dtype == np.float32 else np.float64)
    if std != 1.0:
        out *= out.dtype.type(std)
    return out.astype(dtype, copy=False)


def uniform01(seed: int, stream: int, shape, dtype=np.float32) -> np.ndarray:
    """Uniform samples in the open interval (0, 1)."""
    g = _gen(seed, stream)
    u = g.random(size=shape, dtype=np.float64)
    tiny = np.finfo(np.float32).tiny
    u = np.clip(u, tiny, 1.0 - 2.0 ** -24)
    return u.astype(dtype)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even).

    Returns fp32 whose low 16 mantissa bits are zero; a storage-format
    conversion, so that a bf16 device buffer and an fp64 oracle see the same
    numbers.
    """
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    src, dst = a.reshape(-1).view(np.uint32), out.reshape(-1).view(np.uint32)
    step = 1 << 24                                   # bounded temporaries for multi-GB tensors
    for i in range(0, src.size, step):
        bits = src[i:i + step]
        lsb = (bits >> np.uint32(16)) & np.uint32(1)
        # no finite input of interest is within 0x7fff of overflow, so uint32 arithmetic is exact here
        dst[i:i + step] = (bits + (np.uint32(0x7FFF) + lsb)) & np.uint32(0xFFFF0000)
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable fp32 values (after round_to_bf16)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(a.shape)
