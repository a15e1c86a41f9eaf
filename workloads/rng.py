"""Counter-based integer random numbers: value = f(seed, tensor id, flat index).

All arithmetic is 64-bit integer (wrap-around) until one exact int->float conversion and one IEEE
float32 multiply, so the host (numpy) and the device fill kernel produce bit-identical tensors.

"N(0,1)" values are Irwin-Hall sums: eight 16-bit uniforms taken from two 64-bit hashes, centred and
scaled to unit variance (tails end at about +-4.9 sigma).  No transcendental function is used.
"""
import numpy as np

_U64 = np.uint64
GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_TIDMUL = 0xD1B54A32D192ED03
_TIDADD = 0x8CB92BA72F3D8DD7
_MASK = (1 << 64) - 1

# 1 / std(2*sum - 8*65535) with sum of eight uniform 16-bit integers; stored as an exact float32.
NORMAL_SCALE_F32 = np.float32(1.0 / (2.0 * np.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)))


def _fin_py(x: int) -> int:
    x &= _MASK
    x ^= x >> 30
    x = (x * _M1) & _MASK
    x ^= x >> 27
    x = (x * _M2) & _MASK
    x ^= x >> 31
    return x


def stream_key(seed: int, tid: int) -> int:
    """64-bit key of one tensor: depends on the seed and the tensor id only."""
    return _fin_py(_fin_py(seed + GOLD) ^ ((tid * _TIDMUL + _TIDADD) & _MASK))


def _fin_np(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint64, copy=True)
    x ^= x >> _U64(30)
    x *= _U64(_M1)
    x ^= x >> _U64(27)
    x *= _U64(_M2)
    x ^= x >> _U64(31)
    return x


def mix64(seed: int, tid: int, idx) -> np.ndarray:
    """uint64 hash of every flat index in ``idx`` (array-like of non-negative integers)."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _fin_np(idx * _U64(GOLD) + _U64(stream_key(seed, tid)))


def uniform_f64(seed: int, tid: int, idx) -> np.ndarray:
    """Uniform doubles in [0, 1): top 53 bits of the hash."""
    return (mix64(seed, tid, idx) >> _U64(11)).astype(np.float64) * (2.0 ** -53)


def normal_i32(seed: int, tid: int, idx) -> np.ndarray:
    """Centred integer 2*sum(eight 16-bit uniforms) - 8*65535, in [-524280, 524280]."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h1 = mix64(seed, tid, idx * _U64(2))
        h2 = mix64(seed, tid, idx * _U64(2) + _U64(1))
    s = np.zeros(idx.shape, dtype=np.int64)
    for h in (h1, h2):
        for sh in (0, 16, 32, 48):
            s += ((h >> _U64(sh)) & _U64(0xFFFF)).astype(np.int64)
    return (2 * s - 8 * 65535).astype(np.int32)


def normal_f32(seed: int, tid: int, idx) -> np.ndarray:
    return normal_i32(seed, tid, idx).astype(np.float32) * NORMAL_SCALE_F32


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16). Finite inputs only."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16_bits(seed: int, tid: int, idx) -> np.ndarray:
    return f32_to_bf16_bits(normal_f32(seed, tid, idx))
