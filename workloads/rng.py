"""Counter-based random numbers and keyed bijections for the synthetic workloads.

Everything here is a pure function of (seed, stream, index), so any element of any
input can be regenerated on its own and the streams do not depend on a library's
generator implementation.  The mixing function is the splitmix64 output function
(Steele, Lea & Flood, "Fast splittable pseudorandom number generators", OOPSLA 2014).

This module holds no arithmetic of the contraction method: it only draws numbers.
"""
import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK64 = (1 << 64) - 1


def _mix(z):
    z = z.copy() if isinstance(z, np.ndarray) else np.asarray(z, dtype=np.uint64)
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def _base(seed, stream):
    """Scalar 64-bit key for one (seed, stream) pair."""
    s = (int(seed) * 0xD1342543DE82EF95 + (int(stream) + 1) * 0x9E3779B97F4A7C15) & _MASK64
    # one scalar splitmix round so that nearby seeds give unrelated keys
    s = (s ^ (s >> 30)) * 0xBF58476D1CE4E5B9 & _MASK64
    s = (s ^ (s >> 27)) * 0x94D049BB133111EB & _MASK64
    s ^= s >> 31
    return np.uint64(s)


def u64(seed, stream, idx):
    """64 random bits per entry of ``idx`` (any integer array)."""
    idx = np.asarray(idx).astype(np.uint64, copy=False)
    with np.errstate(over="ignore"):
        return _mix(idx * _GOLD + _base(seed, stream))


def uniform01(seed, stream, idx):
    """float64 in [0, 1) with 53 random bits."""
    return (u64(seed, stream, idx) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def uniform_f32(seed, stream, idx, lo, hi):
    """fp32 uniform on [lo, hi): a 24-bit fraction, exactly representable in fp32."""
    frac = (u64(seed, stream, idx) >> np.uint64(40)).astype(np.float32) * np.float32(1.0 / (1 << 24))
    return (np.float32(lo) + np.float32(hi - lo) * frac).astype(np.float32)


def normal_f32(seed, stream, idx):
    """fp32 standard normal (Box-Muller on two independent uniforms)."""
    idx = np.asarray(idx).astype(np.uint64, copy=False)
    u1 = uniform01(seed, stream, idx * np.uint64(2))
    u2 = uniform01(seed, stream, idx * np.uint64(2) + np.uint64(1))
    r = np.sqrt(-2.0 * np.log1p(-u1))          # 1-u1 is in (0, 1]
    return (r * np.cos(2.0 * np.pi * u2)).astype(np.float32)


def _bits_for(n):
    b = 2
    while (1 << b) < n:
        b += 1
    return b


def _round_fn(x, key, bits, mask):
    """One bijection of [0, 2^bits): odd multiply, key add, xor-shift (each invertible)."""
    h = np.uint64(max(1, bits // 2))
    with np.errstate(over="ignore"):
        x = (x * np.uint64(0x9E3779B1) + key) & mask
        x ^= x >> h
        x = (x * np.uint64(0x85EBCA6B) + (key >> np.uint64(17))) & mask
        x ^= x >> h
        x = (x * np.uint64(0xC2B2AE35) + (key >> np.uint64(31))) & mask
        x ^= x >> h
    return x


def keyed_bijection(c, n, key):
    """Image of ``c`` (values in [0, n)) under a pseudo-random bijection of [0, n).

    ``key`` is a uint64 scalar or an array broadcastable to ``c``: entries that share
    a key share a bijection, so distinct ``c`` under one key give distinct images.
    Built by cycle-walking a bijection of the enclosing power of two.
    """
    c = np.asarray(c).astype(np.uint64)
    n = int(n)
    if n <= 1:
        return np.zeros(c.shape, dtype=np.int64)
    bits = _bits_for(n)
    mask = np.uint64((1 << bits) - 1)
    key = np.asarray(key, dtype=np.uint64)
    if key.ndim == 0:
        key = np.broadcast_to(key, c.shape)
    x = _round_fn(c, key, bits, mask)
    todo = np.nonzero(x >= np.uint64(n))[0]
    while todo.size:
        xt = _round_fn(x[todo], key[todo], bits, mask)
        x[todo] = xt
        todo = todo[xt >= np.uint64(n)]
    return x.astype(np.int64)


def permutation(seed, stream, n):
    """A pseudo-random permutation of range(n) as an int64 array."""
    return keyed_bijection(np.arange(n, dtype=np.uint64), n, _base(seed, stream))
