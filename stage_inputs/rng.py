"""Counter-based random numbers for the synthetic workloads.

Every tensor gets its own SplitMix64 stream, selected by (seed, tensor_id); the
i-th 64-bit word of a stream is a pure function of (seed, tensor_id, i), so any
slice of any tensor can be regenerated independently and in any language.

    key(seed, tid) = mix(mix(seed) + GOLDEN * (tid + 1))
    word_i         = mix(key + GOLDEN * (i + 1))
    mix(z): z ^= z >> 30; z *= 0xBF58476D1CE4E5B9; z ^= z >> 27;
            z *= 0x94D049BB133111EB; z ^= z >> 31          (all mod 2^64)

uniform  u_i = ((word_i >> 11) + 0.5) * 2^-53              in (0, 1)
normal   Box-Muller on the word pair (2j, 2j+1):
         r = sqrt(-2 ln u_2j), t = 2 pi u_2j+1, z_2j = r cos t, z_2j+1 = r sin t
label    floor(u_i * classes)
"""
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z):
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def tensor_key(seed, tensor_id):
    with np.errstate(over="ignore"):
        return _mix(_mix(np.uint64(seed)) + _GOLDEN * np.uint64(tensor_id + 1))


def _words(seed, tensor_id, n, start=0):
    idx = np.arange(start + 1, start + n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(tensor_key(seed, tensor_id) + _GOLDEN * idx)


def uniform(seed, tensor_id, n):
    """n doubles in (0, 1)."""
    w = _words(seed, tensor_id, n)
    return ((w >> np.uint64(11)).astype(np.float64) + 0.5) * (2.0 ** -53)


def normal(seed, tensor_id, shape):
    """N(0,1) samples (float64) of the given shape."""
    n = int(np.prod(shape))
    m = (n + 1) // 2
    u = uniform(seed, tensor_id, 2 * m)
    r = np.sqrt(-2.0 * np.log(u[0::2]))
    t = 2.0 * np.pi * u[1::2]
    z = np.empty(2 * m, dtype=np.float64)
    z[0::2] = r * np.cos(t)
    z[1::2] = r * np.sin(t)
    return z[:n].reshape(shape)


def labels(seed, tensor_id, n, classes):
    """n integer labels uniform on [0, classes)."""
    return np.floor(uniform(seed, tensor_id, n) * classes).astype(np.int32)
