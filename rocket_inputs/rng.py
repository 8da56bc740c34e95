"""Counter-based random numbers: a pure function of (seed, stream, index).

The 64-bit mixer is the published splitmix64 finaliser.  Two rounds are chained so
that a value depends on the seed, on a stream id (the kernel index) and on a slot
within the stream.  The C++ generator inside the library implements the same
function, so both sides can draw identical kernel parameters from one seed.
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


def counter_u64(seed, stream, slot):
    """64 random bits for (seed, stream, slot); arguments broadcast like numpy arrays."""
    seed = np.asarray(seed, dtype=np.uint64)
    stream = np.asarray(stream, dtype=np.uint64)
    slot = np.asarray(slot, dtype=np.uint64)
    with np.errstate(over="ignore"):
        a = _mix(seed + _GOLDEN * (stream + np.uint64(1)))
        return _mix(a + _GOLDEN * (slot + np.uint64(1)))


def counter_uniform(seed, stream, slot):
    """Uniform double in [0, 1) with 53 random bits."""
    return (counter_u64(seed, stream, slot) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)
