"""Counter-based random inputs.

Every value is a pure function of (seed, stream, index): element ``k`` of a
stream is SplitMix64's output for the counter ``k`` (Steele, Lea & Flood 2014,
"Fast splittable pseudorandom number generators": add the golden-gamma
constant, then two xor-shift-multiply rounds).  Normals come from Box-Muller on
two uniforms in double precision and are rounded to float32 once, at the end.
"""
import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# Stream ids keep inputs, labels and each tensor's initial values independent.
STREAM_X = 1
STREAM_LABEL = 2
STREAM_WEIGHT = 3


def splitmix64(seed, stream, index):
    """SplitMix64 output for counter `index` of stream (seed, stream)."""
    index = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        base = (np.uint64(seed) * np.uint64(0xD1342543DE82EF95)
                + np.uint64(stream) * np.uint64(0xA0761D6478BD642F))
        z = base + (index + np.uint64(1)) * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def uniform01(seed, stream, index):
    """Uniform double in (0, 1): top 53 bits, shifted off zero."""
    z = splitmix64(seed, stream, index)
    return ((z >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed, stream, n, offset=0):
    """`n` standard normals (float64) starting at element `offset`."""
    k = np.arange(offset, offset + n, dtype=np.uint64)
    u1 = uniform01(seed, stream, k * np.uint64(2))
    u2 = uniform01(seed, stream, k * np.uint64(2) + np.uint64(1))
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def labels(seed, n, n_classes, offset=0):
    """`n` labels uniform over range(n_classes), int32."""
    k = np.arange(offset, offset + n, dtype=np.uint64)
    z = splitmix64(seed, STREAM_LABEL, k)
    return (z % np.uint64(n_classes)).astype(np.int32)


def make_inputs(seed, n_ticks, sample_elems, n_classes, offset=0):
    """Samples x ~ N(0,1) as float32 [n_ticks, sample_elems] and their labels."""
    x = normal(seed, STREAM_X, n_ticks * sample_elems, offset * sample_elems)
    x = x.astype(np.float32).reshape(n_ticks, sample_elems)
    return x, labels(seed, n_ticks, n_classes, offset)


def he_normal_weights(seed, wl):
    """Initial parameters of a workload as one float32 vector in layer order.

    Conv and FC weights ~ N(0, 2/fan_in) with fan_in = c_in*k*k; FC biases 0;
    GroupNorm scale 1 and shift 0.  Tensor `q` of the list uses stream
    STREAM_WEIGHT + q so that changing one layer leaves the others' draws alone.
    """
    from .configs import param_sizes
    parts = []
    for q, (kind, n, fan_in) in enumerate(param_sizes(wl)):
        if kind == "weight":
            w = normal(seed, STREAM_WEIGHT + q, n) * np.sqrt(2.0 / fan_in)
            parts.append(w.astype(np.float32))
        elif kind == "ones":
            parts.append(np.ones(n, dtype=np.float32))
        else:
            parts.append(np.zeros(n, dtype=np.float32))
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)
