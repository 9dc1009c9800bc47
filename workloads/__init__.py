"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

Only random-number plumbing lives here: no HiF8 arithmetic, no rounding, no scaling.  Every generator
returns numpy arrays of raw encodings (float32, or uint16 holding bfloat16 / binary16 bit patterns) so
that the CPU oracle and the CUDA library receive byte-identical inputs.

The recipes stand in for the tensors of the paper's CNN / Transformer / LLM experiments (whose datasets and
weights are not available): bell-shaped weights and activations, activations with a few outlier channels,
and gradients with a very wide dynamic range.
"""
import numpy as np


def f32_to_bf16_bits(x):
    """float32 array -> uint16 bfloat16 encodings, round-to-nearest-even (input preparation only)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    r = np.where(nan, (u >> 16) | 0x40, r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(h):
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal_f32(shape, seed, std=1.0):
    """i.i.d. N(0, std^2) in float32 (weights / activations / config-2 tensor)."""
    rng = np.random.Generator(np.random.Philox(seed))
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def normal_bf16(shape, seed, std=1.0):
    return f32_to_bf16_bits(normal_f32(shape, seed, std))


def llm_activation_bf16(tokens, hidden, seed, nu=3.0, outlier_frac=0.001, outlier_gain=100.0):
    """Student-t(nu) body with a fraction of hidden channels multiplied by `outlier_gain`
    (LLM activations with outlier channels); returns bfloat16 encodings [tokens, hidden]."""
    rng = np.random.Generator(np.random.Philox(seed))
    z = rng.standard_normal((tokens, hidden), dtype=np.float32)
    chi = np.zeros((tokens, hidden), dtype=np.float32)
    for _ in range(int(nu)):
        g = rng.standard_normal((tokens, hidden), dtype=np.float32)
        chi += g * g
    x = z / np.sqrt(chi / np.float32(nu))
    n_out = max(1, int(round(hidden * outlier_frac)))
    cols = rng.choice(hidden, size=n_out, replace=False)
    x[:, cols] *= np.float32(outlier_gain)
    return f32_to_bf16_bits(x)


def loguniform_f32(n, seed, lo_exp=-40, hi_exp=20):
    """Gradient-like stress tensor: random sign, exponent uniform integer in [lo_exp, hi_exp),
    23 uniform mantissa bits."""
    rng = np.random.Generator(np.random.Philox(seed))
    e = rng.integers(lo_exp, hi_exp, size=n, dtype=np.int64) + 127
    m = rng.integers(0, 1 << 23, size=n, dtype=np.int64)
    s = rng.integers(0, 2, size=n, dtype=np.int64)
    return ((s << 31) | (e << 23) | m).astype(np.uint32).view(np.float32)


def all_u16():
    """All 65,536 16-bit encodings in order."""
    return np.arange(65536, dtype=np.uint32).astype(np.uint16)


def random_bits_f32(n, seed):
    """Uniformly random 32-bit patterns viewed as float32 (covers NaN / Inf / subnormals)."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32).view(np.float32)


def random_codes(shape, seed, finite_only=True):
    """Random HiF8 bytes; with finite_only the NaN and Inf patterns are replaced by 0x08."""
    rng = np.random.Generator(np.random.Philox(seed))
    c = rng.integers(0, 256, size=shape, dtype=np.uint16).astype(np.uint8)
    if finite_only:
        bad = (c == 0x80) | ((c & 0x7F) == 0x6F)
        c = np.where(bad, np.uint8(0x08), c).astype(np.uint8)
    return c
