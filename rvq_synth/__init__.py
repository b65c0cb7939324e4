"""Seeded synthetic inputs for the residual-VQ KV-cache compressor.

This module only draws numbers.  It holds none of the quantizer's arithmetic
(no standard deviation, no grouping, no distance, no codeword search), so both
the CPU oracle's tests and the CUDA path's tests/benchmarks may use it without
sharing any of the method between them.

Random numbers come from one counter-based generator, SplitMix64 (Steele,
Lea & Flood, "Fast splittable pseudorandom number generators", OOPSLA 2014):
value ``i`` of a stream is ``mix(seed + (i + 1) * GOLDEN)``, so every array is a
pure function of ``(seed, stream tag, index)`` and does not depend on a library
version.  Normals use Box-Muller on two uniforms, Laplace the inverse CDF.

The five workloads mirror the shapes the paper works with (Section 3: head
dimension 128, groups of 32 channels, residual depth 8, 1024 or 2048 codes per
codebook, 64K-token batches) with heavy-tailed per-channel scales standing in
for real key/value projections.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22

CONTIGUOUS = 0
STRIDED = 1


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def splitmix64(seed: int, start: int, count: int) -> np.ndarray:
    """Values ``start .. start+count-1`` of the SplitMix64 stream ``seed``."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        return _mix(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GOLDEN)


def stream_seed(seed: int, tag: str) -> int:
    """Derive an independent stream seed from a workload seed and a name."""
    h = seed & 0xFFFFFFFFFFFFFFFF
    for ch in tag.encode():
        h = int(splitmix64(h ^ ch, 0, 1)[0])
    return h


def uniform01(seed: int, start: int, count: int) -> np.ndarray:
    """Uniform doubles in the open interval (0, 1), 53 bits each."""
    u = splitmix64(seed, start, count) >> np.uint64(11)
    return (u.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, count: int) -> np.ndarray:
    """``count`` standard normals (Box-Muller, cosine branch), float64."""
    out = np.empty(count, dtype=np.float64)
    for lo in range(0, count, _CHUNK):
        m = min(_CHUNK, count - lo)
        u = uniform01(seed, 2 * lo, 2 * m)
        out[lo:lo + m] = np.sqrt(-2.0 * np.log(u[0::2])) * np.cos(2.0 * np.pi * u[1::2])
    return out


def laplace(seed: int, count: int) -> np.ndarray:
    """``count`` Laplace(0, 1) draws by the inverse CDF, float64."""
    u = uniform01(seed, 0, count) - 0.5
    return -np.sign(u) * np.log1p(-2.0 * np.abs(u))


def randint(seed: int, count: int, high: int) -> np.ndarray:
    """``count`` integers uniform on ``[0, high)``: bits 20.. of the draw when
    ``high`` is a power of two, else the top 32 bits scaled by ``high``."""
    assert 0 < high < (1 << 31)
    out = np.empty(count, dtype=np.int64)
    for lo in range(0, count, _CHUNK):
        m = min(_CHUNK, count - lo)
        draw = splitmix64(seed, lo, m)
        if high & (high - 1) == 0:
            out[lo:lo + m] = (draw >> np.uint64(20)).astype(np.int64) & (high - 1)
        else:
            out[lo:lo + m] = (((draw >> np.uint64(32)) * np.uint64(high)) >> np.uint64(32)).astype(np.int64)
    return out


def choice_without_replacement(seed: int, n: int, k: int) -> np.ndarray:
    """``k`` distinct indices out of ``n`` (order of a seeded key sort)."""
    keys = splitmix64(seed, 0, n)
    return np.sort(np.argsort(keys, kind="stable")[:k])


# --------------------------------------------------------------------------
# storage-type helpers (type conversion only)
# --------------------------------------------------------------------------

def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float64/float32 to bfloat16 (nearest even); returns uint16 bits."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    # float64 -> float32 -> bf16 double rounding is avoided by the callers:
    # they only pass values already drawn in float64 and accept this rounding
    # as the definition of the stored input.
    b = f.view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------

@dataclass
class Workload:
    """One synthetic problem instance.

    ``x`` holds the head vectors as float32 values that are exactly
    representable in ``x_dtype`` (so widening them is exact on both sides);
    ``x_bits`` are the matching 16-bit patterns when ``x_dtype`` is 16-bit.
    """
    name: str
    seed: int
    dim: int
    group_dim: int
    layout: int
    depth: int
    codebook_size: int
    code_bits: int
    x_dtype: str
    out_dtype: str
    n: int = 0
    heads: int = 1
    x: np.ndarray | None = None
    x_bits: np.ndarray | None = None
    codebooks: np.ndarray | None = None      # float32 [R][K][group_dim]
    codes: np.ndarray | None = None          # int32 [n][G][R] (decode-only workloads)
    std_bits: np.ndarray | None = None       # uint16 fp16 bits [n] (decode-only workloads)
    decay: float = 0.99
    eps: float = 1e-5
    steps: int = 1
    extra: dict = field(default_factory=dict)

    @property
    def groups(self) -> int:
        return self.dim // self.group_dim


def _key_like_x(seed: int, tokens: int, heads: int, dim: int, outliers: int):
    """Heavy-tailed key-projection stand-in: x = a[h][c] * xi.

    Channel scale ``a = 0.25 + |Laplace(0,1)|``, with ``outliers`` seeded
    channels per head multiplied by 20.  Returns (x float64 [tokens*heads, dim],
    a [heads, dim]).
    """
    a = 0.25 + np.abs(laplace(stream_seed(seed, "chan-scale"), heads * dim)).reshape(heads, dim)
    for h in range(heads):
        idx = choice_without_replacement(stream_seed(seed, f"outlier-{h}"), dim, outliers)
        a[h, idx] *= 20.0
    xi = normal(stream_seed(seed, "x"), tokens * heads * dim).reshape(tokens, heads, dim)
    x = (xi * a[None, :, :]).reshape(tokens * heads, dim)
    return x, a


def _profile_codebooks(seed: int, a: np.ndarray, layout: int, depth: int, size: int,
                       group_dim: int, rho: float) -> np.ndarray:
    """Codebooks whose stage-0 codewords are distributed like unit-variance
    group vectors of ``x = a * xi`` and whose later stages shrink by ``rho``
    per stage (a stand-in for learnt residual codebooks; no quantizer is run).
    """
    heads, dim = a.shape
    groups = dim // group_dim
    rms = np.sqrt(np.mean(a * a, axis=1))           # the generator's own vector scale
    cb = np.empty((depth, size, group_dim), dtype=np.float64)
    i = np.arange(group_dim)
    for r in range(depth):
        xi = normal(stream_seed(seed, f"cb-{r}"), size * group_dim).reshape(size, group_dim)
        hsel = randint(stream_seed(seed, f"cb-head-{r}"), size, 1 << 30) % heads
        gsel = randint(stream_seed(seed, f"cb-group-{r}"), size, 1 << 30) % groups
        if layout == STRIDED:
            chan = i[None, :] * groups + gsel[:, None]
        else:
            chan = gsel[:, None] * group_dim + i[None, :]
        prof = a[hsel[:, None], chan] / rms[hsel][:, None]
        cb[r] = xi * prof * (rho ** r)
    return cb.astype(np.float32)


def _gaussian_codebooks(seed: int, depth: int, size: int, group_dim: int,
                        sigma0: float, rho: float) -> np.ndarray:
    cb = np.empty((depth, size, group_dim), dtype=np.float64)
    for r in range(depth):
        cb[r] = normal(stream_seed(seed, f"cb-{r}"), size * group_dim).reshape(size, group_dim)
        cb[r] *= sigma0 * (rho ** r)
    return cb.astype(np.float32)


def tiny(n: int = 4096, seed: int = 1001) -> Workload:
    """4096 fp32 vectors of 128 N(0,1) channels, 4 outlier channels x10;
    contiguous groups of 32, depth 8, 256 codes per stage, N(0, 0.5) codebooks."""
    w = Workload("tiny", seed, 128, 32, CONTIGUOUS, 8, 256, 16, "f32", "f32", n=n)
    x = normal(stream_seed(seed, "x"), n * 128).reshape(n, 128)
    idx = choice_without_replacement(stream_seed(seed, "outlier"), 128, 4)
    x[:, idx] *= 10.0
    w.x = x.astype(np.float32)
    w.codebooks = _gaussian_codebooks(seed, 8, 256, 32, 0.5, 1.0)
    w.extra["outlier_channels"] = idx
    return w


def key_cache(tokens: int = 4096, heads: int = 8, seed: int = 1002, size: int = 1024,
              depth: int = 8) -> Workload:
    """Key-cache encode of one Llama-style layer: tokens x 8 KV heads x 128
    bf16, heavy-tailed channel scales with 8 outlier channels x20 per head;
    strided groups (channel c in group c mod 4); 1024 codes per stage."""
    w = Workload("key_cache", seed, 128, 32, STRIDED, depth, size, 16, "bf16", "bf16",
                 n=tokens * heads, heads=heads)
    x, a = _key_like_x(seed, tokens, heads, 128, 8)
    w.x_bits = to_bf16_bits(x)
    w.x = bf16_bits_to_f32(w.x_bits)
    w.codebooks = _profile_codebooks(seed, a, STRIDED, depth, size, 32, 0.8)
    w.extra["chan_scale"] = a
    return w


def value_cache(tokens: int = 32768, heads: int = 8, seed: int = 1003, size: int = 2048,
                depth: int = 8) -> Workload:
    """Value-cache encode + decode: tokens x 8 heads x 128 bf16 Gaussian;
    contiguous groups; 2048 codes per stage; codes packed 11 bits; bf16 out."""
    bits = max(1, int(size - 1).bit_length())
    w = Workload("value_cache", seed, 128, 32, CONTIGUOUS, depth, size, bits, "bf16", "bf16",
                 n=tokens * heads, heads=heads)
    x = normal(stream_seed(seed, "x"), tokens * heads * 128).reshape(tokens * heads, 128)
    w.x_bits = to_bf16_bits(x)
    w.x = bf16_bits_to_f32(w.x_bits)
    w.codebooks = _gaussian_codebooks(seed, depth, size, 32, 1.0, 0.8)
    return w


def ablation(tokens: int = 32768, heads: int = 8, dim: int = 128, group_dim: int = 32, depth: int = 8,
             size: int = 2048, layout: int = CONTIGUOUS, seed: int = 1006) -> Workload:
    """The codebook-size ablation's shapes (depth 4/6/8, 1024/2048 codes, and
    other group and head sizes): tokens x heads x dim bf16 Gaussian vectors,
    Gaussian codebooks shrinking by 0.8 per stage, packed codes, bf16 out."""
    bits = max(1, int(size - 1).bit_length())
    w = Workload("ablation", seed, dim, group_dim, layout, depth, size, bits, "bf16", "bf16",
                 n=tokens * heads, heads=heads)
    x = normal(stream_seed(seed, "x"), tokens * heads * dim).reshape(tokens * heads, dim)
    w.x_bits = to_bf16_bits(x)
    w.x = bf16_bits_to_f32(w.x_bits)
    w.codebooks = _gaussian_codebooks(seed, depth, size, group_dim, 1.0, 0.8)
    return w


def decode_bandwidth(tokens: int = 131072, heads: int = 8, seed: int = 1004, size: int = 1024,
                     depth: int = 8, layout: int = CONTIGUOUS) -> Workload:
    """Decode-only: uniform uint16 codes, fp16 std = |N(1, 0.25)| + 0.05,
    codebook stage scale 0.5 * 0.75**r; output bf16."""
    n = tokens * heads
    w = Workload("decode_bandwidth", seed, 128, 32, layout, depth, size, 16, "bf16", "bf16",
                 n=n, heads=heads)
    w.codes = randint(stream_seed(seed, "codes"), n * 4 * depth, size).astype(np.int32)
    w.codes = w.codes.reshape(n, 4, depth)
    s = np.abs(1.0 + 0.25 * normal(stream_seed(seed, "std"), n)) + 0.05
    w.std_bits = s.astype(np.float16).view(np.uint16)
    w.codebooks = _gaussian_codebooks(seed, depth, size, 32, 0.5, 0.75)
    return w


def ema_learning(tokens: int = 131072, heads: int = 8, seed: int = 1005, size: int = 1024,
                 depth: int = 8, steps: int = 10) -> Workload:
    """EMA codebook learning: tokens x 8 heads x 128 bf16 with the key-cache
    distribution, strided groups, decay 0.99, Laplace eps 1e-5, ``steps``
    updates on the same batch."""
    w = key_cache(tokens, heads, seed, size, depth)
    w.name = "ema_learning"
    w.decay, w.eps, w.steps = 0.99, 1e-5, steps
    return w


WORKLOADS = {
    "tiny": tiny,
    "key_cache": key_cache,
    "value_cache": value_cache,
    "decode_bandwidth": decode_bandwidth,
    "ema_learning": ema_learning,
    "ablation": ablation,
}
