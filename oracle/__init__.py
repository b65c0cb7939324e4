"""CPU oracle for the residual-VQ KV-cache compressor -- TEST INFRASTRUCTURE.

Thin numpy wrappers over ``rvq_oracle.c`` (plain C, double precision, the
paper's definitions written out: Section 2.2, Algorithm 1, Sections 3.1-3.2,
and the EMA codebook update of Section 3).  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the CUDA library
never does, and this package never imports the CUDA library.

Parity status of each function against something other than itself
(``tests/test_oracle_*.py``):
  encode / check_codes  pinned: brute force, nearest-neighbour special case,
                        prefix property, residual identity, scale invariance,
                        grouping permutation, exact-reconstruction codebooks
  decode                pinned: residual identity, hand-computed example
  f16 / rounding        pinned: numpy's float16, exact rational arithmetic
  pack / unpack         pinned: Python big-integer bit streams, Section 3.2's
                        5.5x compression arithmetic
  ema_stats/normalise   pinned as arithmetic: hand-computed example, k-means
                        (decay 0) and identity (decay 1) special cases,
                        conservation invariants; the FORM of the smoothing and
                        the population (ddof=0) standard deviation are this
                        oracle's reading of a paper that states neither:
                        parity unpinned for those two choices.
  lloyd / kmeans_init   pinned: scipy's kmeans2 from the same start, closed-form
                        cluster means, empty-cluster and zero-iteration cases,
                        and the C encoder reproducing the assignments; WHICH
                        k-means the paper runs (start, iteration count, empty
                        clusters) is not stated: parity unpinned for those.
  learn_step            encode followed by ema_update (both pinned above)
  rope / decode_rope    pinned: the transformers library's Llama rotary helper
                        (half-split pairing), complex multiplication (adjacent
                        pairing), identity at position 0, norm preservation,
                        additivity in the position, the relative-position
                        property of the inner product
  attention_decode      pinned: the library's scaled dot-product attention in
                        float64 (grouped heads spelled out), a pure-Python brute
                        force, one-token / identical-keys / dominant-token /
                        zero-scale special cases, token permutation, kv-head
                        isolation; the paper prints no formula for this step
                        (it is the attention of the models it quantizes)
  check_codes           near-tie verdicts pinned on hand-worked stages
                        (tests/golden/check_codes_near_tie.txt)
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rvq_oracle.c")
_LIB = os.path.join(_HERE, "librvq_oracle.so")

F32, BF16, F16 = 0, 1, 2
CONTIGUOUS, STRIDED = 0, 1
NEAR_TIE = 1e-5


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over head vectors)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None
_dp = ctypes.POINTER(ctypes.c_double)


def _l():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.rvq_oracle_encode.restype = ctypes.c_int64
        _lib.rvq_oracle_check_codes.restype = ctypes.c_int64
        _lib.rvq_oracle_packed_bytes.restype = ctypes.c_int64
        _lib.rvq_oracle_round_scalar.restype = ctypes.c_double
        _lib.rvq_oracle_round_scalar.argtypes = [ctypes.c_double, ctypes.c_int]
        _lib.rvq_oracle_f64_to_f16_bits.restype = ctypes.c_uint16
        _lib.rvq_oracle_f64_to_f16_bits.argtypes = [ctypes.c_double]
        _lib.rvq_oracle_f16_bits_to_f64.restype = ctypes.c_double
        _lib.rvq_oracle_f16_bits_to_f64.argtypes = [ctypes.c_uint16]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def threads() -> int:
    return int(_l().rvq_oracle_threads())


def encode(x, codebooks, group_dim=32, layout=CONTIGUOUS, ddof=0, want_residual=False):
    """Section 2.2 + Algorithm 1.  Returns a dict with ``codes`` int32
    [n][G][R], ``std_bits`` uint16 [n], ``std`` float64 [n], ``d1``/``d2``
    best / second-best squared distance per stage, ``near_tie`` (d2-d1 <
    1e-5*d2), ``degenerate`` count and optionally ``residual`` [n][G][gd]."""
    x = _f64(x)
    cb = _f64(codebooks)
    n, dim = x.shape
    R, K, gd = cb.shape
    assert gd == group_dim and dim % gd == 0 and gd <= 1024
    G = dim // gd
    codes = np.empty((n, G, R), np.int32)
    std16 = np.empty(n, np.uint16)
    std = np.empty(n, np.float64)
    d1 = np.empty((n, G, R), np.float64)
    d2 = np.empty((n, G, R), np.float64)
    resid = np.empty((n, G, gd), np.float64) if want_residual else None
    bad = _l().rvq_oracle_encode(_p(x), ctypes.c_int64(n), dim, gd, layout, R, K, _p(cb), ddof,
                                 _p(codes), _p(std16), _p(std), _p(d1), _p(d2), _p(resid))
    with np.errstate(invalid="ignore"):
        near = (d2 - d1) < NEAR_TIE * d2
    out = dict(codes=codes, std_bits=std16, std=std, d1=d1, d2=d2, near_tie=near, degenerate=int(bad))
    if want_residual:
        out["residual"] = resid
    return out


def decode(codes, std_bits, codebooks, dim=128, layout=CONTIGUOUS, out_dtype=None):
    """Section 2.2 last sentence.  Returns float64 [n][dim]; with ``out_dtype``
    the values are rounded once (nearest even) to that type."""
    cb = _f64(codebooks)
    R, K, gd = cb.shape
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    n = codes.shape[0]
    std_bits = np.ascontiguousarray(std_bits, dtype=np.uint16)
    out = np.empty((n, dim), np.float64)
    _l().rvq_oracle_decode(_p(codes), _p(std_bits), ctypes.c_int64(n), dim, gd, layout, R, K,
                           _p(cb), _p(out))
    return out if out_dtype is None else round_to(out, out_dtype)


def round_to(a, dtype):
    a = _f64(a)
    out = np.empty_like(a)
    _l().rvq_oracle_round(_p(a), ctypes.c_int64(a.size), dtype, _p(out))
    return out


def f16_bits(a):
    a = _f64(np.atleast_1d(a))
    return np.array([_l().rvq_oracle_f64_to_f16_bits(float(v)) for v in a.ravel()],
                    dtype=np.uint16).reshape(a.shape)


def f16_value(bits):
    bits = np.atleast_1d(np.asarray(bits, dtype=np.uint16))
    return np.array([_l().rvq_oracle_f16_bits_to_f64(int(b)) for b in bits.ravel()],
                    dtype=np.float64).reshape(bits.shape)


def ema_stats(x, codes, codebooks, layout=CONTIGUOUS, ddof=0):
    """Per-stage, per-code counts [R][K] and sums [R][K][gd] of the stage inputs."""
    x = _f64(x)
    cb = _f64(codebooks)
    n, dim = x.shape
    R, K, gd = cb.shape
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    cnt = np.empty((R, K), np.float64)
    sm = np.empty((R, K, gd), np.float64)
    _l().rvq_oracle_ema_stats(_p(x), ctypes.c_int64(n), dim, gd, layout, R, K, _p(cb), ddof,
                              _p(codes), _p(cnt), _p(sm))
    return cnt, sm


def ema_normalise(cnt, sm, ema_count, ema_sum, decay, eps):
    """Decayed, Laplace-smoothed update.  Returns new (ema_count, ema_sum, codebooks)."""
    cnt = _f64(cnt)
    sm = _f64(sm)
    R, K, gd = sm.shape
    n2 = _f64(ema_count).copy()
    m2 = _f64(ema_sum).copy()
    cb = np.empty((R, K, gd), np.float64)
    _l().rvq_oracle_ema_normalise(_p(cnt), _p(sm), R, K, gd, ctypes.c_double(decay),
                                  ctypes.c_double(eps), _p(n2), _p(m2), _p(cb))
    return n2, m2, cb


def ema_update(x, codes, codebooks, ema_count, ema_sum, decay, eps, layout=CONTIGUOUS, ddof=0):
    cnt, sm = ema_stats(x, codes, codebooks, layout, ddof)
    n2, m2, cb = ema_normalise(cnt, sm, ema_count, ema_sum, decay, eps)
    return dict(count=cnt, sum=sm, ema_count=n2, ema_sum=m2, codebooks=cb)


ROPE_HALVES, ROPE_ADJACENT = 0, 1


def rope(x, positions, base=10000.0, style=ROPE_HALVES):
    """Rotary position embedding of the rows of ``x`` [n][d] at integer
    ``positions`` [n]: pair k of a row is rotated by the angle
    positions * base**(-2k/d).  Pairs are channels (k, k + d/2)
    (ROPE_HALVES, the Llama checkpoints' convention) or (2k, 2k + 1)
    (ROPE_ADJACENT, RoFormer's).  Section 3: keys are quantized before this
    rotation, so a decoded key gets it afterwards."""
    x = _f64(x)
    n, d = x.shape
    h = d // 2
    ang = np.asarray(positions, dtype=np.float64)[:, None] * base ** (-2.0 * np.arange(h) / d)[None, :]
    c, s_ = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    if style == ROPE_HALVES:
        a, b = x[:, :h], x[:, h:]
        out[:, :h], out[:, h:] = a * c - b * s_, b * c + a * s_
    else:
        a, b = x[:, 0::2], x[:, 1::2]
        out[:, 0::2], out[:, 1::2] = a * c - b * s_, b * c + a * s_
    return out


def decode_rope(codes, std_bits, codebooks, positions, base=10000.0, style=ROPE_HALVES, dim=128,
                layout=CONTIGUOUS, out_dtype=None):
    """Decode followed by the rotary embedding, rounded once at the end."""
    out = rope(decode(codes, std_bits, codebooks, dim, layout), positions, base, style)
    return out if out_dtype is None else round_to(out, out_dtype)


def attention_decode(q, codes_k, std_bits_k, codes_v, std_bits_v, codebooks_k, codebooks_v, kv_heads, scale,
                     positions=None, base=10000.0, style=ROPE_HALVES, dim=128, layout_k=CONTIGUOUS,
                     layout_v=CONTIGUOUS):
    """One new token attending over a compressed cache (Section 1: the cache is what
    long-context decoding loads; Section 3: keys are stored before the rotary
    embedding, so they are rotated as they are read; Section 2.2: a cached vector is
    the sum of its codewords times its deviation).  Rows of the cache are
    [token][kv head]; query head i reads kv head i // (query heads / kv heads).  For
    every query head: scores s_t = scale * q . k_t over the tokens, weights
    softmax(s), output sum_t w_t v_t.  ``positions`` None leaves the keys unrotated.
    The paper gives no formula for this step: it is the usual scaled dot-product
    attention of the models it quantizes.  q [Hq][dim]; returns float64 [Hq][dim]."""
    q = _f64(q)
    n = len(codes_k)
    T = n // kv_heads
    k = decode(codes_k, std_bits_k, codebooks_k, dim, layout_k)
    if positions is not None:
        k = rope(k, np.repeat(np.asarray(positions), kv_heads), base, style)
    v = decode(codes_v, std_bits_v, codebooks_v, dim, layout_v)
    k, v = k.reshape(T, kv_heads, dim), v.reshape(T, kv_heads, dim)
    per = q.shape[0] // kv_heads
    out = np.zeros((q.shape[0], dim))
    for i in range(q.shape[0]):
        h = i // per
        s = scale * (k[:, h, :] @ q[i])
        w = np.exp(s - s.max())
        w /= w.sum()
        out[i] = w @ v[:, h, :]
    return out


def learn_step(x, codebooks, ema_count, ema_sum, decay, eps, group_dim=32, layout=CONTIGUOUS, ddof=0):
    """One codebook-learning step (Section 3): the batch is encoded with the
    current codebooks and these assignments feed the EMA update."""
    enc = encode(x, codebooks, group_dim, layout, ddof)
    out = ema_update(x, enc["codes"], codebooks, ema_count, ema_sum, decay, eps, layout, ddof)
    out["codes"], out["std_bits"] = enc["codes"], enc["std_bits"]
    return out


def scaled_groups(x, group_dim=32, layout=CONTIGUOUS, ddof=0):
    """Section 2.2 / 3.1: every head vector divided by its standard deviation,
    then cut into groups; returns the group rows [n * G][group_dim] (row v*G+g).
    A vector without a usable deviation gives zero rows."""
    x = _f64(x)
    n, d = x.shape
    G = d // group_dim
    mu = x.sum(axis=1, keepdims=True) / d
    s = np.sqrt(((x - mu) ** 2).sum(axis=1, keepdims=True) / (d - ddof))
    ok = np.isfinite(s) & (s > 0)
    z = np.where(ok, x / np.where(ok, s, 1.0), 0.0)
    if layout == CONTIGUOUS:                      # element i of group g is channel g*gd + i
        zg = z.reshape(n, G, group_dim)
    else:                                         # ... or channel i*G + g
        zg = z.reshape(n, group_dim, G).transpose(0, 2, 1)
    return np.ascontiguousarray(zg).reshape(n * G, group_dim)


def nearest(z, c, block=512):
    """Index of the nearest row of ``c`` (squared Euclidean distance, direct
    form, lowest index on ties) for every row of ``z``."""
    z, c = _f64(z), _f64(c)
    out = np.empty(len(z), np.int64)
    for lo in range(0, len(z), block):
        d = ((z[lo:lo + block, None, :] - c[None, :, :]) ** 2).sum(axis=2)
        out[lo:lo + block] = d.argmin(axis=1)
    return out


def lloyd(z, c0, iters):
    """``iters`` iterations of Lloyd's k-means on the rows of ``z`` from the
    centroids ``c0``: assign every row to its nearest centroid, move every
    centroid to the mean of its rows; a centroid without rows stays."""
    z, c = _f64(z), _f64(c0).copy()
    K = len(c)
    for _ in range(iters):
        a = nearest(z, c)
        cnt = np.bincount(a, minlength=K)
        sm = np.zeros_like(c)
        np.add.at(sm, a, z)
        filled = cnt > 0
        c[filled] = sm[filled] / cnt[filled, None]
    return c


def kmeans_init(x, seed_rows, iters, group_dim=32, layout=CONTIGUOUS, ddof=0):
    """Codebook initialisation (Section 3: every codebook starts from k-means):
    stage r runs Lloyd's iterations on the stage-r inputs of the batch (the
    scaled group rows minus the chosen codewords of the earlier stages), from
    the centroids ``z_r[seed_rows[r]]``.  ``seed_rows`` is int [R][K] with group
    row numbers v*G+g.  Returns float64 codebooks [R][K][group_dim]."""
    z = scaled_groups(x, group_dim, layout, ddof)
    seed_rows = np.asarray(seed_rows, dtype=np.int64)
    cbs = []
    for r in range(seed_rows.shape[0]):
        c = lloyd(z, z[seed_rows[r]], iters)
        z = z - c[nearest(z, c)]
        cbs.append(c)
    return np.stack(cbs)


def code_bits(K: int) -> int:
    return max(1, int(K - 1).bit_length())


def packed_bytes(per_vector: int, bits: int) -> int:
    return int(_l().rvq_oracle_packed_bytes(per_vector, bits))


def pack(codes, bits):
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    n = codes.shape[0]
    per = int(np.prod(codes.shape[1:]))
    out = np.empty((n, packed_bytes(per, bits)), np.uint8)
    _l().rvq_oracle_pack(_p(codes), ctypes.c_int64(n), per, bits, _p(out))
    return out


def unpack(packed, shape, bits):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    n = shape[0]
    per = int(np.prod(shape[1:]))
    codes = np.empty(shape, np.int32)
    _l().rvq_oracle_unpack(_p(packed), ctypes.c_int64(n), per, bits, _p(codes))
    return codes


def check_codes(x, codes, codebooks, layout=CONTIGUOUS, ddof=0, tol=NEAR_TIE, want_gap=False):
    """Judge ``codes`` stage by stage, each stage conditioned on the given
    codes of the earlier stages.  Returns (status uint8 [n][G][R], wrong count
    [, gap]); status 0 exact argmin, 1 near tie, 2 mismatch, 3 out of range."""
    x = _f64(x)
    cb = _f64(codebooks)
    n, dim = x.shape
    R, K, gd = cb.shape
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    status = np.empty(codes.shape, np.uint8)
    gap = np.empty(codes.shape, np.float64) if want_gap else None
    wrong = _l().rvq_oracle_check_codes(_p(x), ctypes.c_int64(n), dim, gd, layout, R, K, _p(cb),
                                        ddof, _p(codes), ctypes.c_double(tol), _p(status), _p(gap))
    return (status, int(wrong), gap) if want_gap else (status, int(wrong))
