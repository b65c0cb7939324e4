"""CPU-side checks of the C boundary: the library loads, exports every symbol the
header declares, and rejects bad arguments on the host before any launch."""
import ctypes
import os
import re

import pytest

import paper_2410_15704_b200 as rvq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for header in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(rvq_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported():
    names = declared_symbols()
    assert {"rvq_encode", "rvq_decode", "rvq_ema_update"} <= set(names)
    for name in names:
        assert hasattr(rvq.lib, name), name
    assert set(names) == set(rvq.EXPORTS)


def test_sizes_and_strings():
    cfg = rvq.make_config(128, 32, rvq.CONTIGUOUS, 8, 2048, 11, rvq.BF16)
    assert rvq.rvq_code_bytes(cfg) == 44                 # Section 3.2: 32 indices of 11 bits
    assert rvq.rvq_code_bytes(rvq.make_config(code_bits=16)) == 64
    assert rvq.rvq_code_bytes(rvq.make_config(codebook_size=300, code_bits=9)) == 36
    assert rvq.rvq_prepared_bytes(cfg) >= 256 and rvq.rvq_prepared_bytes(cfg) % 256 == 0
    assert rvq.rvq_workspace_bytes(cfg, 1000) >= 8 * 2048 * 33 * 4
    assert rvq.rvq_status_string(0) == "ok" and "aligned" in rvq.rvq_status_string(-2)
    assert rvq.rvq_version() >= 1000


@pytest.mark.parametrize("kw", [dict(dim=100), dict(group_dim=12), dict(depth=0), dict(depth=17),
                                dict(codebook_size=1), dict(codebook_size=70000), dict(code_bits=12),
                                dict(layout=3), dict(x_dtype=5), dict(std_ddof=2)])
def test_bad_configs_are_rejected(kw):
    cfg = rvq.make_config(**kw)
    assert rvq.rvq_code_bytes(cfg) == 0 and rvq.rvq_prepared_bytes(cfg) == 0
    rc = rvq.lib.rvq_encode(ctypes.byref(cfg), 256, 1, 128, 256, 256, 256, 256, None, None, 0, None, None)
    assert rc in (-1, -3)


def test_bad_pointers_are_rejected_before_launch():
    cfg = rvq.make_config(code_bits=11)
    c = ctypes.byref(cfg)
    assert rvq.lib.rvq_encode(c, None, 4, 128, 256, 256, 256, 256, None, None, 0, None, None) == -1
    assert rvq.lib.rvq_encode(c, 256, -1, 128, 256, 256, 256, 256, None, None, 0, None, None) == -1
    assert rvq.lib.rvq_encode(c, 256, 4, 64, 256, 256, 256, 256, None, None, 0, None, None) == -1      # stride < dim
    assert rvq.lib.rvq_encode(c, 260, 4, 128, 256, 256, 256, 256, None, None, 0, None, None) == -2     # x misaligned
    assert rvq.lib.rvq_encode(c, 256, 4, 132, 256, 256, 256, 256, None, None, 0, None, None) == -2     # stride bytes % 16
    assert rvq.lib.rvq_encode(c, 256, 4, 128, 256, 272, 256, 256, None, None, 0, None, None) == -2     # prepared % 256
    assert rvq.lib.rvq_decode(c, 256, 256, 4, 256, 256, None, 128, None, None) == -1
    assert rvq.lib.rvq_decode(c, 256, 256, 4, 256, 256, 264, 128, None, None) == -2
    assert rvq.lib.rvq_ema_update(c, 256, 4, 128, 256, 256, 256, 256, None, 0.99, 1e-5, 256, 16, None, None) == -4
    assert rvq.lib.rvq_ema_update(c, 256, 4, 128, 256, 256, 256, 256, None, 1.5, 1e-5, 256, 1 << 30, None, None) == -1
    # learning step and k-means initialisation
    assert rvq.lib.rvq_learn_step(c, 256, 4, 128, 256, 256, 256, 256, 256, 256, None, 0.99, 1e-5, 256, 16, None, None) == -4
    assert rvq.lib.rvq_learn_step(c, 256, 4, 128, 256, 256, None, 256, 256, 256, None, 0.99, 1e-5, 256, 1 << 30, None, None) == -1
    big = rvq.rvq_kmeans_workspace_bytes(cfg, 1000)
    assert big >= 1000 * 128 * 4 and big % 256 == 0
    assert rvq.lib.rvq_kmeans_init(c, 256, 4, 128, 256, 3, 256, 256, 256, 16, None, None) == -4       # workspace too small
    assert rvq.lib.rvq_kmeans_init(c, 256, 4, 128, None, 3, 256, 256, 256, 1 << 40, None, None) == -1  # no seed rows
    assert rvq.lib.rvq_kmeans_init(c, 256, 4, 128, 256, -1, 256, 256, 256, 1 << 40, None, None) == -1
    odd = rvq.make_config(128, 16, rvq.CONTIGUOUS, 8, 256, 8, rvq.BF16)                                # group_dim 16
    assert rvq.rvq_kmeans_workspace_bytes(odd, 1000) == 0
    assert rvq.lib.rvq_kmeans_init(ctypes.byref(odd), 256, 4, 128, 256, 3, 256, 256, 256, 1 << 40, None, None) == -3
    assert rvq.lib.rvq_ema_update(c, 256, 4, 128, 256, None, 256, 256, None, 0.9, 1e-5, 256, 1 << 30, None, None) == -1
    assert rvq.lib.rvq_prepare_codebooks(c, None, 256, None) == -1
