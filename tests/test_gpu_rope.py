"""GPU parity of rvq_decode_rope (decode fused with the rotary position embedding) and
rvq_rope_table against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_15704_b200 as rvq
import rvq_synth
from helpers import DT, HALF_ULP, RECON_TOL, codes_to_device

pytestmark = pytest.mark.gpu

BASE = 500000.0


def rope_table(dim, positions):
    t = torch.empty(positions, dim // 2, 2, device="cuda")
    rvq.rvq_rope_table(dim, BASE, positions, t)
    torch.cuda.synchronize()
    return t


def test_rope_table_matches_double_precision():
    t = rope_table(128, 131072).cpu().numpy().astype(np.float64)
    p = np.arange(131072, dtype=np.float64)[:, None]
    ang = p * BASE ** (-2.0 * np.arange(64) / 128)[None, :]
    assert np.abs(t[:, :, 0] - np.cos(ang)).max() <= 1e-7 and np.abs(t[:, :, 1] - np.sin(ang)).max() <= 1e-7


def run_case(dim, gd, R, K, bits, layout, dtype, pairing, tokens=333, heads=8, max_pos=100000, with_prepared=True,
             std_scale=1.0, outlier_every=0):
    g = np.random.default_rng(dim + K + R + layout * 7 + pairing)
    n, G = tokens * heads, dim // gd
    codes = g.integers(0, K, size=(n, G, R)).astype(np.int32)
    std = std_scale * (np.abs(1.0 + 0.25 * g.normal(size=n)) + 0.05)
    if outlier_every:
        std[::outlier_every] *= 50.0                                     # single rows beyond the chosen table's reach
    std_bits = std.astype(np.float16).view(np.uint16)
    cb = np.stack([g.normal(scale=0.5 * 0.75 ** r, size=(K, gd)) for r in range(R)]).astype(np.float32)
    pos = g.integers(0, max_pos, size=tokens).astype(np.int32)
    pos[:3] = [0, max_pos - 1, 1]
    cfg = rvq.make_config(dim, gd, layout, R, K, bits, DT[dtype], 0)
    table = rope_table(dim, max_pos)
    out = torch.full((n, dim + 8), 7.0, dtype=rvq.TORCH_DTYPE[cfg.x_dtype], device="cuda")
    status = rvq.new_status()
    b = rvq.alloc_buffers(cfg, n, cb)
    rvq.rvq_decode_rope(cfg, codes_to_device(cfg, codes), torch.from_numpy(std_bits.view(np.int16)).cuda(), n,
                        b.codebooks, b.prepared if with_prepared else None, torch.from_numpy(pos).cuda(), heads, table,
                        max_pos, pairing, out, dim + 8, status)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(got[:, dim:] == 7.0)                                   # row padding untouched
    ref = oracle.decode_rope(codes, std_bits, cb, np.repeat(pos, heads), BASE, pairing, dim, layout)
    err = np.abs(got[:, :dim] - ref)
    assert np.all(err <= RECON_TOL + HALF_ULP[cfg.x_dtype] * np.abs(ref) * 1.01), f"off by {err.max():.3e}"
    # position 0 leaves the decoded vector as it is
    plain = oracle.decode(codes[:heads], std_bits[:heads], cb, dim, layout)
    assert np.all(np.abs(got[:heads, :dim] - plain) <= RECON_TOL + HALF_ULP[cfg.x_dtype] * np.abs(plain) * 1.01)
    assert rvq.read_status(status)["bad_codes"] == 0
    return float(err.max())


@pytest.mark.parametrize("layout", [rvq_synth.CONTIGUOUS, rvq_synth.STRIDED])
@pytest.mark.parametrize("pairing", [rvq.ROPE_HALVES, rvq.ROPE_ADJACENT])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_decode_rope_table_path(layout, pairing, dtype):
    """dim 128, 1024 codes: float32 shared-memory tables; all four pairings of layout and convention."""
    err = run_case(128, 32, 8, 1024, 16, layout, dtype, pairing)
    print(f"rope layout {layout} pairing {pairing} {dtype}: max-abs {err:.2e}")


@pytest.mark.parametrize("dim,gd,R,K,bits,layout,dtype,pairing", [
    (128, 32, 8, 2048, 11, rvq_synth.STRIDED, "bf16", rvq.ROPE_HALVES),       # the paper's default key quantizer
    (128, 32, 6, 1024, 10, rvq_synth.CONTIGUOUS, "f16", rvq.ROPE_ADJACENT),   # packed codes on the table path
    (256, 32, 4, 512, 16, rvq_synth.STRIDED, "bf16", rvq.ROPE_HALVES),
    (64, 16, 8, 64, 6, rvq_synth.CONTIGUOUS, "f32", rvq.ROPE_ADJACENT),
    (256, 32, 8, 1024, 10, rvq_synth.CONTIGUOUS, "bf16", rvq.ROPE_HALVES),    # head_dim 256 on the table kernels
    (256, 32, 8, 1024, 16, rvq_synth.CONTIGUOUS, "f16", rvq.ROPE_ADJACENT),
    (256, 32, 8, 2048, 11, rvq_synth.STRIDED, "bf16", rvq.ROPE_ADJACENT),
    (256, 32, 8, 2048, 11, rvq_synth.STRIDED, "f32", rvq.ROPE_HALVES),
    (64, 32, 8, 512, 9, rvq_synth.STRIDED, "bf16", rvq.ROPE_HALVES),          # two groups
    (64, 32, 8, 512, 9, rvq_synth.CONTIGUOUS, "bf16", rvq.ROPE_HALVES),
    (32, 32, 4, 256, 8, rvq_synth.CONTIGUOUS, "bf16", rvq.ROPE_HALVES),       # one group: gather kernel
])
def test_decode_rope_other_shapes(dim, gd, R, K, bits, layout, dtype, pairing):
    run_case(dim, gd, R, K, bits, layout, dtype, pairing, tokens=97, heads=4, max_pos=5000)
    run_case(dim, gd, R, K, bits, layout, dtype, pairing, tokens=97, heads=4, max_pos=5000, with_prepared=False)


@pytest.mark.parametrize("layout", [rvq_synth.CONTIGUOUS, rvq_synth.STRIDED])
@pytest.mark.parametrize("pairing", [rvq.ROPE_HALVES, rvq.ROPE_ADJACENT])
def test_decode_rope_level_tables(layout, pairing):
    """2048 and 3072 codes with 16-bit outputs: level tables; large deviations take float32 sums."""
    run_case(128, 32, 8, 2048, 11, layout, "bf16", pairing, tokens=211)
    run_case(128, 32, 8, 3072, 12, layout, "f16", pairing, tokens=57)
    run_case(128, 32, 8, 2048, 16, layout, "bf16", pairing, tokens=57, std_scale=40.0)
    # float32 tables with 2-channel slices: float32 outputs, and 16-bit outputs without a prepared block
    run_case(128, 32, 8, 2048, 11, layout, "f32", pairing, tokens=57)
    run_case(128, 32, 8, 3584, 12, layout, "bf16", pairing, tokens=57, with_prepared=False)


@pytest.mark.parametrize("layout", [rvq_synth.CONTIGUOUS, rvq_synth.STRIDED])
@pytest.mark.parametrize("pairing", [rvq.ROPE_HALVES, rvq.ROPE_ADJACENT])
def test_decode_rope_quoted_shapes_take_every_kind_of_table(layout, pairing):
    """dim 128, depth 8, up to 1536 codes, 16-bit outputs and a prepared block: one launch that picks the
    summed levels (small deviations), the per-stage levels (moderate), or the float32 tables (large); uint16
    and packed codes; a mixed batch sends single rows down the exact route."""
    for std_scale in (0.3, 1.0, 3.0, 40.0):
        run_case(128, 32, 8, 1024, 16, layout, "bf16", pairing, tokens=333, std_scale=std_scale)
    run_case(128, 32, 8, 1024, 10, layout, "f16", pairing, tokens=131, std_scale=0.3)
    run_case(128, 32, 8, 1536, 11, layout, "bf16", pairing, tokens=131, std_scale=1.0)
    run_case(128, 32, 8, 1000, 10, layout, "bf16", pairing, tokens=57, std_scale=2.0)
    run_case(128, 32, 8, 1024, 16, layout, "f16", pairing, tokens=131, std_scale=1.0, outlier_every=11)


def test_decode_rope_clamps_positions_and_rejects_bad_arguments():
    import ctypes
    cfg = rvq.make_config(128, 32, 0, 8, 1024, 16, rvq.BF16, 0)
    c = ctypes.byref(cfg)
    assert rvq.lib.rvq_decode_rope(c, 256, 256, 4, 256, None, 256, 0, 256, 10, 0, 256, 128, None, None) == -1   # 0 vectors per position
    assert rvq.lib.rvq_decode_rope(c, 256, 256, 4, 256, None, 256, 8, 256, 10, 2, 256, 128, None, None) == -1   # unknown pairing
    assert rvq.lib.rvq_decode_rope(c, 256, 256, 4, 256, None, None, 8, 256, 10, 0, 256, 128, None, None) == -1
    assert rvq.lib.rvq_decode_rope(c, 256, 256, 4, 256, 272, 256, 8, 256, 10, 0, 256, 128, None, None) == -2    # prepared % 256
    assert rvq.lib.rvq_rope_table(127, 10000.0, 4, 256, None) == -1
    # a position past the table reads its last row
    w = rvq_synth.decode_bandwidth(tokens=4)
    table = rope_table(128, 50)
    outs = []
    for p in (49, 4000):
        out = torch.empty(w.n, 128, dtype=torch.bfloat16, device="cuda")
        pos = torch.full((4,), p, dtype=torch.int32, device="cuda")
        rvq.rvq_decode_rope(cfg, codes_to_device(cfg, w.codes), torch.from_numpy(w.std_bits.view(np.int16)).cuda(),
                            w.n, torch.from_numpy(w.codebooks).cuda(), None, pos, 8, table, 50, rvq.ROPE_HALVES, out, 128)
        torch.cuda.synchronize()
        outs.append(out.cpu())
    assert torch.equal(outs[0], outs[1])
