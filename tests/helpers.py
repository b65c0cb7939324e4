"""Shared helpers of the GPU parity tests: move a workload to the device, call
the C ABI through the binding, and compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2410_15704_b200 as rvq

DT = {"f32": rvq.F32, "bf16": rvq.BF16, "f16": rvq.F16}
HALF_ULP = {rvq.F32: 0.0, rvq.BF16: 2.0 ** -8, rvq.F16: 2.0 ** -11}
RECON_TOL = 1e-3      # max-abs bound on float32-accumulated reconstructions and EMA codebooks


def config_of(w, code_bits=None, x_dtype=None, ddof=0):
    return rvq.make_config(w.dim, w.group_dim, w.layout, w.depth, w.codebook_size,
                           w.code_bits if code_bits is None else code_bits,
                           DT[w.x_dtype] if x_dtype is None else x_dtype, ddof)


def x_to_device(x: np.ndarray, dtype: int, row_stride=None) -> torch.Tensor:
    """Exact conversion (the values are representable) of float32 rows to the
    device in ``dtype``; with ``row_stride`` the rows are spaced out."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(rvq.TORCH_DTYPE[dtype])
    if row_stride is not None and row_stride != x.shape[1]:
        buf = torch.full((x.shape[0], row_stride), 7.0, dtype=t.dtype)
        buf[:, :x.shape[1]] = t
        t = buf
    return t.cuda()


def codes_to_numpy(cfg, codes_dev: torch.Tensor, n: int) -> np.ndarray:
    """Device code bytes -> int32 [n][G][R] (unpacking is a storage conversion)."""
    G, R = cfg.dim // cfg.group_dim, cfg.depth
    raw = codes_dev.cpu().numpy()[: n * rvq.rvq_code_bytes(cfg)]
    if cfg.code_bits == 16:
        return raw.view(np.uint16).reshape(n, G, R).astype(np.int32)
    return oracle.unpack(raw.reshape(n, -1), (n, G, R), cfg.code_bits)


def codes_to_device(cfg, codes: np.ndarray) -> torch.Tensor:
    if cfg.code_bits == 16:
        return torch.from_numpy(codes.astype(np.uint16).view(np.int16).reshape(-1)).cuda().view(torch.uint8)
    return torch.from_numpy(oracle.pack(codes, cfg.code_bits).reshape(-1)).cuda()


def gpu_encode(cfg, x_dev, n, codebooks, row_stride=None):
    b = rvq.alloc_buffers(cfg, n, codebooks)
    rvq.rvq_encode(cfg, x_dev, n, row_stride or cfg.dim, b.codebooks, b.prepared, b.codes, b.std,
                   b.workspace, b.workspace_bytes, b.status)
    torch.cuda.synchronize()
    codes = codes_to_numpy(cfg, b.codes, n)
    std_bits = b.std.cpu().numpy().view(np.uint16)[:n].copy()
    return codes, std_bits, rvq.read_status(b.status), b


def assert_codes_match(x, codes, codebooks, layout, ddof=0, sample=None):
    """Codes must be the exact argmin at every stage given their own prefix,
    except inside the 1e-5 relative near-tie window; returns the near-tie count."""
    if sample is not None:
        x, codes = x[sample], codes[sample]
    status, wrong = oracle.check_codes(x, codes, codebooks, layout, ddof)
    assert wrong == 0, f"{wrong} (vector, group, stage) positions disagree with the oracle: " \
                       f"{np.argwhere(status >= 2)[:5].tolist()}"
    return int((status == 1).sum())


def assert_std_match(x, std_bits, ddof=0, sample=None):
    """Stored deviation within one binary16 ulp of the oracle's rounding."""
    if sample is not None:
        x, std_bits = x[sample], std_bits[sample]
    x64 = np.asarray(x, dtype=np.float64)
    s = np.std(x64, axis=1, ddof=ddof)          # library routine, pinned against the oracle in the CPU tests
    with np.errstate(over="ignore"):
        want = s.astype(np.float16).view(np.uint16).astype(np.int32)
    got = std_bits.astype(np.int32)
    ok = (s > 0) & np.isfinite(s)
    assert np.all(np.abs(got[ok] - want[ok]) <= 1), "deviation differs by more than one half-precision ulp"
    assert np.all(got[~ok] == 0)
    return float(np.mean(got[ok] != want[ok]))


def gpu_decode(cfg, codes, std_bits, codebooks, n, row_stride=None, prepared_from=None):
    b = prepared_from or rvq.alloc_buffers(cfg, n, codebooks)
    stride = row_stride or cfg.dim
    out = torch.full((max(n, 1), stride), 7.0, dtype=rvq.TORCH_DTYPE[cfg.x_dtype], device="cuda")
    cd = codes_to_device(cfg, codes) if n else torch.zeros(16, dtype=torch.uint8, device="cuda")
    sd = torch.from_numpy(std_bits.view(np.int16).copy()).cuda() if n else torch.zeros(1, dtype=torch.int16, device="cuda")
    rvq.rvq_decode(cfg, cd, sd, n, b.codebooks, b.prepared, out, stride, b.status)
    torch.cuda.synchronize()
    return out[:n].float().cpu().numpy().astype(np.float64), rvq.read_status(b.status)


def assert_recon_match(got, codes, std_bits, codebooks, dim, layout, dtype, rows=None):
    ref = oracle.decode(codes if rows is None else codes[rows], std_bits if rows is None else std_bits[rows],
                        codebooks, dim, layout)
    g = got[:, :dim] if rows is None else got[rows][:, :dim]
    tol = RECON_TOL + HALF_ULP[dtype] * np.abs(ref)
    if dtype != rvq.F32:
        # documented bound of the 16-bit level tables: std * 4.1 * sum_r (max C_r - min C_r) * 2^-17
        # (the tables summed per stage parity; the per-stage ones are four times finer)
        cb = np.asarray(codebooks, dtype=np.float64)
        spread = float(np.sum(cb.max(axis=(1, 2)) - cb.min(axis=(1, 2)))) * 4.1 * 2.0 ** -17
        sd = oracle.f16_value(std_bits if rows is None else std_bits[rows])
        assert np.all(np.abs(g - ref) <= sd[:, None] * spread * 1.01 + HALF_ULP[dtype] * np.abs(ref) * 1.01 + 1e-6), \
            "reconstruction outside the level-table bound"
    err = np.abs(g - ref)
    assert np.all(err <= tol), f"reconstruction off by {err.max():.3e} (worst excess {np.max(err - tol):.3e})"
    return float(err.max())
