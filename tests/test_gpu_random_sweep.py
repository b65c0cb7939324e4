"""Randomized sweeps over shapes the fixed workloads do not visit: codebook sizes that are no multiple of
128, shallow depths, every input type, both deviation conventions, wild per-vector deviations, duplicate
codewords, packed codes.  Encode is checked against the oracle's verdict on the codes and against the
all-float32 kernel; decode (plain and rotary) against the oracle's reconstruction."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_15704_b200 as rvq
from helpers import HALF_ULP, codes_to_device, codes_to_numpy

pytestmark = pytest.mark.gpu


def test_random_encode_cases_against_oracle_and_float32_kernel():
    g = np.random.default_rng(20241)
    near = 0
    for case in range(90):
        K = int(g.choice([64, 100, 128, 300, 512, 1000, 1024, 1536, 2048, 3000]))
        R = int(g.choice([1, 2, 4, 5, 8]))
        layout, ddof = int(g.integers(0, 2)), int(g.integers(0, 2))
        n = int(g.choice([1, 33, 129, 1000, 2049]))
        dt = [rvq.F32, rvq.BF16, rvq.F16][int(g.integers(0, 3))]
        kind = int(g.integers(0, 3))
        if kind == 0:
            x = g.normal(size=(n, 128)) * g.uniform(0.2, 5.0, size=(1, 128))
        elif kind == 1:
            a = 0.25 + np.abs(g.laplace(size=(1, 128)))
            a[0, g.integers(0, 128, size=8)] *= 20.0
            x = a * g.normal(size=(n, 128))
        else:
            x = g.normal(size=(n, 128)) * np.exp(g.normal(size=(n, 1)) * 2.0)
        cb = np.stack([g.normal(scale=float(g.choice([0.3, 1.0, 3.0])) * 0.8 ** r, size=(K, 32)) for r in range(R)]).astype(np.float32)
        if case % 4 == 0:
            cb[0, 1] = cb[0, 0]                                          # duplicate codewords: exact ties
        bits = 16 if case % 2 else max(1, int(np.ceil(np.log2(K))))
        cfg = rvq.make_config(128, 32, layout, R, K, bits, dt, ddof)
        xt = torch.from_numpy(x.astype(np.float32)).to(rvq.TORCH_DTYPE[dt]).cuda()
        xv = xt.float().cpu().numpy()                                    # the values the kernels saw
        b = rvq.alloc_buffers(cfg, n, cb)
        rvq.rvq_encode(cfg, xt, n, 128, b.codebooks, b.prepared, b.codes, b.std, b.workspace, b.workspace_bytes, b.status)
        exact, std2 = torch.empty_like(b.codes), torch.empty_like(b.std)
        rvq.rvq_encode_exact(cfg, xt, n, 128, b.codebooks, b.prepared, exact, std2, b.status)
        torch.cuda.synchronize()
        what = dict(case=case, K=K, R=R, layout=layout, ddof=ddof, n=n, dt=dt, kind=kind, bits=bits)
        assert torch.equal(b.codes, exact) and torch.equal(b.std, std2), what
        status, wrong = oracle.check_codes(xv, codes_to_numpy(cfg, b.codes, n), cb, layout, ddof)
        assert wrong == 0, what
        near += int((status == 1).sum())
        assert rvq.read_status(b.status)["wait_timeouts"] == 0
    print(f"random encode cases: {near} near ties")


def test_random_decode_cases_against_oracle():
    g = np.random.default_rng(20242)
    table = torch.empty(5000, 64, 2, device="cuda")
    rvq.rvq_rope_table(128, 500000.0, 5000, table)
    for case in range(120):
        K = int(g.choice([64, 100, 512, 1000, 1024, 1536, 2048, 3000, 3584]))
        R = int(g.choice([2, 4, 6, 8]))
        layout = int(g.integers(0, 2))
        n = 8 * int(g.choice([1, 5, 130, 700]))
        dt = [rvq.F32, rvq.BF16, rvq.F16][int(g.integers(0, 3))]
        bits = 16 if g.integers(0, 2) else max(1, int(np.ceil(np.log2(K))))
        mode = int(g.integers(0, 4))
        std = float(g.choice([0.2, 1.0, 2.5, 6.0, 40.0])) * (np.abs(1.0 + 0.25 * g.normal(size=n)) + 0.05)
        if mode == 1:
            std[g.integers(0, n, size=max(1, n // 50))] *= 30.0          # single rows beyond any table's reach
        if mode == 2:
            std *= np.exp(g.normal(size=n))                               # a wide mix within the batch
        if mode == 3:
            std[g.integers(0, n, size=max(1, n // 100))] = 0.0
        std_bits = np.minimum(std, 60000.0).astype(np.float16).view(np.uint16)
        codes = g.integers(0, K, size=(n, 4, R)).astype(np.int32)
        cb = np.stack([g.normal(scale=0.5 * 0.75 ** r, size=(K, 32)) for r in range(R)]).astype(np.float32)
        cfg = rvq.make_config(128, 32, layout, R, K, bits, dt, 0)
        b = rvq.alloc_buffers(cfg, n, cb)
        cd, sd = codes_to_device(cfg, codes), torch.from_numpy(std_bits.view(np.int16)).cuda()
        out = torch.empty(n, 128, dtype=rvq.TORCH_DTYPE[dt], device="cuda")
        rope = int(g.integers(0, 3))
        pos = g.integers(0, 5000, size=n // 8).astype(np.int32)
        with_prepared = bool(g.integers(0, 4))
        if rope == 0:
            rvq.rvq_decode(cfg, cd, sd, n, b.codebooks, b.prepared, out, 128, b.status)
            ref = oracle.decode(codes, std_bits, cb, 128, layout)
        else:
            style = rvq.ROPE_HALVES if rope == 1 else rvq.ROPE_ADJACENT
            rvq.rvq_decode_rope(cfg, cd, sd, n, b.codebooks, b.prepared if with_prepared else None, torch.from_numpy(pos).cuda(),
                                8, table, 5000, style, out, 128, b.status)
            ref = oracle.decode_rope(codes, std_bits, cb, np.repeat(pos, 8), 500000.0, style, 128, layout)
        torch.cuda.synchronize()
        err = np.abs(out.float().cpu().numpy().astype(np.float64) - ref)
        # float32 outputs are float32 sums: at values of 1e4 (deviations in the thousands) one float32 ulp is 1e-3
        half = HALF_ULP[dt] if dt != rvq.F32 else 2.0 ** -22
        assert np.all(err <= 1e-3 + half * np.abs(ref) * 1.01), dict(case=case, K=K, R=R, layout=layout, n=n, dt=dt, bits=bits,
                                                                      mode=mode, rope=rope, prepared=with_prepared,
                                                                      excess=float((err - 1e-3 - half * np.abs(ref)).max()))
