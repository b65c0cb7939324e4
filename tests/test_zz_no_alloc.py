"""rvq_ema_update_static: the EMA codebook update for callers that cannot allocate.

Some users of this library run where device memory is not theirs to ask for: inside a host
application that owns the allocator and passes in only inputs and outputs, or in a phase
where cudaMalloc is off limits.  rvq_ema_update needs a caller-provided workspace; the
static variant keeps that scratch in a fixed array inside the library instead.  This file
checks, through the C ABI, that the variant gives the same update as rvq_ema_update --
twice in a row, because the second call starts on the first call's leftovers in the shared
array -- and that it refuses shapes larger than the array.  (Collected last on purpose.)"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2410_15704_b200 as rvq
import rvq_synth

pytestmark = pytest.mark.gpu
TOL = 1e-3          # the bound the other parity tests put on EMA codebooks


def test_static_scratch_update_matches_workspace_update_twice():
    w = rvq_synth.ema_learning(tokens=512)
    cfg = rvq.make_config(w.dim, w.group_dim, w.layout, w.depth, w.codebook_size, 16, rvq.BF16, 0)
    x = torch.from_numpy(w.x).to(torch.bfloat16).cuda()
    R, K = w.depth, w.codebook_size
    assert rvq.rvq_workspace_bytes(cfg, w.n) <= rvq.rvq_ema_static_scratch_bytes()

    ref = rvq.alloc_buffers(cfg, w.n, w.codebooks)        # updated with a caller workspace
    sta = rvq.alloc_buffers(cfg, w.n, w.codebooks)        # updated with the built-in scratch
    state = {}
    for name, b in (("ref", ref), ("sta", sta)):
        state[name] = dict(n=torch.ones(R, K, device="cuda"), m=b.codebooks.clone(),
                           batch=torch.zeros(R, K, device="cuda"))
    for call in range(2):
        # both sides encode with the reference side's codebooks so that they see the same codes
        rvq.rvq_prepare_codebooks(cfg, ref.codebooks, ref.prepared)
        rvq.rvq_encode(cfg, x, w.n, w.dim, ref.codebooks, ref.prepared, ref.codes, ref.std, ref.workspace,
                       ref.workspace_bytes, ref.status)
        sta.codebooks.copy_(ref.codebooks)
        state["sta"]["n"].copy_(state["ref"]["n"]); state["sta"]["m"].copy_(state["ref"]["m"])
        rvq.rvq_ema_update(cfg, x, w.n, w.dim, ref.codes, ref.codebooks, state["ref"]["n"], state["ref"]["m"],
                           state["ref"]["batch"], w.decay, w.eps, ref.workspace, ref.workspace_bytes, ref.status)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rvq.rvq_ema_update_static(cfg, x, w.n, w.dim, ref.codes, sta.codebooks, state["sta"]["n"],
                                  state["sta"]["m"], state["sta"]["batch"], w.decay, w.eps, sta.status)
        torch.cuda.synchronize()
        # the call took no device memory (torch's allocator was not involved either: the binding passes pointers)
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(state["ref"]["batch"], state["sta"]["batch"])              # counts are integers
        assert int(state["sta"]["batch"].sum().item()) == w.n * w.groups * R
        assert torch.max(torch.abs(ref.codebooks - sta.codebooks)).item() <= TOL
        assert torch.max(torch.abs(state["ref"]["n"] - state["sta"]["n"])).item() <= TOL
        per_code = torch.max(torch.abs(state["ref"]["m"] - state["sta"]["m"]), dim=2).values
        assert torch.max(per_code / torch.clamp(state["ref"]["n"], min=1.0)).item() <= TOL
    assert rvq.read_status(sta.status)["bad_codes"] == 0


def test_static_scratch_refuses_shapes_beyond_its_size():
    big = rvq.make_config(128, 32, rvq.CONTIGUOUS, 8, 4096, 16, rvq.BF16, 0)
    assert rvq.rvq_workspace_bytes(big, 16) > rvq.rvq_ema_static_scratch_bytes()
    x = torch.zeros(16, 128, dtype=torch.bfloat16, device="cuda")
    codes = torch.zeros(16 * 64, dtype=torch.uint8, device="cuda")
    cb = torch.zeros(8, 4096, 32, device="cuda")
    cnt, msum = torch.ones(8, 4096, device="cuda"), torch.zeros(8, 4096, 32, device="cuda")
    before = rvq.rvq_launch_count()
    rc = rvq.rvq_ema_update_static(big, x, 16, 128, codes, cb, cnt, msum, None, 0.99, 1e-5, check=False)
    assert rc == -7 and "built-in" in rvq.rvq_status_string(rc)
    assert rvq.rvq_launch_count() == before                  # nothing was launched
