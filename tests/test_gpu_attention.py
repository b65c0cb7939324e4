"""GPU parity of rvq_attention_decode (one new token attending over the compressed cache,
keys rotated as they are read) against the CPU oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2410_15704_b200 as rvq
import rvq_synth
from helpers import codes_to_device

pytestmark = pytest.mark.gpu

BASE = 500000.0
TOL = 1e-3        # the bar of the reconstructions; float32 arithmetic stays two orders below it (asserted)


def rope_table(positions):
    t = torch.empty(positions, 64, 2, device="cuda")
    rvq.rvq_rope_table(128, BASE, positions, t)
    torch.cuda.synchronize()
    return t


def make_cache(g, tokens, K, R, std_scale=1.0):
    n = tokens * 8
    codes = g.integers(0, K, size=(n, 4, R)).astype(np.int32)
    std = std_scale * (np.abs(1.0 + 0.25 * g.normal(size=n)) + 0.05)
    cb = np.stack([g.normal(scale=0.5 * 0.75 ** r, size=(K, 32)) for r in range(R)]).astype(np.float32)
    return codes, std.astype(np.float16).view(np.uint16), cb


def run_case(tokens, q_heads, Kk=256, Kv=256, Rk=8, Rv=8, bits_k=16, bits_v=16, layout_k=rvq_synth.STRIDED,
             layout_v=rvq_synth.CONTIGUOUS, pairing=rvq.ROPE_HALVES, rotate=True, explicit_positions=True,
             q_gain=1.0, std_scale=1.0, max_pos=40000, seed=0):
    g = np.random.default_rng(1000 * tokens + q_heads + Kk + 7 * seed)
    ck, sk, cbk = make_cache(g, tokens, Kk, Rk, std_scale)
    cv, sv, cbv = make_cache(g, tokens, Kv, Rv)
    q = (q_gain * g.normal(size=(q_heads, 128))).astype(np.float32)
    scale = float(128 ** -0.5)
    pos = g.integers(0, max_pos, size=tokens).astype(np.int32) if explicit_positions else np.arange(tokens, dtype=np.int32)
    cfg_k = rvq.make_config(128, 32, layout_k, Rk, Kk, bits_k, rvq.BF16, 0)
    cfg_v = rvq.make_config(128, 32, layout_v, Rv, Kv, bits_v, rvq.BF16, 0)
    table = rope_table(max(max_pos, tokens)) if rotate else None
    ws_bytes = rvq.rvq_attention_workspace_bytes(tokens, q_heads)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    out = torch.full((q_heads, 128), 7.0, device="cuda")
    status = rvq.new_status()
    rvq.rvq_attention_decode(cfg_k, cfg_v, torch.from_numpy(q).cuda(), q_heads, codes_to_device(cfg_k, ck),
                             torch.from_numpy(sk.view(np.int16)).cuda(), codes_to_device(cfg_v, cv),
                             torch.from_numpy(sv.view(np.int16)).cuda(), tokens, 8, torch.from_numpy(cbk).cuda(),
                             torch.from_numpy(cbv).cuda(), torch.from_numpy(pos).cuda() if explicit_positions else None,
                             table, max(max_pos, tokens), pairing, scale, out, ws, ws_bytes, status)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    ref = oracle.attention_decode(q, ck, sk, cv, sv, cbk, cbv, 8, scale, pos if rotate else None, BASE, pairing, 128,
                                  layout_k, layout_v)
    err = np.abs(got - ref).max()
    assert err <= TOL, f"attention output off by {err:.3e}"
    assert err <= 2e-5 * max(1.0, np.abs(ref).max()) * max(1.0, q_gain), f"float32 arithmetic should do better than {err:.3e}"
    assert rvq.read_status(status)["bad_codes"] == 0
    return err


@pytest.mark.parametrize("layout_k", [rvq_synth.CONTIGUOUS, rvq_synth.STRIDED])
@pytest.mark.parametrize("pairing", [rvq.ROPE_HALVES, rvq.ROPE_ADJACENT])
@pytest.mark.parametrize("q_heads", [8, 16, 32])
def test_attention_matches_oracle(layout_k, pairing, q_heads):
    """All pairings of key layout and rotary convention, one to four query heads per kv head, a token
    count that leaves part of the last round of warps idle."""
    err = run_case(1237, q_heads, layout_k=layout_k, pairing=pairing)
    print(f"attention layout {layout_k} pairing {pairing} q_heads {q_heads}: max-abs {err:.2e}")


@pytest.mark.parametrize("tokens", [1, 2, 31, 33, 4097])
def test_attention_ragged_token_counts(tokens):
    run_case(tokens, 32)


def test_attention_other_quantizers():
    # the paper's key quantizer at 1024 codes, values contiguous; then packed codes, shallower and unequal depths
    run_case(2000, 32, Kk=1024, Kv=1024)
    run_case(700, 32, Kk=1024, Kv=512, Rk=6, Rv=4, bits_k=10, bits_v=9)
    run_case(700, 16, Kk=1792, Kv=100, Rk=8, Rv=8, bits_k=11, bits_v=7, layout_v=rvq_synth.STRIDED)
    # keys as stored (no rotation), positions implied by the token index, key-like deviations
    run_case(900, 32, rotate=False)
    run_case(900, 32, explicit_positions=False)
    run_case(900, 32, std_scale=6.0)


def test_attention_peaked_and_flat_weights():
    """Large queries make the softmax pick a handful of tokens (scores in the hundreds); tiny queries make it
    the plain mean of the values."""
    run_case(3000, 32, q_gain=30.0)
    run_case(3000, 32, q_gain=1e-3)


def test_attention_at_cache_size_of_a_long_context_slice():
    """16384 tokens x 8 kv heads = 131072 cached head vectors per side, the paper's 1024-code quantizers."""
    err = run_case(16384, 32, Kk=1024, Kv=1024, max_pos=131072)
    print(f"attention over 16384 tokens: max-abs {err:.2e}")


def test_attention_counts_bad_codes_and_rejects_bad_arguments():
    g = np.random.default_rng(5)
    tokens = 64
    ck, sk, cbk = make_cache(g, tokens, 256, 8)
    cv, sv, cbv = make_cache(g, tokens, 256, 8)
    ck[3, 1, 2] = 300                                                    # past the codebook: read as code 0
    cfg = rvq.make_config(128, 32, rvq_synth.CONTIGUOUS, 8, 256, 16, rvq.BF16, 0)
    q = g.normal(size=(32, 128)).astype(np.float32)
    ws_bytes = rvq.rvq_attention_workspace_bytes(tokens, 32)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    out = torch.empty(32, 128, device="cuda")
    status = rvq.new_status()
    args = [torch.from_numpy(q).cuda(), 32, codes_to_device(cfg, ck), torch.from_numpy(sk.view(np.int16)).cuda(),
            codes_to_device(cfg, cv), torch.from_numpy(sv.view(np.int16)).cuda(), tokens, 8,
            torch.from_numpy(cbk).cuda(), torch.from_numpy(cbv).cuda(), None, None, 0, 0, 0.1, out, ws, ws_bytes]
    rvq.rvq_attention_decode(cfg, cfg, *args, status)
    torch.cuda.synchronize()
    assert rvq.read_status(status)["bad_codes"] == 1                     # every slice sees it, one of them counts it
    ck[3, 1, 2] = 0
    ref = oracle.attention_decode(q, ck, sk, cv, sv, cbk, cbv, 8, 0.1, None)
    assert np.abs(out.cpu().numpy() - ref).max() <= 1e-4
    # shapes outside the kernels' reach, a workspace that is too small, no tokens
    wide = rvq.make_config(256, 32, 0, 8, 256, 16, rvq.BF16, 0)
    assert rvq.rvq_attention_decode(wide, cfg, *args, None, check=False) == -3
    assert rvq.rvq_attention_decode(cfg, cfg, *(args[:7] + [4] + args[8:]), None, check=False) == -3        # four kv heads
    assert rvq.rvq_attention_decode(cfg, cfg, *(args[:-1] + [16]), None, check=False) == -4
    assert rvq.rvq_attention_decode(cfg, cfg, *(args[:6] + [0] + args[7:]), None, check=False) == -1
