"""GPU parity of the codebook-learning calls: rvq_learn_step (encode + EMA update + prepare in one
call) and rvq_kmeans_init (stage-wise Lloyd iterations), against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2410_15704_b200 as rvq
import rvq_synth
from helpers import RECON_TOL, assert_codes_match, codes_to_numpy, config_of, x_to_device

pytestmark = pytest.mark.gpu


def test_learn_step_three_steps_teacher_forced():
    w = rvq_synth.ema_learning(tokens=2048, steps=3)
    cfg = config_of(w)
    x_dev = x_to_device(w.x, cfg.x_dtype)
    b = rvq.alloc_buffers(cfg, w.n, w.codebooks)
    R, K, gd = w.codebooks.shape
    ema_count = torch.ones(R, K, device="cuda")
    ema_sum = b.codebooks.clone()
    exact = torch.empty_like(b.codes)
    for step in range(3):
        cb_before = b.codebooks.cpu().numpy()
        n_before = ema_count.cpu().numpy().astype(np.float64)
        m_before = ema_sum.cpu().numpy().astype(np.float64)
        rvq.rvq_learn_step(cfg, x_dev, w.n, w.dim, b.codebooks, b.prepared, ema_count, ema_sum, b.codes, b.std,
                           w.decay, w.eps, b.workspace, b.workspace_bytes, b.status)
        torch.cuda.synchronize()
        codes = codes_to_numpy(cfg, b.codes, w.n)
        assert_codes_match(w.x, codes, cb_before, w.layout)
        # teacher-forced: the oracle's update from the same codes and the same state
        ref = oracle.ema_update(w.x, codes, cb_before, n_before, m_before, w.decay, w.eps, w.layout)
        e_cb = np.abs(b.codebooks.cpu().numpy() - ref["codebooks"]).max()
        e_n = np.abs(ema_count.cpu().numpy() - ref["ema_count"]).max()
        e_m = (np.abs(ema_sum.cpu().numpy() - ref["ema_sum"]).max(axis=2) / np.maximum(1.0, ref["ema_count"])).max()
        assert e_cb <= RECON_TOL and e_m <= RECON_TOL and e_n <= 1e-3 * max(1.0, ref["ema_count"].max())
        assert np.abs(b.codebooks.cpu().numpy() - cb_before).max() > 1e-4        # the step did move them
        # the prepared block belongs to the NEW codebooks: the tensor-core encode with it
        # agrees with the all-float32 encode, which reads the codebooks only
        rvq.rvq_encode(cfg, x_dev, w.n, w.dim, b.codebooks, b.prepared, b.codes, b.std, b.workspace,
                       b.workspace_bytes, b.status)
        rvq.rvq_encode_exact(cfg, x_dev, w.n, w.dim, b.codebooks, b.prepared, exact, b.std, b.status)
        torch.cuda.synchronize()
        assert torch.equal(b.codes, exact)
    st = rvq.read_status(b.status)
    assert st["bad_codes"] == 0 and st["wait_timeouts"] == 0


def gpu_kmeans(cfg, x, n, seeds, iters):
    R, K, gd = cfg.depth, cfg.codebook_size, cfg.group_dim
    cb = torch.zeros(R, K, gd, device="cuda")
    prepared = torch.empty(rvq.rvq_prepared_bytes(cfg), dtype=torch.uint8, device="cuda")
    nbytes = rvq.rvq_kmeans_workspace_bytes(cfg, n)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = rvq.new_status()
    rvq.rvq_kmeans_init(cfg, x_to_device(x, cfg.x_dtype), n, cfg.dim, torch.from_numpy(seeds).cuda(), iters, cb,
                        prepared, ws, nbytes, status)
    torch.cuda.synchronize()
    st = rvq.read_status(status)
    assert st["wait_timeouts"] == 0
    return cb.cpu().numpy().astype(np.float64), cb, prepared


def residual_energy(x, cbs, layout):
    enc = oracle.encode(x, cbs, 32, layout, want_residual=True)
    return float((enc["residual"] ** 2).mean())


def clustered_vectors(seed, n, K, layout, G=4):
    """Head vectors whose G groups each sit near one of K well-separated centres."""
    g = np.random.default_rng(seed)
    centres = g.normal(size=(K, 32)) * 3.0
    labels = g.integers(0, K, size=(n, G))
    rows = centres[labels] + 0.05 * g.normal(size=(n, G, 32))            # [n][G][32]
    x = rows.reshape(n, 32 * G) if layout == rvq_synth.CONTIGUOUS else rows.transpose(0, 2, 1).reshape(n, 32 * G)
    x = torch.from_numpy(x).to(torch.bfloat16).float().numpy()           # exactly representable
    return x, labels.reshape(-1)


@pytest.mark.parametrize("layout,G", [(rvq_synth.CONTIGUOUS, 4), (rvq_synth.STRIDED, 4), (rvq_synth.STRIDED, 8)])
def test_kmeans_init_on_separated_clusters(layout, G):
    n, K, R, iters = 1500, 16, 3, 4                                      # ragged last tile
    x, labels = clustered_vectors(31, n, K, layout, G)
    seeds = np.stack([np.array([np.flatnonzero(labels == k)[r] for k in range(K)]) for r in range(R)]).astype(np.int64)
    cfg = rvq.make_config(32 * G, 32, layout, R, K, 16, rvq.BF16, 0)
    got, _, _ = gpu_kmeans(cfg, x, n, seeds, iters)
    ref = oracle.kmeans_init(x, seeds, iters, 32, layout)
    # stage 0: every row sits far inside its cluster, so the assignments cannot differ
    assert np.abs(got[0] - ref[0]).max() <= RECON_TOL
    # later stages work on what the clusters leave (noise): a row between two centroids may fall either
    # way in float32, which moves two centroids a little; nearly all centroids still agree
    per_centroid = np.abs(got - ref).max(axis=2)
    assert np.mean(per_centroid > RECON_TOL) <= 0.05
    e_got, e_ref = residual_energy(x, got, layout), residual_energy(x, ref, layout)
    assert abs(e_got - e_ref) <= 1e-3 * e_ref
    print(f"k-means (clusters, layout {layout}): centroid max-abs {per_centroid.max():.2e}, "
          f"residual energy {e_got:.5f} vs {e_ref:.5f}")


def test_kmeans_init_on_key_like_data():
    w = rvq_synth.key_cache(tokens=512, depth=4, size=64)
    cfg = config_of(w)
    g = np.random.default_rng(77)
    seeds = np.stack([g.choice(w.n * 4, 64, replace=False) for _ in range(4)]).astype(np.int64)
    got0, _, _ = gpu_kmeans(cfg, w.x, w.n, seeds, 0)
    ref0 = oracle.kmeans_init(w.x, seeds, 0, 32, w.layout)
    np.testing.assert_allclose(got0[0], ref0[0], rtol=0, atol=1e-5 * np.abs(ref0[0]).max())   # the scaled seed rows
    assert np.mean(np.abs(got0 - ref0).max(axis=2) > RECON_TOL) <= 0.05
    got, cb_dev, prepared = gpu_kmeans(cfg, w.x, w.n, seeds, 5)
    ref = oracle.kmeans_init(w.x, seeds, 5, 32, w.layout)
    e0 = residual_energy(w.x, got0, w.layout)
    e_got, e_ref = residual_energy(w.x, got, w.layout), residual_energy(w.x, ref, w.layout)
    assert e_got < 0.9 * e0                                   # the iterations pay
    assert abs(e_got - e_ref) <= 0.02 * e_ref                 # and land where the oracle's do
    # the prepared block that comes back serves these codebooks
    b = rvq.alloc_buffers(cfg, w.n, got.astype(np.float32))
    x_dev = x_to_device(w.x, cfg.x_dtype)
    rvq.rvq_encode(cfg, x_dev, w.n, w.dim, cb_dev, prepared, b.codes, b.std, b.workspace, b.workspace_bytes, b.status)
    torch.cuda.synchronize()
    assert_codes_match(w.x, codes_to_numpy(cfg, b.codes, w.n), got.astype(np.float32), w.layout)
    print(f"k-means (key-like): residual energy seeds {e0:.4f}, 5 iterations {e_got:.4f}, oracle {e_ref:.4f}")


def gpu_assign(cfg_r, x, n, cbs):
    """Codes the GPU encoder gives `x` with the codebooks `cbs` (float32 [r][K][32])."""
    b = rvq.alloc_buffers(cfg_r, n, cbs)
    rvq.rvq_encode(cfg_r, x_to_device(x, cfg_r.x_dtype), n, cfg_r.dim, b.codebooks, b.prepared, b.codes, b.std,
                   b.workspace, b.workspace_bytes, b.status)
    torch.cuda.synchronize()
    return codes_to_numpy(cfg_r, b.codes, n)


@pytest.mark.parametrize("layout", [rvq_synth.CONTIGUOUS, rvq_synth.STRIDED])
def test_kmeans_lloyd_iterations_teacher_forced(layout):
    """Single Lloyd iterations checked centroid by centroid.  An iteration is an assignment followed
    by cluster means; the assignment the GPU makes from given centroids is the encoder's (checked
    against the oracle's argmin), and with that assignment fixed the means have one right answer,
    which the oracle computes: every centroid must agree within 1e-3.  Done for the first and the
    second iteration of stage 0 and for the first iteration of stage 1 (whose rows are what stage 0
    leaves) on key-like data, where free-running runs may part at near ties."""
    w = rvq_synth.key_cache(tokens=512, depth=2, size=64)
    w.layout = layout
    K, G = 64, w.groups
    g = np.random.default_rng(91)
    seeds = np.stack([g.choice(w.n * G, K, replace=False) for _ in range(2)]).astype(np.int64)

    def cfg_for(depth):
        return rvq.make_config(w.dim, 32, layout, depth, K, 16, rvq.BF16, 0)

    z0 = oracle.scaled_groups(w.x, 32, layout).reshape(-1, 32)           # stage-0 rows [n*G][32], float64

    def means(rows, codes, before):
        out = before.astype(np.float64).copy()
        for j in range(K):
            sel = codes == j
            if sel.any():
                out[j] = rows[sel].mean(axis=0)
        return out

    prev, _, _ = gpu_kmeans(cfg_for(1), w.x, w.n, seeds[:1], 0)          # the seed centroids as the GPU holds them
    for it in (1, 2):
        got, _, _ = gpu_kmeans(cfg_for(1), w.x, w.n, seeds[:1], it)
        codes = gpu_assign(cfg_for(1), w.x, w.n, prev.astype(np.float32))
        assert_codes_match(w.x, codes, prev.astype(np.float32), layout)
        want = means(z0, codes.reshape(-1), prev[0])
        assert np.abs(got[0] - want).max() <= RECON_TOL, f"stage 0, iteration {it}"
        prev = got
    # stage 1 after one iteration per stage: rows = stage-0 rows minus the centroid stage 0 assigned them
    got2, _, _ = gpu_kmeans(cfg_for(2), w.x, w.n, seeds, 1)
    cb0 = got2[0]
    codes0 = gpu_assign(cfg_for(1), w.x, w.n, cb0[None].astype(np.float32)).reshape(-1)
    z1 = z0 - cb0[codes0]
    seed_centroids = z1[seeds[1]]
    both = np.stack([cb0, seed_centroids]).astype(np.float32)
    codes = gpu_assign(cfg_for(2), w.x, w.n, both)
    assert_codes_match(w.x, codes, both, layout)
    assert np.array_equal(codes[:, :, 0].reshape(-1), codes0)
    want1 = means(z1, codes[:, :, 1].reshape(-1), seed_centroids)
    assert np.abs(got2[1] - want1).max() <= RECON_TOL, "stage 1, iteration 1"
