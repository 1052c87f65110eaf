"""Input generators: shapes, sums, fractions and determinism (no hook arithmetic here)."""
import numpy as np

import workloads as W


def test_ragged_lengths():
    rng = np.random.default_rng(0)
    l = W.ragged_lengths_uniform(rng, 64, 8)
    assert l.sum() == 64 and l.min() >= 1 and len(l) == 8
    l = W.ragged_lengths_lognormal(rng, 8192, 64)
    assert l.sum() == 8192 and l.min() >= 1 and l.max() <= 2048 and len(l) == 64


def test_tiny_and_decode_structure_and_determinism():
    a, b = W.make_tiny(), W.make_tiny()
    assert np.array_equal(W.bits(a.hidden), W.bits(b.hidden)) and np.array_equal(a.token_slot, b.token_slot)
    assert a.hidden.shape == (64, 512) and (a.token_slot == -1).sum() > 0
    assert sorted(a.apps) == [0, 1, 2, 3] and a.groups[0].W_enc.shape == (4096, 512)
    n = np.linalg.norm(a.groups[0].W_dec.float().numpy(), axis=1)
    assert np.allclose(n, 1.0, atol=5e-3)
    d = W.make_decode()
    assert d.hidden.shape == (256, 4096) and (d.token_slot == -1).sum() == 64
    assert len(d.apps) == 96 and len(d.meta["outlier_cols"]) == 4
    cols = d.meta["outlier_cols"]
    assert d.hidden.float()[:, cols].abs().mean() > 10 * d.hidden.float().abs().mean() / 2
    counts = np.bincount(d.token_slot[d.token_slot >= 0], minlength=96)
    assert (counts == 2).all()


def test_mixed_and_replay_small():
    w = W.make_mixed(d=128, T=1024, R=64, d_sae=512, cap=256)
    assert (w.token_slot == -1).mean() >= 0.30
    kinds = {a.kind for a in w.apps.values()}
    assert kinds == {W.KIND_PROBE, W.KIND_STEER, W.KIND_SAE}
    r = W.make_replay(d=128, T_max=256, d_sae=1024, k=8, G=2)
    ts0, n0 = W.replay_map(r, 0); ts1, n1 = W.replay_map(r, 1)
    assert n0 == 0 and (ts0 == -1).all() and n1 == 256
    ts5, n5 = W.replay_map(r, 5)
    assert (ts5[n5:] == -1).all()
    assert np.array_equal(ts5, W.replay_map(r, 5)[0])
