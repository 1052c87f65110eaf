"""Pins for the float64 oracle: values and facts fixed by the mathematics (closed forms,
hand-worked numbers, brute force, library routines, invariants), never by the oracle itself."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_d4.json")))


def bf(a):
    """float array -> bf16 bits via torch (a library rounding, independent of the oracle's)."""
    t = torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return W.bits(t)


class _Sae:
    def __init__(self, **kw):
        self.theta = None; self.b_dec = None; self.center_input = False; self.k = 0
        self.__dict__.update(kw)


class _App:
    kind = O.KIND_SAE
    def __init__(self, idx=(), val=(), mode=(), add_error=True, group=0):
        self.edit_idx = np.asarray(idx, dtype=np.int32); self.edit_val = np.asarray(val, dtype=np.float32)
        self.edit_mode = np.asarray(mode, dtype=np.uint8); self.add_error = add_error; self.group = group


# ------------------------------------------------------------------ bf16 conversions
def test_bf16_to_f64_known_bits():
    # 0x3F80 = 1.0, 0xC000 = -2.0, 0x3E80 = 0.25, 0x4049 = 3.140625, 0x0000 = 0, 0x7F80 = inf
    got = O.bf16_to_f64(np.array([0x3F80, 0xC000, 0x3E80, 0x4049, 0x0000, 0x7F80], dtype=np.uint16))
    assert got.tolist() == [1.0, -2.0, 0.25, 3.140625, 0.0, math.inf]


def test_f64_to_bf16_matches_torch_rounding_on_fp32_values():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 65504.0, 1e-40, -3e38]]).astype(np.float32)
    want = W.bits(torch.from_numpy(x).to(torch.bfloat16))
    got = O.f64_to_bf16_bits(x.astype(np.float64))
    assert np.array_equal(got, want)


def test_f64_to_bf16_ties_to_even_and_roundtrip():
    # 1 + 2^-8 is exactly halfway between bf16 1.0 (even mantissa) and 1.0078125 -> 1.0
    assert O.f64_to_bf16_bits(np.array([1.00390625]))[0] == 0x3F80
    # 1.0078125 + 2^-8 halfway between odd 0x3F81 and even 0x3F82 -> 0x3F82
    assert O.f64_to_bf16_bits(np.array([1.01171875]))[0] == 0x3F82
    allbits = np.arange(0, 0x7F80, dtype=np.uint16)          # every finite non-negative bf16
    assert np.array_equal(O.f64_to_bf16_bits(O.bf16_to_f64(allbits)), allbits)


# ------------------------------------------------------------------ probe
def test_probe_hand_worked():
    h = np.array(GOLD["h"])
    for key, act in [("probe_sigmoid", O.ACT_SIGMOID), ("probe_sigmoid_2", O.ACT_SIGMOID),
                     ("probe_softmax", O.ACT_SOFTMAX), ("probe_softmax_2", O.ACT_SOFTMAX)]:
        g = GOLD[key]
        s = O.probe_scores(h, np.array(g["W"], dtype=np.float64), np.array(g["b"]), act)
        assert np.allclose(s, g["score"], rtol=0, atol=1e-15), key
        z = O.probe_scores(h, np.array(g["W"], dtype=np.float64), np.array(g["b"]), O.ACT_NONE)
        assert z.tolist() == g["z"], key


def test_probe_closed_forms():
    rng = np.random.default_rng(1)
    h = rng.standard_normal(64)
    assert O.probe_scores(h, np.zeros((1, 64)), None, O.ACT_SIGMOID)[0] == 0.5
    assert np.allclose(O.probe_scores(h, np.zeros((7, 64)), np.zeros(7), O.ACT_SOFTMAX), 1 / 7, atol=1e-16)
    assert O.probe_scores(h, rng.standard_normal((1, 64)), None, O.ACT_SOFTMAX).tolist() == [1.0]   # softmax of one class
    e = np.zeros((1, 64)); e[0, 5] = 1.0
    assert O.probe_scores(h, e, None, O.ACT_SIGMOID)[0] == pytest.approx(1 / (1 + math.exp(-h[5])), rel=1e-15)
    Wm = rng.standard_normal((5, 64)); b = rng.standard_normal(5)
    s = O.probe_scores(h, Wm, b, O.ACT_SOFTMAX)
    assert s.sum() == pytest.approx(1.0, abs=1e-15)
    assert np.allclose(s, O.probe_scores(h, Wm, b + 3.25, O.ACT_SOFTMAX), atol=1e-15)   # shift invariance
    # softmax over two classes equals the sigmoid of the logit difference
    s2 = O.probe_scores(h, Wm[:2], b[:2], O.ACT_SOFTMAX)
    z2 = O.probe_scores(h, Wm[:2], b[:2], O.ACT_NONE)
    assert s2[0] == pytest.approx(1 / (1 + math.exp(-(z2[0] - z2[1]))), rel=1e-14)
    # a transposed or mis-indexed W would fail this term-by-term sum
    z = [b[c] + math.fsum(Wm[c, i] * h[i] for i in range(64)) for c in range(5)]
    assert np.allclose(O.probe_scores(h, Wm, b, O.ACT_NONE), z, rtol=1e-13)


# ------------------------------------------------------------------ steering
def test_steer_hand_worked_and_invariants():
    g = GOLD["steer"]
    assert O.steer(np.array(GOLD["h"]), np.array(g["v"]), g["alpha"]).tolist() == g["out"]
    rng = np.random.default_rng(2)
    h = rng.standard_normal(32); v = rng.standard_normal(32)
    assert np.array_equal(O.steer(h, v, 0.0), h)
    e = np.zeros(32); e[7] = 1.0
    out = O.steer(h, e, 2.5)
    assert out[7] == h[7] + 2.5 and np.array_equal(np.delete(out, 7), np.delete(h, 7))
    back = O.steer(O.steer(h, v, 3.0), v, -3.0)
    assert np.allclose(back, h, rtol=0, atol=1e-15)
    assert np.array_equal(O.steer(h, v, -1.0), h - v)          # "subtract a vector"


# ------------------------------------------------------------------ SAE pieces
def _gold_sae(act=O.SAE_TOPK, theta=None):
    g = GOLD["sae"]
    return _Sae(d_sae=6, act=act, k=g["k"], W_enc=bf(g["W_enc"]), b_enc=np.array(g["b_enc"], dtype=np.float32),
                W_dec=bf(g["W_dec"]), theta=theta)


def test_sae_hand_worked():
    g = GOLD["sae"]; h = np.array(GOLD["h"])
    sae = _gold_sae()
    z = O.sae_preact(h, sae.W_enc, sae.b_enc)[0]
    assert z.tolist() == g["z"]
    f, K = O.sae_activate(z, O.SAE_TOPK, k=g["k"])
    assert K.tolist() == g["topk"] and f.tolist() == g["f"]
    assert O.sae_activate(z, O.SAE_RELU)[0].tolist() == g["relu_f"]
    assert O.sae_activate(z, O.SAE_JUMPRELU, theta=np.array(g["jumprelu_theta"]))[0].tolist() == g["jumprelu_f"]
    assert O.sae_reconstruct(f, sae.W_dec, None).tolist() == g["xhat_f"]
    f2 = O.sae_edit(f, g["edit_idx"], g["edit_val"], g["edit_mode"])
    assert f2.tolist() == g["f_edit"]
    assert O.sae_reconstruct(f2, sae.W_dec, None).tolist() == g["xhat_f_edit"]
    app = _App(g["edit_idx"], g["edit_val"], g["edit_mode"], add_error=True)
    y, K2, n_act, _ = O.sae_row(h, z, sae, app)
    assert y.tolist() == g["out_with_error"] and K2.tolist() == g["topk"] and n_act == 3
    app.add_error = False
    assert O.sae_row(h, z, sae, app)[0].tolist() == g["out_without_error"]


def test_sae_preact_is_dgemm_and_identity_encoder():
    rng = np.random.default_rng(3)
    d, S, n = 48, 200, 5
    Wb = bf(rng.standard_normal((S, d)) / math.sqrt(d)); b = rng.standard_normal(S).astype(np.float32)
    X = O.bf16_to_f64(bf(rng.standard_normal((n, d))))
    Z = O.sae_preact(X, Wb, b)
    Wf = torch.from_numpy(Wb.view(np.int16)).view(torch.bfloat16).to(torch.float64)     # library conversion
    ref = (torch.from_numpy(X) @ Wf.T + torch.from_numpy(b.astype(np.float64))).numpy()
    assert np.allclose(Z, ref, rtol=1e-13, atol=1e-13)
    # term-by-term sum for one entry (catches a transposed operand)
    Wf = Wf.numpy()
    assert Z[2, 17] == pytest.approx(float(b[17]) + math.fsum(Wf[17, i] * X[2, i] for i in range(d)), rel=1e-13)
    # identity encoder [I; 0]: z_j = h_j for j < d, 0 beyond
    Wi = np.zeros((S, d)); Wi[:d] = np.eye(d)
    Zi = O.sae_preact(X, bf(Wi), np.zeros(S, dtype=np.float32))
    assert np.array_equal(Zi[:, :d], X) and not Zi[:, d:].any()
    # input centering subtracts b_dec before the encoder
    bd = rng.standard_normal(d).astype(np.float32)
    Zc = O.sae_preact(X, Wb, b, bd, center_input=True)
    assert np.allclose(Zc, O.sae_preact(X - bd.astype(np.float64), Wb, b), rtol=0, atol=1e-14)


def test_topk_brute_force_and_tie_rule():
    rng = np.random.default_rng(4)
    for n, k in [(6, 2), (7, 3), (8, 4), (9, 1)]:
        z = rng.standard_normal(n)
        K = O.topk_indices(z, k)
        best = max(itertools.combinations(range(n), k), key=lambda c: sum(z[list(c)]))
        assert sorted(K.tolist()) == sorted(best)
        assert list(z[K]) == sorted(z[K], reverse=True)
        assert z[K].min() >= np.delete(z, K).max()
    # ties: lower index wins and comes first
    z = np.array([1.0, 3.0, 3.0, 0.5, 3.0, 2.0])
    assert O.topk_indices(z, 2).tolist() == [1, 2]
    assert O.topk_indices(z, 4).tolist() == [1, 2, 4, 5]
    assert O.topk_indices(np.zeros(5), 3).tolist() == [0, 1, 2]
    # against a library selection on distinct values
    z = rng.standard_normal(5000)
    assert O.topk_indices(z, 40).tolist() == torch.topk(torch.from_numpy(z), 40).indices.tolist()


def test_topk_k_equals_d_sae_is_relu_and_negative_members_stay():
    rng = np.random.default_rng(5)
    z = rng.standard_normal(50)
    f_top, K = O.sae_activate(z, O.SAE_TOPK, k=50)
    f_relu, _ = O.sae_activate(z, O.SAE_RELU)
    assert np.array_equal(f_top, f_relu) and len(K) == 50
    z = np.array([-1.0, -3.0, -2.0])
    f, K = O.sae_activate(z, O.SAE_TOPK, k=2)
    assert K.tolist() == [0, 2] and not f.any()          # kept index, value ReLU'd to zero


def test_jumprelu_special_cases():
    rng = np.random.default_rng(6)
    z = rng.standard_normal(100)
    assert np.array_equal(O.sae_activate(z, O.SAE_JUMPRELU, theta=np.zeros(100))[0], np.maximum(z, 0))
    assert not O.sae_activate(z, O.SAE_JUMPRELU, theta=np.full(100, np.inf))[0].any()
    th = z.copy()                                          # strict: z == theta is inactive
    assert not O.sae_activate(z, O.SAE_JUMPRELU, theta=th)[0].any()


def _rand_sae(rng, d, S, act, k=0, b_dec=False):
    Wd = rng.standard_normal((S, d)); Wd /= np.linalg.norm(Wd, axis=1, keepdims=True)
    return _Sae(d_sae=S, act=act, k=k, W_enc=bf(rng.standard_normal((S, d)) / math.sqrt(d)),
                b_enc=(rng.standard_normal(S) * 0.02 - 0.1).astype(np.float32), W_dec=bf(Wd),
                theta=rng.uniform(0.05, 0.3, S).astype(np.float32) if act == O.SAE_JUMPRELU else None,
                b_dec=rng.standard_normal(d).astype(np.float32) if b_dec else None)


@pytest.mark.parametrize("act", [O.SAE_RELU, O.SAE_JUMPRELU, O.SAE_TOPK])
def test_no_edit_plus_error_reproduces_h(act):
    rng = np.random.default_rng(7)
    sae = _rand_sae(rng, 32, 256, act, k=8, b_dec=True)
    xb = bf(rng.standard_normal(32)); x = O.bf16_to_f64(xb)
    z = O.sae_preact(x, sae.W_enc, sae.b_enc)[0]
    y = O.sae_row(x, z, sae, _App(add_error=True))[0]
    assert np.allclose(y, x, rtol=0, atol=1e-14)
    assert np.array_equal(O.f64_to_bf16_bits(y), xb)
    assert np.array_equal(O.sae_row_delta(x, z, sae, _App(add_error=True)), x)      # delta form: exact


@pytest.mark.parametrize("act", [O.SAE_RELU, O.SAE_JUMPRELU, O.SAE_TOPK])
def test_single_clamp_moves_along_decoder_row_and_delta_form_agrees(act):
    rng = np.random.default_rng(8)
    sae = _rand_sae(rng, 32, 256, act, k=8)
    x = O.bf16_to_f64(bf(rng.standard_normal(32)))
    z = O.sae_preact(x, sae.W_enc, sae.b_enc)[0]
    f, K = O.sae_activate(z, act, 8, sae.theta)
    j_act = int(np.argmax(f)); j_off = int(np.argmin(z))
    Wd = O.bf16_to_f64(sae.W_dec)
    for j in (j_act, j_off):
        y = O.sae_row(x, z, sae, _App([j], [5.0], [O.EDIT_CLAMP]))[0]
        assert np.allclose(y - x, (5.0 - f[j]) * Wd[j], rtol=0, atol=1e-13)
    # ablating an inactive feature is the identity; ablating an active one removes f_j W_dec[j]
    assert np.allclose(O.sae_row(x, z, sae, _App([j_off], [0.0], [O.EDIT_ABLATE]))[0], x, atol=1e-14)
    y = O.sae_row(x, z, sae, _App([j_act], [0.0], [O.EDIT_ABLATE]))[0]
    assert np.allclose(y - x, -f[j_act] * Wd[j_act], rtol=0, atol=1e-13)
    # several edits (with a duplicate: the later entry wins); literal and delta forms agree
    app = _App([j_act, 3, j_off, 3], [2.0, 1.0, 4.0, 7.0], [0, 0, 0, 0])
    y_lit = O.sae_row(x, z, sae, app)[0]
    assert np.allclose(y_lit, O.sae_row_delta(x, z, sae, app), rtol=0, atol=1e-12)
    want = x + (2.0 - f[j_act]) * Wd[j_act] + (7.0 - f[3]) * Wd[3] + (4.0 - f[j_off]) * Wd[j_off]
    assert np.allclose(y_lit, want, rtol=0, atol=1e-12)


def test_identity_sae_without_error_is_relu_of_h_and_jumprelu_inf_gives_b_dec():
    rng = np.random.default_rng(9)
    d, S = 16, 40
    I = np.zeros((S, d)); I[:d] = np.eye(d)
    xb = bf(rng.standard_normal(d)); x = O.bf16_to_f64(xb)
    sae = _Sae(d_sae=S, act=O.SAE_RELU, W_enc=bf(I), b_enc=np.zeros(S, dtype=np.float32), W_dec=bf(I))
    z = O.sae_preact(x, sae.W_enc, sae.b_enc)[0]
    assert np.array_equal(O.sae_row(x, z, sae, _App(add_error=False))[0], np.maximum(x, 0))
    # TopK over the identity encoder picks the row's own largest coordinates
    sae_k = _Sae(d_sae=S, act=O.SAE_TOPK, k=3, W_enc=bf(I), b_enc=np.zeros(S, dtype=np.float32), W_dec=bf(I))
    K = O.sae_row(x, z, sae_k, _App(add_error=False))[1]
    assert K.tolist() == torch.topk(torch.from_numpy(z), 3).indices.tolist()
    bd = rng.standard_normal(d).astype(np.float32)
    sae_j = _Sae(d_sae=S, act=O.SAE_JUMPRELU, W_enc=bf(I), b_enc=np.zeros(S, dtype=np.float32), W_dec=bf(I),
                 theta=np.full(S, np.inf, dtype=np.float32), b_dec=bd)
    assert np.array_equal(O.sae_row(x, z, sae_j, _App(add_error=False))[0], bd.astype(np.float64))
    assert np.allclose(O.sae_row(x, z, sae_j, _App(add_error=True))[0], x, atol=1e-15)


# ------------------------------------------------------------------ whole hook
def test_hook_passthrough_routing_and_invariants():
    w = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=11))
    res = O.apply_hook(w, keep_z=True)
    hidden = w.hidden
    for t in range(w.T_max):
        s = w.token_slot[t]
        if s < 0:
            assert res.kind[t] == 0 and not res.modified[t] and np.array_equal(res.out_bits[t], hidden[t])
            assert t not in res.scores
        elif s == 0:
            assert t in res.scores and np.array_equal(res.out_bits[t], hidden[t])
        elif s == 1:
            v = O.bf16_to_f64(w.apps[1].v)
            assert np.array_equal(res.y[t], O.bf16_to_f64(hidden[t]) + 4.0 * v)
        else:
            assert res.modified[t] and len(res.topk[t]) == 8
            z = res.z[t]; K = res.topk[t]
            assert z[K].min() >= np.delete(z, K).max()
    # rows beyond T_live are pass-through whatever the map says
    w2 = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=11)); w2.T_live = 20
    r2 = O.apply_hook(w2)
    assert all(r2.kind[t] == 0 for t in range(20, 48))
    assert all(np.array_equal(r2.out_bits[t], res.out_bits[t]) for t in range(20))
    # invalid / unregistered slot ids are pass-through
    w3 = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=11))
    w3.token_slot[:] = np.where(w3.token_slot == 0, 7, w3.token_slot)       # slot 7: never registered
    w3.token_slot[0] = 1000; w3.token_slot[1] = -5
    r3 = O.apply_hook(w3)
    assert all(r3.kind[t] == 0 for t in range(48) if w3.token_slot[t] in (7, 1000, -5))


def test_hook_permutation_and_relabel_equivariance_and_row_subset():
    w = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=12))
    base = O.apply_hook(w)
    rng = np.random.default_rng(0)
    perm = rng.permutation(48)
    wp = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=12))
    wp.hidden = w.hidden[perm].copy(); wp.token_slot = w.token_slot[perm].copy()
    rp = O.apply_hook(wp)
    for i, t in enumerate(perm):
        assert np.array_equal(rp.out_bits[i], base.out_bits[int(t)])
        assert (i in rp.scores) == (int(t) in base.scores)
        if i in rp.scores:
            assert np.array_equal(rp.scores[i], base.scores[int(t)])
    # relabel slots 0<->5 and 2<->6
    wr = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=12))
    remap = {0: 5, 1: 1, 2: 6, 3: 3, -1: -1}
    wr.apps = {remap[s]: a for s, a in w.apps.items()}
    wr.token_slot = np.array([remap[int(s)] for s in w.token_slot], dtype=np.int32)
    rr = O.apply_hook(wr)
    assert all(np.array_equal(rr.out_bits[t], base.out_bits[t]) for t in range(48))
    # a row subset gives the same rows (rows are independent)
    sub = O.apply_hook(w, rows=[3, 17, 40])
    assert all(np.array_equal(sub.out_bits[t], base.out_bits[t]) for t in (3, 17, 40)) and len(sub.y) == 3


def test_hook_all_unhooked_is_identity_and_topk_override():
    w = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=13))
    w0 = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=13)); w0.token_slot[:] = -1
    r0 = O.apply_hook(w0)
    assert all(np.array_equal(r0.out_bits[t], w.hidden[t]) for t in range(48)) and not r0.scores
    t = int(np.nonzero(w.token_slot == 2)[0][0])
    r = O.apply_hook(w, rows=[t], keep_z=True)
    K = r.topk[t].copy()
    other = int(np.setdiff1d(np.argsort(-r.z[t])[:9], K)[0])        # the 9th largest
    K2 = K.copy(); K2[-1] = other
    r_over = O.apply_hook(w, rows=[t], topk_override={t: K2})
    assert r_over.topk[t].tolist() == K2.tolist()


# ------------------------------------------------------------------ activation-driven gates
def test_gate_closed_form_cases():
    sc = np.array([[0.0, -1.0], [0.5, 2.0], [np.nan, 0.5], [0.5, 0.5]], dtype=np.float32)
    G = lambda col, cmp, thr: W.Gate(sc, col, cmp, thr)
    assert [O.gate_open(G(0, O.GATE_GE, 0.5), t) for t in range(4)] == [False, True, False, True]
    assert [O.gate_open(G(0, O.GATE_LT, 0.5), t) for t in range(4)] == [True, False, False, False]   # NaN fails both
    assert [O.gate_open(G(1, O.GATE_GE, 0.5), t) for t in range(4)] == [False, True, True, True]     # == threshold: GE open
    assert all(O.gate_open(G(1, O.GATE_GE, -np.inf), t) for t in range(4))
    assert not any(O.gate_open(G(1, O.GATE_GE, np.inf), t) for t in range(4))


def test_gated_hook_limits_and_complement():
    w = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=14))
    base = O.apply_hook(w)
    rng = np.random.default_rng(3)
    sc = rng.standard_normal((48, 2)).astype(np.float32)

    def run(cmp, thr):
        wg = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=14))
        for a in wg.apps.values():
            a.gate = W.Gate(sc, 1, cmp, thr)
        return O.apply_hook(wg)

    always, never = run(O.GATE_GE, -np.inf), run(O.GATE_GE, np.inf)
    ge, lt = run(O.GATE_GE, 0.1), run(O.GATE_LT, 0.1)
    for t in range(48):
        assert np.array_equal(always.out_bits[t], base.out_bits[t]) and (t in always.scores) == (t in base.scores)
        assert never.kind[t] == 0 and np.array_equal(never.out_bits[t], w.hidden[t]) and t not in never.scores
        # the two comparisons split the hooked rows between them
        assert (ge.kind[t] != 0) + (lt.kind[t] != 0) == (base.kind[t] != 0)
        src = ge if sc[t, 1] >= np.float32(0.1) else lt
        assert np.array_equal(src.out_bits[t], base.out_bits[t])


# ------------------------------------------------------------------ directional ablation
def test_project_hand_worked_and_invariants():
    g = GOLD["project"]; h = np.array(GOLD["h"]); r = np.array(g["r"])
    assert float(h @ r) == g["dot"]
    assert O.project(h, r, g["beta"]).tolist() == g["out"]
    assert O.project(h, r, 0.5).tolist() == g["beta_half_out"]
    rng = np.random.default_rng(21)
    h = rng.standard_normal(48); r = rng.standard_normal(48); r /= np.linalg.norm(r)
    y = O.project(h, r, 1.0)
    assert abs(y @ r) < 1e-14                                      # nothing left along r
    assert np.allclose(O.project(y, r, 1.0), y, rtol=0, atol=1e-14)   # idempotent
    assert np.array_equal(O.project(h, r, 0.0), h)
    assert np.allclose(h - y, (h @ r) * r, rtol=0, atol=1e-15)     # what was removed is parallel to r
    e = np.zeros(48); e[9] = 1.0
    out = O.project(h, e, 0.25)
    assert out[9] == h[9] * 0.75 and np.array_equal(np.delete(out, 9), np.delete(h, 9))
    # through the hook
    w = W.host(W.make_tiny(d=64, T=48, d_sae=256, k=8, seed=15))
    rv = bf(rng.standard_normal(64) / 8.0)
    w.apps[1] = W.Project(rv, 1.0)
    res = O.apply_hook(w)
    for t in np.nonzero(w.token_slot == 1)[0]:
        hh = O.bf16_to_f64(w.hidden[t]); rr = O.bf16_to_f64(rv)
        assert np.array_equal(res.y[int(t)], hh - (hh @ rr) * rr) and res.kind[int(t)] == O.KIND_PROJECT


# ------------------------------------------------------------------ router-logit steering
def test_router_hook_adds_delta_only_where_the_app_is():
    rng = np.random.default_rng(31)
    T, E = 12, 8
    logits = rng.standard_normal((T, E)).astype(np.float32)
    delta = np.array([0, 1.5, -np.inf, 0, 0, np.inf, -2.0, 0], dtype=np.float32)
    slots = np.array([0, -1, 1, 0, 2, 0, -1, 1, 0, 0, 5, 0], dtype=np.int32)
    apps = {0: W.Router(delta), 1: W.Steer(bf(np.zeros(4)), 1.0), 2: W.Router(np.zeros(4, dtype=np.float32))}
    w = W.Workload("r", 4, T, 10, bf(np.zeros((T, 4))), slots, apps, {}, n_slots_max=4)
    out = O.apply_router_hook(w, logits)
    for t in range(T):
        hit = t < 10 and slots[t] == 0
        want = logits[t].astype(np.float64) + (delta.astype(np.float64) if hit else 0.0)
        assert np.array_equal(out[t], want), t            # other kinds, other widths, rows past T_live: untouched
    assert out[0, 2] == -np.inf and out[0, 5] == np.inf    # forced out / forced in
    # the hidden-state hook ignores router apps
    r = O.apply_hook(w)
    assert all(r.kind[t] == 0 for t in range(T) if slots[t] in (0, 2))
    # gated
    sc = np.where(np.arange(T) % 2 == 0, 1.0, -1.0).astype(np.float32)[:, None]
    apps[0].gate = W.Gate(sc, 0, O.GATE_GE, 0.0)
    out = O.apply_router_hook(w, logits)
    assert np.array_equal(out[3], logits[3].astype(np.float64)) and out[8, 1] == np.float64(logits[8, 1]) + 1.5
