"""Property tests of the oracle (hypothesis): algebraic facts that hold for every input."""
import numpy as np
import torch
from hypothesis import given, settings, strategies as st

import workloads as W
from oracle import mi_hook as O


def _bf(a):
    return W.bits(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


class _Sae:
    def __init__(self, **kw):
        self.theta = None; self.b_dec = None; self.center_input = False; self.k = 0
        self.__dict__.update(kw)


class _App:
    kind = O.KIND_SAE
    def __init__(self, idx=(), val=(), mode=(), add_error=True):
        self.edit_idx = np.asarray(idx, dtype=np.int32); self.edit_val = np.asarray(val, dtype=np.float32)
        self.edit_mode = np.asarray(mode, dtype=np.uint8); self.add_error = add_error; self.group = 0


@settings(max_examples=60, deadline=None)
@given(st.integers(0, 2 ** 32 - 1), st.integers(2, 40), st.integers(1, 12))
def test_topk_dominates_and_is_stable_under_permutation(seed, n, k):
    rng = np.random.default_rng(seed)
    k = min(k, n)
    z = np.round(rng.standard_normal(n), 1)            # rounding forces ties
    K = O.topk_indices(z, k)
    assert len(set(K.tolist())) == k
    assert z[K].min() >= np.delete(z, K).max(initial=-np.inf)
    assert all(z[K[i]] > z[K[i + 1]] or (z[K[i]] == z[K[i + 1]] and K[i] < K[i + 1]) for i in range(k - 1))
    # the multiset of selected values does not depend on where the entries sit
    perm = rng.permutation(n)
    assert sorted(z[perm][O.topk_indices(z[perm], k)].tolist()) == sorted(z[K].tolist())


@settings(max_examples=40, deadline=None)
@given(st.integers(0, 2 ** 32 - 1), st.sampled_from([O.SAE_RELU, O.SAE_JUMPRELU, O.SAE_TOPK]),
       st.integers(0, 5), st.booleans())
def test_literal_and_delta_forms_agree_and_noops_are_identities(seed, act, n_edit, with_b_dec):
    rng = np.random.default_rng(seed)
    d, S, k = 24, 96, 6
    Wd = rng.standard_normal((S, d)); Wd /= np.linalg.norm(Wd, axis=1, keepdims=True)
    sae = _Sae(d_sae=S, act=act, k=k, W_enc=_bf(rng.standard_normal((S, d)) / np.sqrt(d)),
               b_enc=(rng.standard_normal(S) * 0.1).astype(np.float32), W_dec=_bf(Wd),
               theta=rng.uniform(0, 0.3, S).astype(np.float32) if act == O.SAE_JUMPRELU else None,
               b_dec=rng.standard_normal(d).astype(np.float32) if with_b_dec else None)
    x = O.bf16_to_f64(_bf(rng.standard_normal(d)))
    z = O.sae_preact(x, sae.W_enc, sae.b_enc)[0]
    idx = rng.integers(0, S, n_edit); mode = rng.integers(0, 2, n_edit); val = rng.uniform(-3, 3, n_edit)
    app = _App(idx, val, mode, add_error=True)
    y = O.sae_row(x, z, sae, app)[0]
    assert np.allclose(y, O.sae_row_delta(x, z, sae, app), rtol=0, atol=1e-11)
    # edits that restore the current value change nothing
    f, _ = O.sae_activate(z, act, k, sae.theta)
    same = _App(idx, np.float32(f[idx]) if n_edit else [], np.zeros(n_edit, dtype=np.uint8), add_error=True)
    if n_edit and np.array_equal(np.float32(f[idx]).astype(np.float64), f[idx]):
        assert np.allclose(O.sae_row(x, z, sae, same)[0], x, rtol=0, atol=1e-12)
    # without the error term the output is a reconstruction: independent of x given f'
    app.add_error = False
    y2 = O.sae_row(x, z, sae, app)[0]
    f2 = O.sae_edit(f, idx, val, mode)
    assert np.allclose(y2, O.sae_reconstruct(f2, sae.W_dec, sae.b_dec), rtol=0, atol=1e-12)


@settings(max_examples=40, deadline=None)
@given(st.integers(0, 2 ** 32 - 1), st.floats(-8, 8, width=32), st.floats(-8, 8, width=32))
def test_steering_is_additive_and_projection_is_linear(seed, a, b):
    rng = np.random.default_rng(seed)
    h, g, v = rng.standard_normal(32), rng.standard_normal(32), rng.standard_normal(32)
    r = rng.standard_normal(32); r /= np.linalg.norm(r)
    assert np.allclose(O.steer(O.steer(h, v, a), v, b), O.steer(h, v, 0.0) + (float(np.float32(a)) + float(np.float32(b))) * v,
                       rtol=0, atol=1e-12)
    assert np.allclose(O.project(h + g, r, 1.0), O.project(h, r, 1.0) + O.project(g, r, 1.0), rtol=0, atol=1e-12)
    assert np.allclose(O.project(h, r, a) @ r, (1 - float(np.float32(a))) * (h @ r), rtol=0, atol=1e-12)


@settings(max_examples=200, deadline=None)
@given(st.floats(allow_nan=False, allow_infinity=False, width=32))
def test_bf16_rounding_is_nearest_and_monotone(x):
    bits = O.f64_to_bf16_bits(np.array([float(x)]))
    y = float(O.bf16_to_f64(bits)[0])
    if np.isfinite(y):
        up = float(O.bf16_to_f64(np.array([(int(bits[0]) + 1) & 0xFFFF], dtype=np.uint16))[0])
        dn = float(O.bf16_to_f64(np.array([(int(bits[0]) - 1) & 0xFFFF], dtype=np.uint16))[0])
        for nb in (up, dn):
            if np.isfinite(nb) and (nb > 0) == (y > 0) and y != 0:
                assert abs(y - x) <= abs(nb - x) + 0.0        # no neighbour is closer


@settings(max_examples=40, deadline=None)
@given(st.integers(0, 2 ** 32 - 1), st.integers(1, 4), st.booleans())
def test_chain_is_hook_after_hook_and_commutes_with_row_permutation(seed, length, with_gate):
    """Random chains of read / write apps: the chained hook equals the single-app hook applied once per app to
    the bf16 output of the previous one; probe columns follow the static layout; permuting the rows permutes
    the results."""
    rng = np.random.default_rng(seed)
    d, T = 32, 9
    apps, chains, cols = {}, {}, []
    C_total = 0
    for s in range(length):
        kind = int(rng.integers(0, 3))
        if kind == 0:
            C = int(rng.integers(1, 4))
            apps[s] = W.Probe(_bf(rng.standard_normal((C, d))), rng.standard_normal(C).astype(np.float32),
                              W.ACT_SOFTMAX if C > 1 else W.ACT_SIGMOID)
            cols.append((s, C_total, C)); C_total += C
        elif kind == 1:
            apps[s] = W.Steer(_bf(rng.standard_normal(d)), float(np.float32(rng.uniform(-3, 3))))
        else:
            r = rng.standard_normal(d); apps[s] = W.Project(_bf(r / np.linalg.norm(r)), 1.0)
        if s + 1 < length:
            chains[s] = s + 1
    hidden = _bf(rng.standard_normal((T, d)))
    if with_gate:
        sc = rng.standard_normal((T, 1)).astype(np.float32)
        apps[0].gate = W.Gate(sc, 0, W.GATE_GE, 0.0)
    slot = np.where(rng.random(T) < 0.7, 0, -1).astype(np.int32)
    w = W.Workload("c", d, T, T, hidden, slot, apps, {}, n_slots_max=length, C_max=max(C_total, 1), chains=chains)
    r = O.apply_chain_hook(w)
    for t in range(T):
        cur = hidden[t:t + 1].copy()
        want_scores = {}
        if slot[t] == 0:
            for s in range(length):
                one_apps = {0: apps[s]}
                if getattr(apps[s], "gate", None) is not None:       # the gate indexes rows of the full batch
                    if not O.gate_open(apps[s].gate, t):
                        continue
                    import copy
                    a2 = copy.copy(apps[s]); a2.gate = None
                    one_apps = {0: a2}
                w1 = W.Workload("s", d, 1, 1, cur, np.array([0], np.int32), one_apps, {}, n_slots_max=1, C_max=4)
                one = O.apply_hook(w1)
                cur = one.out_bits[0][None, :].copy()
                if 0 in one.scores:
                    c0 = [c for (ss, c, n) in cols if ss == s][0]
                    for j, v in enumerate(one.scores[0]):
                        want_scores[c0 + j] = float(v)
        assert np.array_equal(r.out_bits[t], cur[0])
        assert r.scores[t] == want_scores
    perm = rng.permutation(T)
    wp = W.Workload("p", d, T, T, hidden[perm], slot[perm], apps, {}, n_slots_max=length, C_max=max(C_total, 1), chains=chains)
    if with_gate:
        import copy
        apps_p = dict(apps); g0 = copy.copy(apps[0]); g0.gate = W.Gate(sc[perm], 0, W.GATE_GE, 0.0); apps_p[0] = g0
        wp.apps = apps_p
    rp = O.apply_chain_hook(wp)
    for i, t in enumerate(perm):
        assert np.array_equal(rp.out_bits[i], r.out_bits[int(t)]) and rp.scores[i] == r.scores[int(t)]
