"""CPU pins of the oracle's slot chains (several apps on one row): hand-worked values, closed forms and
agreement with hook-after-hook application of the single-app oracle."""
import json
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked_chain_d4.json")))
ACT = {"none": O.ACT_NONE, "sigmoid": O.ACT_SIGMOID, "softmax": O.ACT_SOFTMAX}


def bf(a):
    return W.bits(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def _gold_workload(case):
    g = GOLD[case]
    T = 2
    apps, chains, groups = {}, {}, {}
    closed = np.full((T, 1), -1.0, dtype=np.float32)           # gate "score >= 0" is closed everywhere
    for i, a in enumerate(g["apps"]):
        gate = W.Gate(closed, 0, W.GATE_GE, 0.0) if a.get("gate_open") is False else None
        if a["kind"] == "probe":
            apps[i] = W.Probe(bf(a["W"]), np.asarray(a["b"], np.float32), ACT[a["act"]], gate=gate)
        elif a["kind"] == "steer":
            apps[i] = W.Steer(bf(a["v"]), a["alpha"], gate=gate)
        elif a["kind"] == "project":
            apps[i] = W.Project(bf(a["r"]), a["beta"], gate=gate)
        else:
            apps[i] = W.SaeApp(0, np.asarray(a["edit_idx"], np.int32), np.asarray(a["edit_val"], np.float32),
                               np.asarray(a["edit_mode"], np.uint8), a["add_error"], gate=gate)
            sw = g["sae"]
            groups[0] = W.SaeWeights(len(sw["W_enc"]), W.SAE_TOPK, sw["k"], bf(sw["W_enc"]),
                                     np.asarray(sw["b_enc"], np.float32), bf(sw["W_dec"]), None, None, False)
        if i + 1 < len(g["apps"]):
            chains[i] = i + 1
    hidden = np.stack([bf(GOLD["h"]), bf(GOLD["h"])])
    slot = np.array([0, -1], dtype=np.int32)                   # row 1 carries no app
    return W.Workload(case, 4, T, T, hidden, slot, apps, groups, n_slots_max=len(apps), n_groups_max=len(groups),
                      C_max=4, k_max=3, r_max=2, d_sae_max=6, chains=chains), g


@pytest.mark.parametrize("case", ["chain_read_write_read_write", "chain_steer_then_sae",
                                  "chain_closed_gate_keeps_columns"])
def test_chain_hand_worked(case):
    w, g = _gold_workload(case)
    r = O.apply_chain_hook(w)
    assert O.bf16_to_f64(r.out_bits[0]).tolist() == g["out"]
    want = {int(c): v for c, v in g.get("scores", {}).items()}
    assert set(r.scores[0]) == set(want)
    for c, v in want.items():
        assert r.scores[0][c] == pytest.approx(v, rel=0, abs=1e-15)
    if "topk" in g:
        assert list(r.topk[0]) == g["topk"]
    # the row without an app passes through
    assert np.array_equal(r.out_bits[1], w.hidden[1]) and not r.modified[1] and r.scores[1] == {}


def test_chain_of_one_equals_the_single_app_hook():
    w = W.host(W.make_tiny("cpu"))
    a = O.apply_hook(w)
    b = O.apply_chain_hook(w)
    for t in range(w.T_max):
        assert np.array_equal(a.out_bits[t], b.out_bits[t])
        if t in a.scores:
            assert [b.scores[t][c] for c in range(len(a.scores[t]))] == list(a.scores[t])
        if t in a.topk:
            assert np.array_equal(a.topk[t], b.topk[t])


def test_chain_equals_hook_after_hook():
    """A chain s0 -> s1 -> s2 gives, bit for bit, what three successive single-app hooks give when the
    bf16 output of one is the input of the next."""
    rng = np.random.default_rng(5)
    d, T = 64, 12
    g = torch.Generator().manual_seed(3)
    sae = W.make_sae_weights(g, "cpu", d, 256, W.SAE_TOPK, k=8)
    apps = {0: W.Probe(bf(rng.standard_normal((3, d))), rng.standard_normal(3).astype(np.float32), W.ACT_SOFTMAX),
            1: W.Steer(bf(rng.standard_normal(d)), 1.5),
            2: W.SaeApp(0, np.array([7, 100], np.int32), np.array([2.0, 0.0], np.float32), np.array([0, 1], np.uint8), True),
            3: W.Project(bf(rng.standard_normal(d) / 8.0), 1.0)}
    hidden = bf(rng.standard_normal((T, d)))
    slot = np.array([0, 1, 2, 3, -1, 0, 0, 1, 3, 2, -1, 0], dtype=np.int32)
    base = dict(d_model=d, T_max=T, T_live=T, n_slots_max=4, n_groups_max=1, C_max=3, k_max=8, r_max=2, d_sae_max=256)
    wc = W.host(W.Workload("c", hidden=hidden, token_slot=slot, apps=apps, groups={0: sae},
                           chains={0: 1, 1: 2, 3: 1}, **base))
    r = O.apply_chain_hook(wc)
    for t in range(T):
        cur = wc.hidden[t:t + 1].copy()
        scores = {}
        for sl in O.chain_slots(wc, int(slot[t])):
            w1 = W.Workload("s", d, 1, 1, cur, np.array([sl], np.int32), wc.apps, wc.groups, 4, 1, 3, 8, 2, 256)
            one = O.apply_hook(w1)
            cur = one.out_bits[0][None, :].copy()
            if 0 in one.scores:
                scores = {c: float(v) for c, v in enumerate(one.scores[0])}
        assert np.array_equal(r.out_bits[t], cur[0]), t
        assert r.scores[t] == scores, t                 # one probe per chain here: columns 0..2
    assert O.chain_slots(wc, 3) == [3, 1, 2] and O.chain_slots(wc, 2) == [2] and O.chain_slots(wc, -1) == []


def test_chain_closed_forms():
    d = 16
    e = np.zeros(d); e[3] = 1.0
    h = bf(np.arange(d, dtype=np.float32))[None, :]
    mk = lambda apps, chains: W.Workload("x", d, 1, 1, h, np.array([0], np.int32), apps, {}, n_slots_max=len(apps),
                                         C_max=2, chains=chains)
    # two steering vectors add up; order does not matter when everything is exact
    a = {0: W.Steer(bf(e), 2.0), 1: W.Steer(bf(np.ones(d)), -1.0)}
    r01 = O.apply_chain_hook(mk(a, {0: 1}))
    r10 = O.apply_chain_hook(mk({0: a[1], 1: a[0]}, {0: 1}))
    want = np.arange(d, dtype=np.float64) - 1.0; want[3] += 2.0
    assert O.bf16_to_f64(r01.out_bits[0]).tolist() == want.tolist() == O.bf16_to_f64(r10.out_bits[0]).tolist()
    # projecting a direction out and then probing along it reads exactly zero; probing first reads h.r
    p = {0: W.Project(bf(e), 1.0), 1: W.Probe(bf(e[None, :]), None, W.ACT_NONE)}
    assert O.apply_chain_hook(mk(p, {0: 1})).scores[0] == {0: 0.0}
    q = {0: p[1], 1: p[0]}
    assert O.apply_chain_hook(mk(q, {0: 1})).scores[0] == {0: 3.0}
    # steering twice with alpha and -alpha restores the row when no rounding intervenes
    s = {0: W.Steer(bf(np.ones(d)), 4.0), 1: W.Steer(bf(np.ones(d)), -4.0)}
    assert np.array_equal(O.apply_chain_hook(mk(s, {0: 1})).out_bits[0], h[0])
    # a chain is cut at MAX_CHAIN apps
    five = {i: W.Steer(bf(np.ones(d)), 1.0) for i in range(5)}
    r5 = O.apply_chain_hook(mk(five, {0: 1, 1: 2, 2: 3, 3: 4}))
    assert O.bf16_to_f64(r5.out_bits[0]).tolist() == (np.arange(d) + float(O.MAX_CHAIN)).tolist()
