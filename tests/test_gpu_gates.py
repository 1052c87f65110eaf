"""Activation-gated conditional writes on the GPU (a score buffer decides, per row, on the device,
whether a later app runs) against the oracle."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

from parity import CANARY_F32, check_parity, oracle_edit_hint, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gate_scores(T, seed, stride=3):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    sc = torch.randn((T, stride), generator=g, device=DEV, dtype=torch.float32)
    sc[::17, 1] = float("nan")                      # NaN closes the gate
    sc[5::19, 1] = 0.25                             # exactly the threshold: >= opens, < stays closed
    return sc


@pytest.mark.parametrize("graph", [False, True])
@pytest.mark.parametrize("cmp", [W.GATE_GE, W.GATE_LT])
def test_tiny_every_app_gated_on_a_given_buffer(graph, cmp):
    w = W.make_tiny(DEV)
    sc = _gate_scores(w.T_max, 31)
    for a in w.apps.values():
        a.gate = W.Gate(sc, 1, cmp, 0.25)
    out = run_gpu(w, graph=graph)
    wh = W.host(w)
    check_parity(wh, out)
    ref = O.apply_hook(wh)
    closed = [t for t in range(w.T_max) if w.token_slot[t] >= 0 and ref.kind[t] == 0]
    assert len(closed) > 5 and all(np.array_equal(out["hidden"][t], wh.hidden[t]) for t in closed)


def test_gates_in_the_large_batch_kernel_and_sae_routing():
    w = W.make_mixed(DEV, d=320, T=2601, R=48, d_sae=1024, cap=300, mu=4.0, edit_hint=oracle_edit_hint)
    sc = _gate_scores(w.T_max, 32)
    for s, a in w.apps.items():
        if s % 2 == 0:                              # half of the slots, of every kind
            a.gate = W.Gate(sc, 1, W.GATE_GE, 0.25)
    out = run_gpu(w)
    check_parity(W.host(w), out)


def test_two_hooks_in_one_graph_probe_at_layer_a_gates_steering_at_layer_b():
    """The paper's conditional-write example: a probe read at one layer, a write at a later layer
    gated on `probe >= 0`, with no host involvement in between (both calls in one graph)."""
    import paper_2607_22595_b200 as mixlib
    d, T = 512, 192
    g = torch.Generator(device=DEV); g.manual_seed(41)
    hA = torch.randn((T, d), generator=g, device=DEV).to(torch.bfloat16)       # hidden at layer A
    hB = torch.randn((T, d), generator=g, device=DEV).to(torch.bfloat16)       # hidden at layer B
    Wp = (torch.randn((1, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16)
    v = torch.randn((d,), generator=g, device=DEV).to(torch.bfloat16)
    token_slot = np.where(np.arange(T) % 5 == 0, -1, 0).astype(np.int32)
    mA = mixlib.Mix(d_model=d, T_max=T, n_slots_max=1)
    mB = mixlib.Mix(d_model=d, T_max=T, n_slots_max=1)
    mA.register_probe(0, Wp, None, mixlib.MIX_ACT_NONE)                         # raw logit
    mB.register_steer(0, v, 3.0)
    scores = torch.from_numpy(np.full((T, 1), CANARY_F32, dtype=np.uint32).view(np.float32)).to(DEV)
    mB.set_gate(0, scores, 0, mixlib.MIX_GATE_GE, 0.0)
    mA.set_slot_map(token_slot); mB.set_slot_map(token_slot)
    hA_s, hB_s = hA.clone(), hB.clone()
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        mA.apply(hA_s, scores, stream=s); mB.apply(hB_s, None, stream=s)
        hB_s.copy_(hB)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=s):
            mA.apply(hA_s, scores, stream=s)
            mB.apply(hB_s, None, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    gr.replay(); torch.cuda.synchronize()
    # oracle: its own float64 probe at layer A, rounded to fp32, then the gated write at layer B
    wA = W.Workload("A", d, T, T, hA, token_slot, {0: W.Probe(Wp, None, W.ACT_NONE)}, {}, n_slots_max=1)
    refA = O.apply_hook(W.host(wA))
    sc_ref = np.zeros((T, 1), dtype=np.float32)
    for t, z in refA.scores.items():
        sc_ref[t, 0] = np.float32(z[0])
    wB = W.Workload("B", d, T, T, hB, token_slot,
                    {0: W.Steer(v, 3.0, gate=W.Gate(sc_ref, 0, W.GATE_GE, 0.0))}, {}, n_slots_max=1)
    whB = W.host(wB)
    refB = O.apply_hook(whB)
    got = W.bits(hB_s)
    sc_gpu = scores.cpu().numpy()
    hmax = float(hB.float().abs().max())
    n_steered = n_near = 0
    for t in range(T):
        if token_slot[t] < 0:
            assert np.array_equal(got[t], whB.hidden[t]) and sc_gpu.view(np.uint32)[t, 0] == CANARY_F32
            continue
        assert abs(sc_gpu[t, 0] - sc_ref[t, 0]) <= 1e-3 * abs(sc_ref[t, 0]) + 1e-6
        steered = O.bf16_to_f64(got[t])
        untouched = np.array_equal(got[t], whB.hidden[t])
        if abs(sc_ref[t, 0]) < 1e-4:                # the two sides may round the logit to either side of 0
            n_near += 1
            y = O.steer(O.bf16_to_f64(whB.hidden[t]), O.bf16_to_f64(W.bits(v)), 3.0)
            assert untouched or np.abs(steered - y).max() <= 1e-2 * hmax
        elif refB.kind[t] == 0:
            assert untouched, "row %d: gate is closed in the oracle but the GPU wrote the row" % t
        else:
            n_steered += 1
            assert np.abs(steered - refB.y[t]).max() <= 1e-2 * hmax
    assert n_steered > 30 and n_near < 5
    assert mA.get_status() == 0 and mB.get_status() == 0


def test_gate_toggles_without_recapture_and_api_errors():
    import paper_2607_22595_b200 as mixlib
    w = W.make_tiny(DEV)
    m = W.make_context(mixlib.Mix, w)
    sc = _gate_scores(w.T_max, 33)
    h_static = w.hidden.clone()
    scores = torch.zeros((w.T_max, 1), dtype=torch.float32, device=DEV)
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h_static, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply(h_static, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)

    def replay_and_check():
        h_static.copy_(w.hidden)
        scores.copy_(torch.from_numpy(np.full((w.T_max, 1), CANARY_F32, dtype=np.uint32).view(np.float32)))
        g.replay(); torch.cuda.synchronize()
        out = dict(hidden=W.bits(h_static), scores=scores.cpu().numpy(), status=m.get_status())
        check_parity(W.host(w), out, check_features=False)

    replay_and_check()
    w.apps[1].gate = W.Gate(sc, 0, W.GATE_LT, -0.3); m.set_gate(1, sc, 0, mixlib.MIX_GATE_LT, -0.3)
    w.apps[2].gate = W.Gate(sc, 2, W.GATE_GE, 0.4); m.set_gate(2, sc, 2, mixlib.MIX_GATE_GE, 0.4)
    replay_and_check()
    w.apps[1].gate = W.Gate(sc, 1, W.GATE_GE, 0.25); m.set_gate(1, sc, 1, mixlib.MIX_GATE_GE, 0.25)   # replace
    replay_and_check()
    w.apps[2].gate = None; m.set_gate(2, None)                                                       # remove
    replay_and_check()
    with pytest.raises(mixlib.MixError) as e:
        m.set_gate(6, sc)                               # slot 6 has no app
    assert e.value.code == -1
    with pytest.raises(mixlib.MixError) as e:
        m.set_gate(1, sc, column=3)                     # column outside the stride
    assert e.value.code == -1
    with pytest.raises(mixlib.MixError) as e:
        m.set_gate(1, sc, cmp=7)
    assert e.value.code == -1


def test_several_apps_on_the_same_rows_by_chaining_contexts_in_one_graph():
    """Composition of apps on one model instance: a probe, a steering vector and an SAE edit all act
    on the SAME token rows, as three hook contexts applied back to back inside one captured graph.
    The oracle applies the three hooks in the same order."""
    import paper_2607_22595_b200 as mixlib
    base = W.make_tiny(DEV)
    T, d = base.T_max, base.d_model
    rows = np.where(np.arange(T) % 3 != 0, 0, -1).astype(np.int32)          # two thirds of the rows, slot 0
    def ctx(app, groups=None):
        w = W.Workload("c", d, T, T, base.hidden, rows, {0: app}, groups or {}, n_slots_max=1,
                       n_groups_max=1 if groups else 0, C_max=1, k_max=base.k_max, r_max=base.r_max,
                       d_sae_max=base.d_sae_max if groups else 0)
        return w, W.make_context(mixlib.Mix, w)
    wP, mP = ctx(base.apps[0])
    wS, mS = ctx(base.apps[1])
    wE, mE = ctx(base.apps[2], {0: base.groups[0]})
    h = base.hidden.clone()
    scores = torch.from_numpy(np.full((T, 1), CANARY_F32, dtype=np.uint32).view(np.float32)).to(DEV)
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for m in (mP, mS, mE):
            m.apply(h, scores, stream=s)
        h.copy_(base.hidden)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            mP.apply(h, scores, stream=s)       # read first: the probe sees the unmodified row
            mS.apply(h, None, stream=s)
            mE.apply(h, None, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    g.replay(); torch.cuda.synchronize()
    # oracle, hook after hook (each stage's bf16 output is the next stage's input)
    whP = W.host(wP)
    rP = O.apply_hook(whP)
    whS = W.host(wS)
    rS = O.apply_hook(whS)
    whE = W.host(wE)
    whE.hidden = np.stack([rS.out_bits[t] for t in range(T)])
    rE = O.apply_hook(whE, keep_z=True)
    got = W.bits(h)
    hmax = float(np.abs(O.bf16_to_f64(whE.hidden)).max())
    sc = scores.cpu().numpy()
    for t in range(T):
        if rows[t] < 0:
            assert np.array_equal(got[t], whP.hidden[t]) and sc.view(np.uint32)[t, 0] == CANARY_F32
            continue
        assert abs(sc[t, 0] - rP.scores[t][0]) <= 1e-3 * abs(rP.scores[t][0])
        assert np.abs(O.bf16_to_f64(got[t]) - rE.y[t]).max() <= 1e-2 * hmax
    assert mP.get_status() == 0 and mS.get_status() == 0 and mE.get_status() == 0


def test_router_logit_steering_matches_oracle_and_leaves_hidden_alone():
    import paper_2607_22595_b200 as mixlib
    rng = np.random.default_rng(51)
    T, E, d = 300, 8, 128
    g = torch.Generator(device=DEV); g.manual_seed(51)
    hidden = torch.randn((T, d), generator=g, device=DEV).to(torch.bfloat16)
    logits = torch.randn((T, E), generator=g, device=DEV)
    d0 = torch.tensor([0, 1.5, float("-inf"), 0, 0, float("inf"), -2.0, 0.25], device=DEV)
    d1 = torch.randn(E, generator=g, device=DEV)
    v = torch.randn(d, generator=g, device=DEV).to(torch.bfloat16)
    sc = torch.randn((T, 1), generator=g, device=DEV)
    apps = {0: W.Router(d0), 1: W.Router(d1, gate=W.Gate(sc, 0, W.GATE_LT, 0.1)), 2: W.Steer(v, 2.0),
            3: W.Router(torch.zeros(16, device=DEV))}                       # 16 experts: not this tensor's width
    slots = rng.choice([-1, 0, 1, 2, 3, 7], size=T).astype(np.int32)
    w = W.Workload("router", d, T, 280, hidden, slots, apps, {}, n_slots_max=8)
    m = W.make_context(mixlib.Mix, w)
    lg, h = logits.clone(), hidden.clone()
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply_router(lg, stream=s); lg.copy_(logits)
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=s):
            m.apply_router(lg, stream=s)
            m.apply(h, None, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    gr.replay(); torch.cuda.synchronize()
    wh = W.host(w)
    want = O.apply_router_hook(wh, logits.cpu().numpy())
    got = lg.cpu().numpy().astype(np.float64)
    touched = 0
    for t in range(T):
        if np.array_equal(want[t], logits[t].cpu().numpy().astype(np.float64)):
            assert np.array_equal(lg[t].cpu().numpy().view(np.uint32), logits[t].cpu().numpy().view(np.uint32))   # bit-exact
        else:
            touched += 1
            fin = np.isfinite(want[t])
            assert np.array_equal(got[t][~fin], want[t][~fin])
            assert np.abs(got[t][fin] - want[t][fin]).max() <= 1e-6 * np.maximum(1.0, np.abs(want[t][fin])).max()
    assert touched > 40
    # the hidden-state hook saw the same map: steering rows changed, router rows did not
    out = dict(hidden=W.bits(h), scores=np.full((T, 1), 0, dtype=np.float32).view(np.uint32).view(np.float32),
               status=m.get_status())
    ref = O.apply_hook(wh)
    for t in range(T):
        if ref.kind[t] == 0:
            assert np.array_equal(out["hidden"][t], wh.hidden[t])
    assert out["status"] == mixlib.MIX_STATUS_BAD_SLOT              # slot 7 was never registered
