"""GPU: slot chains (several apps applied in order to one row in one mix_apply) against the oracle and,
bit for bit, against the same apps applied by separate calls."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

from parity import CANARY_F32, CANARY_I32, HIDDEN_TOL_FRAC, TOPK_TIE_TOL, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"
SCORE_TOL = 2e-3        # a probe behind a write inherits the +-1 bf16 ulp the written row may differ by


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


def check_chain_parity(wh, out, scale_with_output=False, expect_status=0):
    ref = O.apply_chain_hook(wh)
    hmax = float(np.abs(O.bf16_to_f64(wh.hidden)).max())
    if scale_with_output:      # an app's output may dwarf the hidden state (see parity.check_parity)
        hmax = max([hmax] + [float(np.abs(ref.y[t]).max()) for t in range(wh.T_max) if ref.modified[t]])
    sb = out["scores"].view(np.uint32)
    redo = {}
    for t in range(wh.T_max):
        if t in ref.topk:                         # TopK ids: equal up to near-ties at the k-th value
            K_ref, k = ref.topk[t], len(ref.topk[t])
            K_gpu = out["topk_idx"][t, :k].astype(np.int64)
            if set(K_gpu.tolist()) != set(K_ref.tolist()):
                redo[t] = K_gpu
    if redo:
        ref2 = O.apply_chain_hook(wh, list(redo), topk_override=redo)
        for t in redo:
            assert np.abs(ref2.y[t] - ref.y[t]).max() <= 10 * TOPK_TIE_TOL * max(1.0, hmax), "row %d: not a near-tie" % t
            ref.y[t], ref.n_active[t] = ref2.y[t], ref2.n_active[t]
    n_mod = n_scores = 0
    for t in range(wh.T_max):
        if not ref.modified[t]:
            assert np.array_equal(out["hidden"][t], wh.hidden[t]), "row %d must be bit-identical" % t
        else:
            err = np.abs(O.bf16_to_f64(out["hidden"][t]) - ref.y[t]).max()
            assert err <= HIDDEN_TOL_FRAC * hmax, "row %d hidden off by %g" % (t, err)
            n_mod += 1
        cols = ref.scores[t]
        for c in range(out["scores"].shape[1]):
            if c in cols:
                got = float(out["scores"][t, c])
                assert abs(got - cols[c]) <= SCORE_TOL * max(1.0, abs(cols[c])), "row %d col %d: %g vs %g" % (t, c, got, cols[c])
                n_scores += 1
            else:
                assert sb[t, c] == CANARY_F32, "row %d col %d was written" % (t, c)
        if t in ref.n_active and t in ref.topk:
            assert int(out["n_active"][t]) == ref.n_active[t]
        elif t not in ref.n_active:
            assert int(out["n_active"][t]) == int(CANARY_I32)
    if expect_status is not None:
        assert out["status"] == expect_status
    return dict(modified=n_mod, scores=n_scores, swaps=len(redo))


@pytest.mark.parametrize("graph", [False, True])
def test_chained_workload_matches_oracle(graph):
    w = W.make_chained(DEV)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_SLOT_CHAINS, graph=graph)
    st = check_chain_parity(W.host(w), out)
    assert st["modified"] > 150 and st["scores"] > 300


def test_chained_large_batch_and_conditional_graph():
    # T_max above the one-CTA-per-row limit of the unchained kernels; SAE chain inside a graph IF node
    w = W.make_chained(DEV, T=2600, d=320, d_sae=1024, k=8, C=7)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_SLOT_CHAINS, graph=True, conditional=True)
    check_chain_parity(W.host(w), out)


def test_chain_equals_separate_calls_bit_for_bit():
    """chain 0 -> 1 -> 2 -> 3 in one call == four contexts, one app each, applied one after the other."""
    mixlib = _mixlib()
    w = W.make_chained(DEV)
    slot = np.where(np.arange(w.T_max) % 3 == 0, -1, 0).astype(np.int32)       # two thirds of the rows start chain 0
    wc = W.Workload("c", w.d_model, w.T_max, w.T_max, w.hidden, slot, w.apps, w.groups, w.n_slots_max, w.n_groups_max,
                    w.C_max, w.k_max, w.r_max, w.d_sae_max, chains=w.chains)
    a = run_gpu(wc, flags=mixlib.MIX_FLAG_SLOT_CHAINS)
    h = w.hidden.clone()
    C = w.C_max
    scores = torch.from_numpy(np.full((w.T_max, C), CANARY_F32, dtype=np.uint32).view(np.float32)).cuda()
    col = 0
    for s in O.chain_slots(W.host(wc), 0):
        app = w.apps[s]
        one = W.Workload("one", w.d_model, w.T_max, w.T_max, h, slot.copy(), {0: app},
                         w.groups if app.kind == W.KIND_SAE else {}, n_slots_max=1,
                         n_groups_max=w.n_groups_max if app.kind == W.KIND_SAE else 0, C_max=C, k_max=w.k_max,
                         r_max=w.r_max, d_sae_max=w.d_sae_max)
        m = W.make_context(mixlib.Mix, one)
        sc = torch.zeros((w.T_max, C), dtype=torch.float32, device=DEV)
        m.apply(h, sc)
        torch.cuda.synchronize()
        if app.kind == W.KIND_PROBE:
            n = app.W.shape[0]
            rows = torch.from_numpy(slot == 0).cuda()
            scores[rows, col:col + n] = sc[rows, :n]
            col += n
        assert m.get_status() == 0
        m.destroy()
    assert np.array_equal(a["hidden"], W.bits(h))
    got, want = a["scores"], scores.cpu().numpy()
    assert np.array_equal(got.view(np.uint32) == CANARY_F32, want.view(np.uint32) == CANARY_F32)
    live = want.view(np.uint32) != CANARY_F32
    # the probes run in different kernels (different summation order): equal to rounding, not bitwise
    assert np.abs(got[live] - want[live]).max() <= 1e-5


def test_chain_links_can_change_between_replays():
    mixlib = _mixlib()
    w = W.make_chained(DEV)
    m = W.make_context(mixlib.Mix, w, flags=mixlib.MIX_FLAG_SLOT_CHAINS)
    out = run_gpu(w, mix=m, graph=True)
    check_chain_parity(W.host(w), out)
    # cut chain 0 after its steering app, and let the projection run alone
    m.set_chain(1, -1)
    m.set_chain(4, -1)
    w2 = W.Workload(w.name, w.d_model, w.T_max, w.T_live, w.hidden, w.token_slot, w.apps, w.groups, w.n_slots_max,
                    w.n_groups_max, w.C_max, w.k_max, w.r_max, w.d_sae_max, chains={0: 1, 2: 3, 6: 1})
    out2 = run_gpu(w2, mix=m, graph=True)
    check_chain_parity(W.host(w2), out2)
    m.destroy()


def test_set_chain_error_codes():
    mixlib = _mixlib()
    w = W.make_chained(DEV)
    plain = W.make_context(mixlib.Mix, W.Workload(w.name, w.d_model, w.T_max, w.T_live, w.hidden, w.token_slot, w.apps,
                                                  w.groups, w.n_slots_max, w.n_groups_max, w.C_max, w.k_max, w.r_max,
                                                  w.d_sae_max))
    with pytest.raises(mixlib.MixError) as e:
        plain.set_chain(0, 1)                                  # context created without the flag
    assert e.value.code == -1
    plain.destroy()
    m = W.make_context(mixlib.Mix, w, flags=mixlib.MIX_FLAG_SLOT_CHAINS)
    for bad in [(3, 0),       # an SAE app can only end a chain
                (2, 0),       # cycle 0 -> 1 -> 2 -> 0
                (7, 0),       # 7 -> 0 -> 1 -> 2 -> 3: five apps
                (7, 7)]:      # a slot cannot follow itself
        with pytest.raises(mixlib.MixError) as e:
            m.set_chain(*bad)
        assert e.value.code == -1, bad
    with pytest.raises(mixlib.MixError) as e:
        m.set_chain(0, 99)
    assert e.value.code == -2
    # class columns: chain 0 -> 1 -> 2 writes 1 + 5 of the C_max = 7 columns; a 7-class probe in slot 2
    # is fine on its own but no longer fits behind the probe of slot 0
    g = torch.Generator(device=DEV); g.manual_seed(1)
    wide = torch.randn((7, w.d_model), generator=g, device=DEV).to(torch.bfloat16)
    with pytest.raises(mixlib.MixError) as e:
        m.register_probe(2, wide, None, mixlib.MIX_ACT_SOFTMAX)
    assert e.value.code == -1
    # the failed calls changed nothing: the original chains still give the oracle's result
    out = run_gpu(w, mix=m)
    check_chain_parity(W.host(w), out)
    # unregistering a slot removes the links that point to it
    m.unregister_app(1)
    w4 = W.Workload(w.name, w.d_model, w.T_max, w.T_live, w.hidden, w.token_slot,
                    {s: a for s, a in w.apps.items() if s != 1}, w.groups, w.n_slots_max, w.n_groups_max, w.C_max,
                    w.k_max, w.r_max, w.d_sae_max, chains={2: 3, 4: 5})
    out = run_gpu(w4, mix=m)
    ref_rows_slot1 = np.nonzero(w.token_slot[:w.T_live] == 1)[0]
    assert np.array_equal(out["hidden"][ref_rows_slot1], W.bits(w.hidden)[ref_rows_slot1])
    m.destroy()


# ------------------------------------------------------------------ seeded random chains
def _random_chained_workload(seed):
    from test_gpu_fuzz import random_workload
    w = random_workload(seed)
    rng = np.random.default_rng(seed + 77)
    light = [s for s, a in w.apps.items() if a.kind in (W.KIND_PROBE, W.KIND_STEER, W.KIND_PROJECT)]
    sae = [s for s, a in w.apps.items() if a.kind == W.KIND_SAE]
    rng.shuffle(light)
    chains, C_need = {}, w.C_max
    i = 0
    while i < len(light):
        n = int(rng.integers(1, 4))                                   # 1..3 light apps, then maybe an SAE app
        members = light[i:i + n]
        i += n
        if sae and rng.random() < 0.5:
            members = members + [int(rng.choice(sae))]
        classes = sum(w.apps[s].W.shape[0] for s in members if w.apps[s].kind == W.KIND_PROBE)
        if classes > 64 or len(members) < 2:
            continue
        for a, b in zip(members[:-1], members[1:]):
            chains[a] = b
        C_need = max(C_need, classes)
    return W.Workload(w.name + "c", w.d_model, w.T_max, w.T_live, w.hidden, w.token_slot, w.apps, w.groups, w.n_slots_max,
                      w.n_groups_max, C_need, w.k_max, w.r_max, w.d_sae_max, chains=chains)


@pytest.mark.parametrize("seed", range(16))
def test_random_chains(seed):
    mixlib = _mixlib()
    w = _random_chained_workload(3000 + seed)
    out = run_gpu(w, flags=mixlib.MIX_FLAG_SLOT_CHAINS, graph=bool(seed % 2), conditional=bool(seed % 4 == 1))
    check_chain_parity(W.host(w), out, scale_with_output=True, expect_status=None)
    assert out["status"] & ~mixlib.MIX_STATUS_TOPK_GENERAL == 0
