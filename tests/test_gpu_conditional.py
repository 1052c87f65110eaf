"""GPU: mix_apply_conditional — the SAE chain as the body of a graph IF node whose condition the
route kernel sets on the device.  Results must equal mix_apply()'s in both branches."""
import numpy as np
import pytest
import torch

import workloads as W

from parity import check_parity, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


def test_conditional_graph_matches_plain_apply_and_oracle():
    w = W.make_tiny(DEV)
    a = run_gpu(w, graph=True)
    b = run_gpu(w, graph=True, conditional=True, replays=3)
    assert b["status"] == 0
    for key in ("hidden", "topk_idx", "n_active"):
        assert np.array_equal(a[key], b[key]), key
    assert np.array_equal(a["scores"].view(np.uint32), b["scores"].view(np.uint32))
    check_parity(W.host(w), b)


def test_body_is_skipped_and_taken_by_the_same_captured_graph():
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    sae_slots = {s for s, a in w.apps.items() if a.kind == W.KIND_SAE}
    full = np.asarray(w.token_slot, dtype=np.int32).copy()
    no_sae = np.where(np.isin(full, list(sae_slots)), -1, full).astype(np.int32)
    assert (no_sae != full).any() and (no_sae >= 0).any()

    m = W.make_context(mixlib.Mix, w)
    T, C = w.T_max, max(w.C_max, 1)
    h = w.hidden.clone()
    scores = torch.zeros((T, C), dtype=torch.float32, device=DEV)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply_conditional(h, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)

    def replay(slot_map):
        m.set_slot_map(slot_map)
        h.copy_(w.hidden)
        g.replay()
        torch.cuda.synchronize()
        return W.bits(h)

    for slot_map in (no_sae, full, no_sae, full):
        got = replay(slot_map)
        # the same workload through the plain entry point, uncaptured
        w2 = W.Workload(w.name, w.d_model, w.T_max, w.T_live, w.hidden, slot_map, w.apps, w.groups, w.n_slots_max,
                        w.n_groups_max, w.C_max, w.k_max, w.r_max, w.d_sae_max)
        ref = run_gpu(w2)
        assert np.array_equal(got, ref["hidden"])
        check_parity(W.host(w2), dict(ref, hidden=got), check_features=False)
        if slot_map is no_sae:                      # rows that lost their SAE app are bit-exact pass-through
            rows = np.nonzero(full != no_sae)[0]
            assert np.array_equal(got[rows], W.bits(w.hidden)[rows])
    assert m.get_status() == 0
    m.destroy()


def test_conditional_outside_capture_is_an_error_and_no_sae_context_is_plain():
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    m = W.make_context(mixlib.Mix, w)
    h = w.hidden.clone()
    with pytest.raises(mixlib.MixError) as e:
        m.apply_conditional(h)
    assert e.value.code == -1
    assert np.array_equal(W.bits(h), W.bits(w.hidden))     # nothing was enqueued
    m.destroy()
    # a context without weight sets has no SAE chain: the call is mix_apply(), capturing or not
    wd = W.make_decode(DEV)
    md = W.make_context(mixlib.Mix, wd)
    hd = wd.hidden.clone()
    sc = torch.zeros((wd.T_max, max(wd.C_max, 1)), dtype=torch.float32, device=DEV)
    md.apply_conditional(hd, sc)
    torch.cuda.synchronize()
    ref = run_gpu(wd)
    assert np.array_equal(W.bits(hd), ref["hidden"])
    md.destroy()


def test_param_update_measurement_entry_runs_and_agrees():
    """mix_bench_param_update: the two mechanisms (device-table write, kernel-node parameter update) accumulate
    the same sum; both times are positive; bad arguments are rejected."""
    mixlib = _mixlib()
    m = mixlib.Mix(d_model=64, T_max=8, n_slots_max=1)
    a, b = m.bench_param_update(iters=300)
    assert 0.0 < a < 1e4 and 0.0 < b < 1e4
    with pytest.raises(mixlib.MixError) as e:
        m.bench_param_update(iters=0)
    assert e.value.code == -1
    m.destroy()
