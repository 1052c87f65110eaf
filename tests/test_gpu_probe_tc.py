"""GPU: the tensor-core probe kernel (large batches whose tiles with multi-class probe rows are mostly full,
contexts without SAE weight sets), the census of those tiles, and the device-side choice between that kernel
and the 16-row kernel."""
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


def _probe_workload(T_max, T_live, d, slot, classes, acts, seed=3, gate_rows=None):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    hidden = torch.randn((T_max, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    apps = {}
    for s, (C, act) in enumerate(zip(classes, acts)):
        if C == 0:       # a steering vector among the probes
            v = torch.randn(d, generator=g, device=DEV); apps[s] = W.Steer((v / v.norm()).to(torch.bfloat16), 2.0)
        else:
            apps[s] = W.Probe((torch.randn((C, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16),
                              torch.randn(C, generator=g, device=DEV) if s % 2 == 0 else None, act)
    if gate_rows is not None:
        gs = torch.full((T_max, 1), -1.0, device=DEV); gs[torch.from_numpy(gate_rows).to(DEV)] = 1.0
        apps[0].gate = W.Gate(gs, 0, W.GATE_GE, 0.0)
    return W.Workload("ptc", d, T_max, T_live, hidden, slot.astype(np.int32), apps, {}, n_slots_max=len(classes),
                      C_max=max(max(classes), 1))


@pytest.mark.parametrize("graph", [False, True])
def test_dense_batch_many_probes_per_tile(graph):
    # requests of 37 rows over 6 probes: every 128-row tile holds 4-5 different probes (several passes per
    # tile), class counts 2..32, all three activations, a live count that cuts the last tile, d = 320
    T_max, T_live, d = 4000, 3901, 320
    classes = [2, 5, 16, 32, 8, 31]
    acts = [W.ACT_SOFTMAX, W.ACT_NONE, W.ACT_SOFTMAX, W.ACT_SOFTMAX, W.ACT_SIGMOID if False else W.ACT_NONE, W.ACT_SOFTMAX]
    slot = (np.arange(T_max) // 37) % 6
    w = _probe_workload(T_max, T_live, d, slot, classes, acts)
    out = run_gpu(w, graph=graph)
    st = check_parity(W.host(w), out)
    assert st["rows"] == T_max and out["mix"].STAGES == ["probe_decide", "probe_steer", "probe_multiclass", "probe_tc"]


def test_dense_batch_with_other_kinds_unhooked_rows_and_a_gate():
    # 70 % multi-class probe rows (dense), the rest steering, one-class probes, a 40-class probe (too wide for
    # the kernel: stays with the streaming kernel) and unhooked rows; the gate of probe 0 is open on half its rows
    T_max, d = 2600, 512
    rng = np.random.default_rng(4)
    classes = [16, 3, 0, 1, 40]
    acts = [W.ACT_SOFTMAX, W.ACT_SOFTMAX, 0, W.ACT_SIGMOID, W.ACT_SOFTMAX]
    req = rng.choice(np.array([0, 0, 0, 1, 1, 1, 1, 2, 3, 4, -1]), size=T_max // 20 + 1)
    slot = np.repeat(req, 20)[:T_max]
    gate_rows = np.nonzero((slot == 0) & (np.arange(T_max) % 2 == 0))[0]
    w = _probe_workload(T_max, T_max, d, slot, classes, acts, gate_rows=gate_rows)
    out = run_gpu(w, graph=True)
    check_parity(W.host(w), out)
    unhooked = np.nonzero(slot < 0)[0]
    assert np.array_equal(out["hidden"][unhooked], W.bits(w.hidden)[unhooked])


@pytest.mark.parametrize("fill", [0.40, 0.60])
def test_both_sides_of_the_fill_threshold(fill):
    # every 128-row tile holds multi-class probe rows in its first `fill` part, nothing in the rest: below half
    # the 16-row kernel takes the call, above half the tensor-core one.  Either way the result is the oracle's.
    T_max, d = 2304, 256
    t = np.arange(T_max)
    slot = np.where((t % 128) < int(fill * 128), (t // 64) % 2, -1)
    w = _probe_workload(T_max, T_max, d, slot, [4, 12], [W.ACT_SOFTMAX, W.ACT_SOFTMAX])
    out = run_gpu(w)
    check_parity(W.host(w), out)


@pytest.mark.parametrize("graph", [False, True])
def test_sparse_batch_of_clustered_requests_takes_the_tile_list(graph):
    # a quarter of the requests (of 200 rows each) carry a multi-class probe, the rest are unhooked or steered:
    # the census lists about a third of the tiles, nearly full, and the tensor-core kernel shares THEM out;
    # replayed twice with another slot map in between, so that the census counters are seen to start from zero
    T_max, d = 6000, 384
    req = np.arange(T_max) // 200
    slot = np.where(req % 4 == 0, (req // 4) % 2, np.where(req % 4 == 1, 2, -1))
    w = _probe_workload(T_max, T_max - 57, d, slot, [16, 5, 0], [W.ACT_SOFTMAX, W.ACT_SOFTMAX, 0])
    out = run_gpu(w, graph=graph, replays=2)
    check_parity(W.host(w), out)
    m = out["mix"]
    slot2 = np.where(req % 2 == 0, 1, 0)                                   # every tile full of probe rows now
    w2 = _probe_workload(T_max, T_max, d, slot2, [16, 5, 0], [W.ACT_SOFTMAX, W.ACT_SOFTMAX, 0])
    w2.apps = w.apps
    m.set_slot_map(slot2.astype(np.int32), T_max)
    w2.hidden = w.hidden
    out2 = run_gpu(w2, mix=m)
    check_parity(W.host(w2), out2)
    m.set_slot_map(slot.astype(np.int32), T_max - 57)
    out3 = run_gpu(w, mix=m)
    check_parity(W.host(w), out3)
    unhooked = np.nonzero(slot < 0)[0]
    assert np.array_equal(out3["hidden"][unhooked], W.bits(w.hidden)[unhooked])


def test_same_scores_from_both_kernels():
    """One batch, once as it is (dense: tensor-core kernel) and once inside a context that also registers an SAE
    weight set (16-row kernel): scores agree to accumulation-order rounding."""
    mixlib = _mixlib()
    T_max, d = 2500, 384
    slot = (np.arange(T_max) // 50) % 3
    w = _probe_workload(T_max, T_max, d, slot, [7, 20, 32], [W.ACT_SOFTMAX] * 3)
    a = run_gpu(w)
    g = torch.Generator(device=DEV); g.manual_seed(9)
    sae = W.make_sae_weights(g, DEV, d, 256, W.SAE_TOPK, k=4)
    w2 = W.Workload("ptc2", d, T_max, T_max, w.hidden, w.token_slot, w.apps, {0: sae}, n_slots_max=3, n_groups_max=1,
                    C_max=32, k_max=4, r_max=1, d_sae_max=256)
    b = run_gpu(w2)
    assert "probe_tc" in a["mix"].STAGES and "probe_tc" not in b["mix"].STAGES
    written = ~np.isnan(a["scores"])                                    # unwritten entries keep their NaN canary
    assert np.array_equal(written, ~np.isnan(b["scores"])) and written.any()
    assert np.abs(a["scores"][written] - b["scores"][written]).max() <= 2e-6
    assert np.array_equal(a["hidden"], b["hidden"])


def test_time_out_path_of_the_tensor_core_probe_kernel():
    """With the test hook the producer delivers nothing and every wait is capped at about a millisecond: each
    CTA gives up, raises the status bit, frees its tensor memory and returns; nothing hangs, no row is written,
    and the device runs an ordinary call right afterwards."""
    mixlib = _mixlib()
    T_max, d = 2304, 256
    slot = (np.arange(T_max) // 64) % 2
    w = _probe_workload(T_max, T_max, d, slot, [4, 12], [W.ACT_SOFTMAX, W.ACT_SOFTMAX])
    out = run_gpu(w, flags=mixlib.MIX_FLAG_TEST_STALL_ENCODE)
    assert out["status"] & mixlib.MIX_STATUS_WAIT_TIMEOUT
    assert np.array_equal(out["hidden"], W.bits(w.hidden))
    assert np.isnan(out["scores"]).all()                               # the canary: no score was written
    good = run_gpu(w)
    assert good["status"] == 0
    check_parity(W.host(w), good)
