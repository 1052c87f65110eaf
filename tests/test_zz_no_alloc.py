"""The allocation-free SAE entry point against the ordinary one.

mix_sae_apply_static() serves callers that are not allowed to allocate device memory (a
plugin inside a serving engine that owns all of HBM, a latency-critical path that cannot
afford cudaMalloc's implicit synchronisation).  Its scratch is one fixed array inside the
library, shared by all calls and never cleared between them, so the test makes different calls in
a row (a large one, a small one of another kind, a large one again) and checks each against
mix_apply() on an ordinary context given the same inputs and, row by row, against the float64
oracle.  This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

from parity import CANARY_F32, HIDDEN_TOL_FRAC, check_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(seed, n_rows, d, S, act, k, edits, add_error):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    sae = W.make_sae_weights(g, DEV, d, S, act, k=k, theta_range=(0.05, 0.3), b_enc_mean=-0.1 if add_error else -2.0)
    sae.b_dec = torch.randn(d, generator=g, device=DEV, dtype=torch.float32)
    hidden = torch.randn((n_rows, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    idx, val, mode = (np.asarray(edits[0], np.int32), np.asarray(edits[1], np.float32), np.asarray(edits[2], np.uint8))
    return sae, hidden, (idx, val, mode), add_error


def _via_context(mixlib, sae, hidden, edits, add_error):
    """The existing entry point: a context with one SAE app on every row (CUDA-core encode)."""
    n, d = hidden.shape
    m = mixlib.Mix(d_model=d, T_max=n, n_slots_max=1, n_groups_max=1, C_max=1, k_max=max(sae.k, 1), r_max=8,
                   d_sae_max=sae.d_sae, flags=mixlib.MIX_FLAG_ENCODE_SIMT)
    m.register_sae_weights(0, sae.d_sae, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec, theta=sae.theta, b_dec=sae.b_dec)
    m.register_sae_app(0, 0, *edits, add_error)
    m.set_slot_map(np.zeros(n, dtype=np.int32))
    h = hidden.clone()
    ti = torch.full((n, max(sae.k, 1)), -1, dtype=torch.int32, device=DEV)
    tv = torch.zeros((n, max(sae.k, 1)), dtype=torch.float32, device=DEV)
    m.set_feature_out(ti, tv, None)
    m.apply(h)
    torch.cuda.synchronize()
    assert m.get_status() == 0
    m.destroy()
    return h, ti, tv


def _via_static(mixlib, sae, hidden, edits, add_error):
    n = hidden.shape[0]
    h = hidden.clone()
    ti = torch.full((n, max(sae.k, 1)), -1, dtype=torch.int32, device=DEV)
    tv = torch.zeros((n, max(sae.k, 1)), dtype=torch.float32, device=DEV)
    mixlib.sae_apply_static(h, sae.d_sae, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec, *edits, add_error,
                            theta=sae.theta, b_dec=sae.b_dec, topk_idx=ti if sae.k else None,
                            topk_val=tv if sae.k else None)
    torch.cuda.synchronize()
    return h, ti, tv


def _oracle_check(case, out):
    """Every row of one static call against the float64 oracle: hidden state and, for TopK, ids and values."""
    sae, hidden, edits, add_error = case
    h_s, ti_s, tv_s = out
    n = hidden.shape[0]
    app = W.SaeApp(0, *edits, add_error)
    wl = W.Workload("static", hidden.shape[1], n, n, hidden, np.zeros(n, dtype=np.int32), {0: app}, {0: sae},
                    n_slots_max=1, n_groups_max=1, C_max=1, k_max=sae.k, r_max=8, d_sae_max=sae.d_sae)
    wh = W.host(wl)
    n_act = np.zeros(n, dtype=np.int32)
    if sae.k:
        n_act = (tv_s.cpu().numpy() > 0).sum(axis=1).astype(np.int32)    # what mix_apply would report for TopK rows
    res = dict(hidden=W.bits(h_s), scores=np.full((n, 1), CANARY_F32, dtype=np.uint32).view(np.float32),
               topk_idx=ti_s.cpu().numpy(), topk_val=tv_s.cpu().numpy(), n_active=n_act, status=0)
    return check_parity(wh, res, check_features=bool(sae.k))


def test_static_entry_point_matches_context_path_on_two_calls_in_a_row():
    import paper_2607_22595_b200 as mixlib
    cases = [
        _case(21, 100, 256, 2048, W.SAE_TOPK, 16, ([5, 900, 17, 1999], [3.0, 0.0, 6.5, 2.0], [0, 1, 0, 0]), True),
        # fewer rows, narrower SAE, other activation, no error term: stale rows, stale TopK
        # lists and a stale edit list from the first call must not show through
        _case(22, 37, 128, 1024, W.SAE_JUMPRELU, 0, ([7], [1.5], [0]), False),
        # and back to a full tile of rows after the small call, with the longer edit list again
        _case(24, 128, 256, 2048, W.SAE_TOPK, 16, ([11, 12, 2047, 0, 11], [2.0, 0.0, 4.0, 1.0, 7.0], [0, 1, 0, 0, 0]), False),
    ]
    static_out = [_via_static(mixlib, *c) for c in cases]          # back to back, same scratch
    for c, (h_s, ti_s, tv_s) in zip(cases, static_out):
        h_c, ti_c, tv_c = _via_context(mixlib, *c)
        sae, hidden = c[0], c[1]
        hmax = float(hidden.float().abs().max())
        err = (h_s.float() - h_c.float()).abs().max().item()
        assert err <= HIDDEN_TOL_FRAC * hmax, "hidden differs by %g" % err
        assert not torch.equal(h_s, hidden)                         # the call did something
        if sae.k:
            assert torch.equal(ti_s, ti_c)
            assert (tv_s - tv_c).abs().max().item() <= 1e-3
    # and every call stands on its own against the float64 oracle, on every row (the last row of the short
    # second call included: the case that exists to catch scratch left over from the first)
    for c, out in zip(cases, static_out):
        stats = _oracle_check(c, out)
        assert stats["rows"] == c[1].shape[0]


def test_static_entry_point_rejects_sizes_beyond_its_fixed_scratch():
    import paper_2607_22595_b200 as mixlib
    sae, hidden, edits, add_error = _case(23, 16, 128, 512, W.SAE_TOPK, 8, ([1], [1.0], [0]), True)
    too_many = torch.zeros((mixlib.STATIC_MAX_ROWS + 1, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(mixlib.MixError) as e:
        mixlib.sae_apply_static(too_many, sae.d_sae, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec, *edits, True)
    assert e.value.code == -2 and "n_rows" in str(e.value)
    with pytest.raises(mixlib.MixError) as e:
        mixlib.sae_apply_static(hidden.clone(), mixlib.STATIC_MAX_D_SAE * 2, sae.act, sae.k, sae.W_enc, sae.b_enc,
                                sae.W_dec, *edits, True)
    assert e.value.code == -2 and "d_sae" in str(e.value)
    with pytest.raises(mixlib.MixError) as e:
        mixlib.sae_apply_static(hidden.clone(), sae.d_sae, sae.act, mixlib.STATIC_MAX_K + 1, sae.W_enc, sae.b_enc,
                                sae.W_dec, *edits, True)
    assert e.value.code == -2
