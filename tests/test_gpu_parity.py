"""GPU parity: the CUDA path (through the C ABI) against the float64 oracle, row by row."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

from parity import CANARY_F32, check_parity, oracle_edit_hint, run_gpu, sample_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


# ------------------------------------------------------------------ config 0
@pytest.mark.parametrize("graph", [False, True])
@pytest.mark.parametrize("simt", [False, True])
def test_tiny_full(graph, simt):
    w = W.make_tiny(DEV)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_ENCODE_SIMT if simt else 0, graph=graph)
    st = check_parity(W.host(w), out)
    assert st["rows"] == 64


def test_tiny_graph_replay_is_repeatable():
    w = W.make_tiny(DEV)
    a = run_gpu(w, graph=True, replays=1)
    b = run_gpu(w, graph=True, replays=5)
    assert np.array_equal(a["hidden"], b["hidden"]) and np.array_equal(a["topk_idx"], b["topk_idx"])


# ------------------------------------------------------------------ config 1
@pytest.mark.parametrize("graph", [False, True])
def test_decode_full(graph):
    w = W.make_decode(DEV)
    out = run_gpu(w, graph=graph)
    st = check_parity(W.host(w), out, check_features=False)
    assert st["max_hidden_ulp"] <= 1.0 + 1e-9          # steering is one rounding away from the exact value


# ------------------------------------------------------------------ shrunk configs 2-4 (several tiles, ragged tails)
@pytest.mark.parametrize("simt", [False, True])
def test_sae_heavy_small(simt):
    w = W.make_sae_heavy(DEV, d=256, d_sae=2048, k=16, T=700, R=12, G=3, n_edit=8, edit_hint=oracle_edit_hint)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_ENCODE_SIMT if simt else 0)
    check_parity(W.host(w), out)


def test_retiled_w_enc_matches_oracle():
    # the tile-contiguous copy of W_enc (several feature tiles, several k-blocks, two row tiles)
    mixlib = _mixlib()
    w = W.make_sae_heavy(DEV, d=320, d_sae=1280, k=16, T=400, R=8, G=2, n_edit=8, edit_hint=oracle_edit_hint)
    out = run_gpu(w, flags=mixlib.MIX_FLAG_RETILE_W_ENC, graph=True)
    check_parity(W.host(w), out)
    w = W.make_mixed(DEV, d=320, T=1500, R=40, d_sae=1024, cap=200, mu=3.5, edit_hint=oracle_edit_hint)
    check_parity(W.host(w), run_gpu(w, flags=mixlib.MIX_FLAG_RETILE_W_ENC))


@pytest.mark.parametrize("simt", [False, True])
def test_edit_only_shortcut_gives_the_same_hidden(simt):
    # ReLU / JumpReLU rows with the error term skip the encode; TopK rows and replace-mode rows do not
    mixlib = _mixlib()
    flags = mixlib.MIX_FLAG_SAE_EDIT_ONLY | (mixlib.MIX_FLAG_ENCODE_SIMT if simt else 0)
    w = W.make_mixed(DEV, d=320, T=1500, R=40, d_sae=1024, cap=200, mu=3.5, edit_hint=oracle_edit_hint)
    g = torch.Generator(device=DEV); g.manual_seed(3)
    sc = torch.randn((w.T_max, 1), generator=g, device=DEV)
    sae_slots = [s for s, a in w.apps.items() if a.kind == W.KIND_SAE]
    w.apps[sae_slots[0]].gate = W.Gate(sc, 0, W.GATE_GE, 0.0)          # a gated edit-only app
    w.apps[sae_slots[1]].add_error = False                              # this one still needs the encode
    w.groups[1].b_enc = w.groups[1].b_enc - 2.0                         # keep its replace-mode decode sparse
    w.apps[sae_slots[1]].group = 1
    out = run_gpu(w, flags=flags, graph=True)
    check_parity(W.host(w), out, check_features=False)
    for act in (W.SAE_RELU, W.SAE_TOPK):
        w1 = _one_sae_workload(192, 1024, act, 24, 150, True, ([5, 900, 17, 5], [3.0, 0.0, 6.5, 4.0], [0, 1, 0, 0]),
                               b_dec=True, center=True)
        check_parity(W.host(w1), run_gpu(w1, flags=flags), check_features=False)


def test_mixed_small():
    w = W.make_mixed(DEV, d=320, T=1500, R=40, d_sae=1024, cap=200, mu=3.5, edit_hint=oracle_edit_hint)
    out = run_gpu(w, graph=True)
    st = check_parity(W.host(w), out)
    assert st["rows"] == 1500


@pytest.mark.parametrize("t_live", [2601, 1999])
def test_mixed_large_batch_kernel(t_live):
    # T_max > 2048 selects the warp-per-row kernel and its cooperative multi-class probe pass;
    # 2601 rows leave a ragged last CTA, and a live count below T_max cuts a request in two
    w = W.make_mixed(DEV, d=320, T=2601, R=48, d_sae=1024, cap=300, mu=4.0, edit_hint=oracle_edit_hint)
    w.T_live = t_live
    out = run_gpu(w)
    st = check_parity(W.host(w), out)
    assert st["rows"] == 2601


def test_replay_small_fresh_maps_one_capture():
    mixlib = _mixlib()
    w = W.make_replay(DEV, d=256, T_max=512, d_sae=4096, k=16, G=3, n_probe=6, n_steer=4, n_sae_slots=9, n_edit=6)
    m = W.make_context(mixlib.Mix, w)
    T, k_max = w.T_max, w.k_max
    h_static = w.hidden.clone()
    scores = torch.empty((T, 1), dtype=torch.float32, device=DEV)
    tk_idx = torch.empty((T, k_max), dtype=torch.int32, device=DEV)
    tk_val = torch.empty((T, k_max), dtype=torch.float32, device=DEV)
    n_act = torch.empty((T,), dtype=torch.int32, device=DEV)
    m.set_feature_out(tk_idx, tk_val, n_act)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h_static, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply(h_static, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    for r in range(8):
        token_slot, n_live = W.replay_map(w, r)
        m.set_slot_map(token_slot, n_live)
        h_static.copy_(w.hidden)
        scores.copy_(torch.from_numpy(np.full((T, 1), CANARY_F32, dtype=np.uint32).view(np.float32)))
        tk_idx.fill_(-559038737); n_act.fill_(-559038737)
        g.replay()
        torch.cuda.synchronize()
        w.token_slot, w.T_live = token_slot, n_live
        out = dict(hidden=W.bits(h_static), scores=scores.cpu().numpy(), topk_idx=tk_idx.cpu().numpy(),
                   topk_val=tk_val.cpu().numpy(), n_active=n_act.cpu().numpy(), status=m.get_status())
        check_parity(W.host(w), out)


# ------------------------------------------------------------------ edge cases
def test_all_unhooked_zero_live_and_single_row():
    w = W.make_tiny(DEV)
    base = w.token_slot.copy()
    w.token_slot = np.full_like(base, -1)
    out = run_gpu(w)
    assert np.array_equal(out["hidden"], W.bits(w.hidden)) and (out["scores"].view(np.uint32) == CANARY_F32).all()
    w.token_slot = base
    w.T_live = 0
    out = run_gpu(w)
    assert np.array_equal(out["hidden"], W.bits(w.hidden)) and out["status"] == 0
    w.T_live = 1
    check_parity(W.host(w), run_gpu(w))
    for s in (0, 1, 2, 3):                 # every row on one slot
        w.T_live = w.T_max
        w.token_slot = np.full_like(base, s)
        check_parity(W.host(w), run_gpu(w))


def test_bad_slots_raise_status_and_pass_through():
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    w.token_slot[0] = 1000
    w.token_slot[1] = -7
    w.token_slot[2] = 6                     # in range, never registered
    out = run_gpu(w)
    check_parity(W.host(w), out, expect_status=mixlib.MIX_STATUS_BAD_SLOT)


def test_alpha_zero_and_opposite_alphas():
    w = W.make_decode(DEV, d=512, T=64, n_probe=2, n_steer=2)
    steer_slots = [s for s, a in w.apps.items() if a.kind == W.KIND_STEER]
    for s in steer_slots:
        w.apps[s].alpha = 0.0
    # negative zeros in the input must survive alpha = 0
    hb = W.bits(w.hidden).copy(); hb[:, 3] = 0x8000
    w.hidden = W.from_bits(hb, DEV)
    out = run_gpu(w)
    assert np.array_equal(out["hidden"], hb)
    w.apps[steer_slots[0]].alpha = 3.0
    out = run_gpu(w)
    check_parity(W.host(w), out, check_features=False)
    # +alpha then -alpha returns within one bf16 ulp
    h1 = W.from_bits(out["hidden"], DEV)
    w.apps[steer_slots[0]].alpha = -3.0
    out2 = run_gpu(w, hidden=h1)
    a, b = O.bf16_to_f64(out2["hidden"]), O.bf16_to_f64(hb)
    from parity import bf16_ulp
    assert (np.abs(a - b) <= bf16_ulp(np.maximum(np.abs(b), np.abs(O.bf16_to_f64(out["hidden"]))))).all()


def test_project_rows_small_and_large_batch_kernels():
    for T in (96, 2304):                              # team kernel / warp-per-row kernel
        w = W.make_decode(DEV, d=1024, T=T, n_probe=2, n_steer=2)
        g = torch.Generator(device=DEV); g.manual_seed(77)
        for s, a in list(w.apps.items()):
            if a.kind == W.KIND_STEER:
                r = torch.randn(1024, generator=g, device=DEV); r = (r / r.norm()).to(torch.bfloat16)
                w.apps[s] = W.Project(r, 1.0 if s % 2 else 0.5)
        out = run_gpu(w, graph=True)
        st = check_parity(W.host(w), out, check_features=False)
        # with beta = 1 nothing (beyond rounding) is left along r
        wh = W.host(w)
        for t in range(T):
            a = wh.apps.get(int(wh.token_slot[t]))
            if a is not None and a.kind == W.KIND_PROJECT and a.beta == 1.0:
                y = O.bf16_to_f64(out["hidden"][t]); r = O.bf16_to_f64(a.r)
                assert abs(y @ r) <= 2e-2 * np.abs(O.bf16_to_f64(wh.hidden[t])).max()
        assert st["max_hidden_ulp"] <= 1.0 + 1e-6 or st["max_hidden_err"] < 1e-2


def _one_sae_workload(d, S, act, k, T, add_error, edits, b_dec=False, center=False, seed=5, W_enc=None,
                      b_enc=None, b_enc_mean=-0.1):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    sae = W.make_sae_weights(g, DEV, d, S, act, k=k, theta_range=(0.05, 0.3), b_enc_mean=b_enc_mean)
    if W_enc is not None:
        sae.W_enc = W_enc
    if b_enc is not None:
        sae.b_enc = b_enc
    if b_dec:
        sae.b_dec = torch.randn(d, generator=g, device=DEV, dtype=torch.float32)
        sae.center_input = center
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    idx, val, mode = edits
    app = W.SaeApp(0, np.asarray(idx, np.int32), np.asarray(val, np.float32), np.asarray(mode, np.uint8), add_error)
    return W.Workload("one_sae", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=2,
                      n_groups_max=1, C_max=1, k_max=max(k, 1), r_max=max(len(idx), 1), d_sae_max=S)


@pytest.mark.parametrize("act", [W.SAE_RELU, W.SAE_JUMPRELU, W.SAE_TOPK])
@pytest.mark.parametrize("add_error", [True, False])
def test_sae_modes_with_b_dec_and_centering(act, add_error):
    # replace mode on ReLU / JumpReLU sums every active feature: keep them sparse with a low bias
    w = _one_sae_workload(192, 1024, act, 24, 150, add_error, ([5, 900, 17, 5], [3.0, 0.0, 6.5, 4.0], [0, 1, 0, 0]),
                          b_dec=True, center=True, b_enc_mean=-0.1 if add_error else -2.0)
    out = run_gpu(w)
    check_parity(W.host(w), out)


@pytest.mark.parametrize("act", [W.SAE_JUMPRELU, W.SAE_TOPK])
def test_interleaved_slots_in_one_weight_set(act):
    # consecutive packed rows alternate between five slots of ONE weight set: different edit lists
    # (one with a repeated feature, one empty, one that clamps to the value it already has), rows that
    # keep the error term next to rows that replace the residual, and unhooked rows in between
    d, S, k, T = 320, 1024, 16, 203
    g = torch.Generator(device=DEV); g.manual_seed(11)
    sae = W.make_sae_weights(g, DEV, d, S, act, k=k, theta_range=(0.05, 0.3), b_enc_mean=-1.0)
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    def app(idx, val, mode, err):
        return W.SaeApp(0, np.asarray(idx, np.int32), np.asarray(val, np.float32), np.asarray(mode, np.uint8), err)
    apps = {0: app([3, 700, 3], [2.0, 0.0, 5.0], [0, 1, 0], True),
            1: app([], [], [], True),
            2: app([9, 10, 11, 12, 1000], [1.0, 1.5, 0.0, 2.5, 4.0], [0, 0, 1, 0, 0], True),
            3: app([44], [3.0], [0], False),
            4: app([1023], [0.0], [1], True)}            # ablating a feature that is almost never active
    slot = np.array([(t % 6) - 1 for t in range(T)], dtype=np.int32)   # -1 = unhooked
    w = W.Workload("interleaved", d, T, T, hidden, slot, apps, {0: sae}, n_slots_max=5, n_groups_max=1, C_max=1,
                   k_max=k, r_max=5, d_sae_max=S)
    out = run_gpu(w, graph=True)
    st = check_parity(W.host(w), out)
    assert st["rows"] == T
    h0 = W.bits(w.hidden)
    for t in range(T):
        if slot[t] in (-1, 1):
            assert np.array_equal(out["hidden"][t], h0[t])            # unhooked / no edit: bit-exact


def test_no_edit_with_error_leaves_rows_bit_exact():
    w = _one_sae_workload(128, 512, W.SAE_TOPK, 8, 40, True, ([], [], []))
    out = run_gpu(w)
    assert np.array_equal(out["hidden"], W.bits(w.hidden))
    check_parity(W.host(w), out)


def test_topk_exact_ties_pick_lower_index():
    # duplicate encoder rows give exactly equal pre-activations; the lower feature id must win
    d, S, k = 128, 512, 8
    g = torch.Generator(device=DEV); g.manual_seed(3)
    We = (torch.randn((S, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16)
    We[256:] = We[:256]
    be = torch.full((S,), -0.1, dtype=torch.float32, device=DEV)
    w = _one_sae_workload(d, S, W.SAE_TOPK, k, 33, True, ([1], [2.0], [0]), W_enc=We, b_enc=be)
    out = run_gpu(w)
    check_parity(W.host(w), out)
    ref = O.apply_hook(W.host(w), keep_z=False)
    for t in range(33):
        assert out["topk_idx"][t, :k].tolist() == ref.topk[t].tolist()      # exact, order included


def test_topk_massive_ties_use_general_path():
    # W_enc = 0: every pre-activation equals the bias -> more ties than the candidate buffer holds
    mixlib = _mixlib()
    d, S, k = 128, 8192, 16
    We = torch.zeros((S, d), dtype=torch.bfloat16, device=DEV)
    be = torch.full((S,), 0.25, dtype=torch.float32, device=DEV)
    be[5000] = 1.0; be[77] = 0.5
    w = _one_sae_workload(d, S, W.SAE_TOPK, k, 5, False, ([77], [0.0], [1]), W_enc=We, b_enc=be)
    out = run_gpu(w)
    check_parity(W.host(w), out, expect_status=mixlib.MIX_STATUS_TOPK_GENERAL)
    assert out["topk_idx"][0, :k].tolist() == [5000, 77] + list(range(14))


def test_identity_encoder_topk_of_own_coordinates():
    d, S, k = 128, 512, 8
    I = torch.zeros((S, d), dtype=torch.bfloat16, device=DEV); I[:d] = torch.eye(d, dtype=torch.bfloat16, device=DEV)
    w = _one_sae_workload(d, S, W.SAE_TOPK, k, 20, False, ([], [], []), W_enc=I,
                          b_enc=torch.zeros(S, dtype=torch.float32, device=DEV))
    w.groups[0].W_dec = I.clone()
    out = run_gpu(w)
    check_parity(W.host(w), out)
    h = O.bf16_to_f64(W.bits(w.hidden))
    for t in range(20):                      # output = ReLU of the row's own k largest coordinates
        K = out["topk_idx"][t, :k]
        want = np.zeros(d); want[K] = np.maximum(h[t, K], 0)
        assert np.array_equal(O.bf16_to_f64(out["hidden"][t]), want)


# ------------------------------------------------------------------ toggling under one captured graph
def test_toggle_without_recapture():
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    m = W.make_context(mixlib.Mix, w)
    T = w.T_max
    h_static = w.hidden.clone()
    scores = torch.zeros((T, 1), dtype=torch.float32, device=DEV)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h_static, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply(h_static, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)

    def replay_and_check(expect_status=0):
        h_static.copy_(w.hidden)
        scores.copy_(torch.from_numpy(np.full((T, 1), CANARY_F32, dtype=np.uint32).view(np.float32)))
        g.replay()
        torch.cuda.synchronize()
        out = dict(hidden=W.bits(h_static), scores=scores.cpu().numpy(), status=m.get_status())
        check_parity(W.host(w), out, check_features=False, expect_status=expect_status)

    replay_and_check()
    w.apps[1].alpha = -2.5; m.update_steer_alpha(1, -2.5)                 # change a parameter
    replay_and_check()
    idx, val, mode = np.array([7, 9], np.int32), np.array([1.5, 0], np.float32), np.array([0, 1], np.uint8)
    w.apps[2].edit_idx, w.apps[2].edit_val, w.apps[2].edit_mode = idx, val, mode
    m.update_sae_edits(2, idx, val, mode)                                 # change an edit list
    replay_and_check()
    rng = np.random.default_rng(1)
    w.token_slot = rng.permutation(w.token_slot).astype(np.int32); m.set_slot_map(w.token_slot)
    replay_and_check()
    del w.apps[0]; m.unregister_app(0)                                    # rows still naming slot 0 pass through
    replay_and_check(expect_status=mixlib.MIX_STATUS_BAD_SLOT)
    g2 = torch.Generator(device=DEV); g2.manual_seed(9)
    w.apps[5] = W.Steer(v=torch.randn(w.d_model, generator=g2, device=DEV).to(torch.bfloat16), alpha=0.75)
    m.register_steer(5, w.apps[5].v, 0.75)
    w.token_slot = np.where(w.token_slot == 0, 5, w.token_slot).astype(np.int32); m.set_slot_map(w.token_slot)
    replay_and_check()


def test_request_map_two_level_matches_flat_map():
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    m = W.make_context(mixlib.Mix, w)
    token_req = w.meta["token_req"].astype(np.int32)
    m.set_request_map(token_req, w.meta["req_slot"].astype(np.int32))
    out = run_gpu(w, mix=m)
    check_parity(W.host(w), out)
    m.set_request_map(torch.from_numpy(token_req).cuda(), torch.from_numpy(w.meta["req_slot"].astype(np.int32)).cuda())
    check_parity(W.host(w), run_gpu(w, mix=m))


def test_permutation_equivariance_on_gpu():
    w = W.make_tiny(DEV)
    a = run_gpu(w)
    perm = np.random.default_rng(0).permutation(w.T_max)
    w2 = W.make_tiny(DEV)
    w2.hidden = w.hidden[torch.from_numpy(perm).cuda()].contiguous()
    w2.token_slot = w.token_slot[perm].copy()
    b = run_gpu(w2)
    assert np.array_equal(b["hidden"], a["hidden"][perm])
    assert np.array_equal(b["scores"].view(np.uint32), a["scores"].view(np.uint32)[perm])


def test_api_error_codes():
    mixlib = _mixlib()
    with pytest.raises(mixlib.MixError) as e:
        mixlib.Mix(d_model=100, T_max=8, n_slots_max=2)                    # d % 64
    assert e.value.code == -3
    m = mixlib.Mix(d_model=128, T_max=8, n_slots_max=2, n_groups_max=1, C_max=2, k_max=4, r_max=2, d_sae_max=256)
    v = torch.zeros(128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(mixlib.MixError) as e:
        m.register_steer(5, v, 1.0)
    assert e.value.code == -2 and "slot" in str(e.value)
    Wp = torch.zeros((3, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(mixlib.MixError) as e:
        m.register_probe(0, Wp, None, mixlib.MIX_ACT_SOFTMAX)              # C > C_max
    assert e.value.code == -2
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_app(0, 0, [1], [1.0], [0], True)                   # group not registered
    assert e.value.code == -2
    We = torch.zeros((256, 128), dtype=torch.bfloat16, device=DEV); be = torch.zeros(256, device=DEV)
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_weights(0, 256, mixlib.MIX_SAE_TOPK, 9, We, be, We)  # k > k_max
    assert e.value.code == -2
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_weights(0, 256, mixlib.MIX_SAE_JUMPRELU, 0, We, be, We)  # no theta
    assert e.value.code == -1
    m.register_sae_weights(0, 256, mixlib.MIX_SAE_TOPK, 4, We, be, We)
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_app(0, 0, [256], [1.0], [0], True)                 # feature id out of range
    assert e.value.code == -2
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_app(0, 0, [1, 2, 3], [1.0, 1, 1], [0, 0, 0], True)  # n_edit > r_max
    assert e.value.code == -2
    with pytest.raises(mixlib.MixError) as e:
        m.set_slot_map(np.zeros(9, dtype=np.int32))                       # T_live > T_max
    assert e.value.code == -2
    assert m.launches_per_apply() == 7                                # hook kernel + front, encode x 2, tail, flagged encode, flagged tail
    m.destroy()


def test_replacing_a_weight_set_and_failed_edit_updates_change_nothing():
    """A weight set may be replaced under attached apps only if the new width still covers their edited
    features (the device indexes W_enc / W_dec rows with them), and an edit update that fails validation
    leaves the app exactly as it was.  API checks only: no call here reaches a kernel with a bad index."""
    mixlib = _mixlib()
    d, S = 128, 512
    g = torch.Generator(device=DEV); g.manual_seed(5)
    sae = W.make_sae_weights(g, DEV, d, S, W.SAE_TOPK, k=4)
    hidden = torch.randn((8, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    m = mixlib.Mix(d_model=d, T_max=8, n_slots_max=2, n_groups_max=1, C_max=1, k_max=4, r_max=4, d_sae_max=S)
    m.register_sae_weights(0, S, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec)
    m.register_sae_app(0, 0, [3, 300], [2.0, 0.0], [0, 1], True)
    with pytest.raises(mixlib.MixError) as e:           # 256 features no longer cover feature 300
        m.register_sae_weights(0, 256, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec)
    assert e.value.code == -1 and "300" in str(e.value)
    m.set_slot_map(np.zeros(8, dtype=np.int32))
    h1 = hidden.clone(); m.apply(h1); torch.cuda.synchronize()
    with pytest.raises(mixlib.MixError) as e:           # second entry out of range: nothing may change
        m.update_sae_edits(0, [5, 512], [1.0, 1.0], [0, 0])
    assert e.value.code == -2
    with pytest.raises(mixlib.MixError) as e:
        m.update_sae_edits(0, [5], [1.0], [7])          # bad mode, shorter list: the count must not shrink
    assert e.value.code == -1
    h2 = hidden.clone(); m.apply(h2); torch.cuda.synchronize()
    assert torch.equal(h1, h2) and not torch.equal(h1, hidden)
    m.update_sae_edits(0, [3], [2.0], [0])              # feature 300 is gone from the list ...
    m.register_sae_weights(0, 256, sae.act, sae.k, sae.W_enc, sae.b_enc, sae.W_dec)   # ... so the narrower set fits
    h3 = hidden.clone(); m.apply(h3); torch.cuda.synchronize()
    assert m.get_status() == 0
    m.destroy()


def test_one_class_probe_bias_and_raw_logit_in_a_decode_context():
    """One-class probes with non-zero biases in a context of at most 2048 rows (the one-CTA-per-row kernel, which
    takes the bias from the app entry): sigmoid and raw-logit probes, a probe without a bias, and a re-registration
    with another bias under the same captured graph."""
    mixlib = _mixlib()
    d, T = 512, 96
    g = torch.Generator(device=DEV); g.manual_seed(77)
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    def probe(bias, act):
        Wp = (torch.randn((1, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16)
        b = None if bias is None else torch.tensor([bias], dtype=torch.float32, device=DEV)
        return W.Probe(W=Wp, b=b, act=act)
    apps = {0: probe(1.75, W.ACT_SIGMOID), 1: probe(-3.5, W.ACT_NONE), 2: probe(None, W.ACT_SIGMOID), 3: probe(0.25, W.ACT_NONE)}
    token_slot = (np.arange(T) % 5 - 1).astype(np.int32)
    w = W.Workload("bias", d, T, T, hidden, token_slot, apps, {}, n_slots_max=4, C_max=1)
    out = run_gpu(w, graph=True)
    st = check_parity(W.host(w), out)
    assert st["max_score_rel"] < 1e-4
    # a new registration of slot 1 with another bias takes effect without a new capture
    m = out["mix"]
    apps[1] = W.Probe(W=apps[1].W, b=torch.tensor([2.0], dtype=torch.float32, device=DEV), act=W.ACT_NONE)
    m.register_probe(1, apps[1].W, apps[1].b, apps[1].act)
    w2 = W.Workload("bias2", d, T, T, hidden, token_slot, apps, {}, n_slots_max=4, C_max=1)
    out2 = run_gpu(w2, mix=m)
    check_parity(W.host(w2), out2)
    m.destroy()


# ------------------------------------------------------------------ full-size configs, sampled rows
def test_sae_heavy_full_size_sampled_rows():
    w = W.make_sae_heavy(DEV, edit_hint=oracle_edit_hint)
    out = run_gpu(w, graph=True)
    wh = W.host(w)
    rows = sample_rows(wh, per_kind=6, seed=2)
    st = check_parity(wh, out, rows=rows)
    assert st["rows"] >= 24


def test_mixed_full_size_sampled_rows():
    w = W.make_mixed(DEV, edit_hint=oracle_edit_hint)
    out = run_gpu(w, graph=True)
    wh = W.host(w)
    # every unhooked row is bit-identical, at full size
    unh = np.nonzero(wh.token_slot < 0)[0]
    assert np.array_equal(out["hidden"][unh], wh.hidden[unh])
    rows = sample_rows(wh, per_kind=16, seed=3)
    check_parity(wh, out, rows=rows)


def test_replay_full_size_sampled_rows():
    """Config 4 at full size (8 SAEs of 131072 x 8192, 32 GiB of weights), replay 1 (all 2048 rows
    live) under the captured graph; the oracle checks every probe / steer / unhooked row of a sample
    and SAE rows of two weight sets (their weights alone are copied to the host)."""
    mixlib = _mixlib()
    w = W.make_replay(DEV)
    w.token_slot, w.T_live = W.replay_map(w, 1)
    out = run_gpu(w, graph=True)
    assert out["status"] == 0
    present = {}
    for t in range(w.T_max):
        a = w.apps.get(int(w.token_slot[t]))
        if a is not None and a.kind == W.KIND_SAE:
            present[a.group] = present.get(a.group, 0) + 1
    keep = sorted(present, key=present.get)[-2:]          # the two busiest weight sets of this replay
    wh = W.host(w, only_groups=keep)
    rows, per_group = [], {}
    for t in range(w.T_max):
        a = w.apps.get(int(w.token_slot[t]))
        if a is None or a.kind != W.KIND_SAE:
            if t % 16 == 0:
                rows.append(t)
        elif a.group in keep and per_group.get(a.group, 0) < 3:
            per_group[a.group] = per_group.get(a.group, 0) + 1
            rows.append(t)
    assert len(per_group) == 2
    st = check_parity(wh, out, rows=rows, expect_status=None)
    assert st["rows"] == len(rows)
    # unhooked rows: all of them, bit for bit
    unh = np.nonzero(w.token_slot < 0)[0]
    assert np.array_equal(out["hidden"][unh], W.bits(w.hidden)[unh])
    out["mix"].destroy()
    torch.cuda.empty_cache()


def test_encode_timeout_path_raises_status_and_leaves_the_context_usable():
    """Failure detection without a GPU fault: with the test hook the encode kernel's producer never
    delivers a tile, every CTA's bounded wait (capped at ~1 ms) runs out, the kernel returns with
    MIX_STATUS_WAIT_TIMEOUT, and the next, ordinary call on the same device is correct."""
    mixlib = _mixlib()
    w = W.make_tiny(DEV)
    m = W.make_context(mixlib.Mix, w, flags=mixlib.MIX_FLAG_TEST_STALL_ENCODE)
    h = w.hidden.clone()
    scores = torch.zeros((w.T_max, 1), dtype=torch.float32, device=DEV)
    m.apply(h, scores)
    torch.cuda.synchronize()                                   # returns: nothing hangs
    st = m.get_status()
    assert st & mixlib.MIX_STATUS_WAIT_TIMEOUT
    assert m.get_status() == 0                                 # reading the word clears it
    # rows without an SAE app are unaffected by the failed encode
    wh = W.host(w)
    ref = O.apply_hook(wh)
    for t in range(w.T_max):
        if ref.kind[t] in (0, O.KIND_PROBE):
            assert np.array_equal(W.bits(h)[t], wh.hidden[t])
    m.destroy()
    check_parity(wh, run_gpu(w))                               # a fresh ordinary context works


# ------------------------------------------------------------------ the interface's maximum sizes
@pytest.mark.parametrize("T", [48, 2100])
def test_maximum_width_and_class_count(T):
    """d = 8192 (widest hidden state), 64-class softmax probes (most classes), next to 33-class ones (one more
    than the tensor-core probe kernel takes), in the small-batch and the large-batch kernels."""
    d = 8192
    g = torch.Generator(device=DEV); g.manual_seed(21)
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    mk = lambda C, act: W.Probe((torch.randn((C, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16),
                                torch.randn(C, generator=g, device=DEV), act)
    v = torch.randn(d, generator=g, device=DEV); v = (v / v.norm()).to(torch.bfloat16)
    apps = {0: mk(64, W.ACT_SOFTMAX), 1: mk(33, W.ACT_SOFTMAX), 2: mk(32, W.ACT_NONE), 3: W.Steer(v, 3.0), 4: W.Project(v, 1.0)}
    slot = (np.arange(T) % 6 - 1).astype(np.int32)
    w = W.Workload("max", d, T, T, hidden, slot, apps, {}, n_slots_max=5, C_max=64)
    out = run_gpu(w, graph=True)
    check_parity(W.host(w), out)


@pytest.mark.parametrize("add_error", [True, False])
def test_maximum_k_and_edit_list(add_error):
    """TopK with k = 1024 (largest k) and 64 edits per app (longest list, with a repeated feature), on rows
    that span two row tiles."""
    d, S, k, T = 256, 4096, 1024, 150
    g = torch.Generator(device=DEV); g.manual_seed(22)
    sae = W.make_sae_weights(g, DEV, d, S, W.SAE_TOPK, k=k)
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    rng = np.random.default_rng(22)
    idx = rng.choice(S, size=64, replace=False).astype(np.int32); idx[63] = idx[0]
    val = rng.uniform(0.5, 4.0, size=64).astype(np.float32)
    mode = (np.arange(64) % 3 == 0).astype(np.uint8)
    app = W.SaeApp(0, idx, val, mode, add_error)
    w = W.Workload("maxk", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=k, r_max=64, d_sae_max=S)
    out = run_gpu(w)
    check_parity(W.host(w), out, expect_status=None)
    assert out["status"] & ~_mixlib().MIX_STATUS_TOPK_GENERAL == 0


def test_create_destroy_returns_all_device_memory():
    """Every allocation of every kind of context (SAE with both encoder forms, chains, the large-batch probe
    kernels, registrations that make the library keep copies) is released by mix_destroy."""
    mixlib = _mixlib()
    g = torch.Generator(device=DEV); g.manual_seed(0)

    def cycle():
        w = W.make_tiny(DEV)
        m = W.make_context(mixlib.Mix, w, flags=mixlib.MIX_FLAG_RETILE_W_ENC | mixlib.MIX_FLAG_SLOT_CHAINS)
        m.apply(w.hidden.clone()); m.destroy()
        sae = W.make_sae_weights(g, DEV, 128, 512, W.SAE_TOPK, k=4, fp8=True)
        m = mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=512,
                       flags=mixlib.MIX_FLAG_FP8_W_ENC)
        m.register_sae_weights(0, 512, sae.act, 4, sae.W_enc, sae.b_enc, sae.W_dec, w_scale=sae.w_scale)
        m.destroy()
        sae = W.make_sae_weights(g, DEV, 128, 512, W.SAE_RELU)
        m = mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, r_max=1, d_sae_max=512)
        m.register_sae_weights(0, 512, sae.act, 0, sae.W_enc, sae.b_enc, sae.W_dec, b_dec=torch.zeros(128, device=DEV),
                               center_input=True)
        m.destroy()
        m = mixlib.Mix(d_model=128, T_max=4096, n_slots_max=4, C_max=8)          # both multi-class probe kernels
        m.register_probe(0, torch.zeros((8, 128), device=DEV, dtype=torch.bfloat16), None, mixlib.MIX_ACT_SOFTMAX)
        m.destroy()

    cycle()                                              # first use may load modules and grow caches
    torch.cuda.synchronize(); torch.cuda.empty_cache()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(20):
        cycle()
    torch.cuda.synchronize(); torch.cuda.empty_cache()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < (8 << 20), "device memory shrank by %d bytes over 20 create/destroy cycles" % (free0 - free1)


@pytest.mark.parametrize("which", ["tiny", "mixed", "dense_probes"])
def test_guard_bands_around_the_callers_buffers_stay_intact(which):
    """hidden, scores and the feature read-out buffers sit inside larger allocations whose extra rows before and
    after carry a canary pattern: no kernel of the call may write (or, for hidden, change) a byte outside the
    [T_max, ...] window it was given."""
    mixlib = _mixlib()
    if which == "tiny":
        w = W.make_tiny(DEV)
    elif which == "mixed":
        w = W.make_mixed(DEV, d=320, T=2601, R=48, d_sae=1024, cap=300, mu=4.0, edit_hint=oracle_edit_hint)
    else:
        T, d = 2560, 256
        g = torch.Generator(device=DEV); g.manual_seed(5)
        apps = {s: W.Probe((torch.randn((C, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16), None, W.ACT_SOFTMAX)
                for s, C in enumerate([3, 17])}
        hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        w = W.Workload("dense", d, T, T, hidden, ((np.arange(T) // 100) % 2).astype(np.int32), apps, {}, n_slots_max=2, C_max=17)
    T, d, C, k_max = w.T_max, w.d_model, max(w.C_max, 1), max(w.k_max, 1)
    G = 3                                                   # guard rows on each side
    def guarded(cols, dtype, fill):
        big = torch.full((T + 2 * G, cols), fill, dtype=dtype, device=DEV)
        return big, big[G:G + T]
    h_big, h = guarded(d, torch.bfloat16, 0.0)
    h_big[:G] = 123.0; h_big[G + T:] = -77.0
    h.copy_(w.hidden)
    s_big, scores = guarded(C, torch.float32, 4242.0)
    i_big, tk_idx = guarded(k_max, torch.int32, -99)
    v_big, tk_val = guarded(k_max, torch.float32, 4242.0)
    n_big, n_act = guarded(1, torch.int32, -99)
    m = W.make_context(mixlib.Mix, w)
    if w.n_groups_max > 0:
        m.set_feature_out(tk_idx, tk_val, n_act.view(-1))
    m.apply(h, scores)
    torch.cuda.synchronize()
    assert (h_big[:G] == 123.0).all() and (h_big[G + T:] == -77.0).all()
    for big, fill in ((s_big, 4242.0), (i_big, -99), (v_big, 4242.0), (n_big, -99)):
        assert (big[:G] == fill).all() and (big[G + T:] == fill).all()
    assert m.get_status() == 0
    # and inside the window the result is the usual one
    ref = run_gpu(w)
    assert np.array_equal(W.bits(h), ref["hidden"])
    m.destroy()


# ------------------------------------------------------------------ the encode epilogue's running TopK bound
@pytest.mark.parametrize("k", [1, 7, 64, 128, 129])
@pytest.mark.parametrize("case", ["plain", "all_negative", "winners_in_one_tile", "equal_across_tiles"])
def test_topk_running_bound_adversarial(k, case):
    """Many feature tiles per CTA-wave on few rows, so later tiles start from the bound earlier tiles published:
    k at the slot count's edges (128 slots; 129 switches the bound off), pre-activations that are all negative,
    more than eight winners inside one tile (the candidate lists overflow: flagged rows, exact fallback), and
    values repeated exactly in every tile (ties across tiles: the lower feature id wins)."""
    d, S, T = 128, 256 * 40, 70                          # 40 feature tiles, one ragged row tile
    g = torch.Generator(device=DEV); g.manual_seed(100 + k)
    We = (torch.randn((S, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16)
    be = torch.randn((S,), generator=g, device=DEV) * 0.05
    if case == "all_negative":
        be = be - 50.0
    elif case == "winners_in_one_tile":
        be[256 * 17 + 3: 256 * 17 + 3 + 12] += 30.0       # twelve of the largest values sit in tile 17
    elif case == "equal_across_tiles":
        We[256:] = We[:256].repeat(39, 1)                 # every tile repeats tile 0: 40-fold exact ties
        be[256:] = be[:256].repeat(39)
    w = _one_sae_workload(d, S, W.SAE_TOPK, k, T, True, ([3, 256 * 17 + 5], [2.0, 0.0], [0, 1]), W_enc=We, b_enc=be)
    out = run_gpu(w, graph=True, replays=2)
    check_parity(W.host(w), out, expect_status=None)
    assert out["status"] & ~_mixlib().MIX_STATUS_TOPK_GENERAL == 0
    if case == "equal_across_tiles":
        # the tie rule across tiles, free of fp32-vs-fp64 near-ties between DIFFERENT base features: a copy in
        # tile m is selected only if the copies in all lower tiles are
        for t in range(T):
            ids = set(out["topk_idx"][t, :k].tolist())
            for j in ids:
                assert all((j % 256) + 256 * m in ids for m in range(j // 256)), "row %d id %d" % (t, j)


def test_edit_only_rows_of_different_slots_share_a_cta():
    """The edit-only kernel takes eight consecutive token rows per CTA and shares the edited encoder / decoder rows
    among rows of one slot: here the slot changes every one to three rows, two weight sets (ReLU and JumpReLU)
    alternate, unhooked, probe and steering rows sit in between, the batch ends in the middle of a CTA's rows, and
    d = 8192 uses the largest shared-memory layout."""
    mixlib = _mixlib()
    d, S, T = 8192, 512, 77
    g = torch.Generator(device=DEV); g.manual_seed(21)
    rng = np.random.default_rng(21)
    groups = {0: W.make_sae_weights(g, DEV, d, S, W.SAE_RELU, b_enc_mean=-0.05),
              1: W.make_sae_weights(g, DEV, d, S, W.SAE_JUMPRELU, theta_range=(0.05, 0.3))}
    apps = {}
    for s in range(6):                                   # six SAE apps, three per weight set, different edit lists
        n_edit = int(rng.integers(1, 9))
        idx = rng.integers(0, S, size=n_edit).astype(np.int32)
        if n_edit >= 3:
            idx[-1] = idx[0]                             # a repeated feature: the later entry wins
        mode = rng.integers(0, 2, size=n_edit).astype(np.uint8)
        val = np.where(mode == W.EDIT_CLAMP, rng.uniform(0.5, 6, size=n_edit), 0).astype(np.float32)
        apps[s] = W.SaeApp(s % 2, idx, val, mode, True)
    apps[6] = W.Steer((torch.randn(d, generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16), 3.0)
    apps[7] = W.Probe((torch.randn((1, d), generator=g, device=DEV) * d ** -0.5).to(torch.bfloat16), None, W.ACT_SIGMOID)
    token_slot = np.full(T, -1, dtype=np.int32)
    t = 0
    while t < T:
        seg = int(rng.integers(1, 4))
        token_slot[t:t + seg] = int(rng.choice([-1, 0, 1, 2, 3, 4, 5, 6, 7]))
        t += seg
    hidden = torch.randn((T, d), generator=g, device=DEV).to(torch.bfloat16)
    w = W.Workload("eo8", d, T, T - 3, hidden, token_slot, apps, groups, n_slots_max=8, n_groups_max=2, C_max=1,
                   k_max=1, r_max=8, d_sae_max=S)
    out = run_gpu(w, flags=mixlib.MIX_FLAG_SAE_EDIT_ONLY, graph=True)
    st = check_parity(W.host(w), out, check_features=False)
    assert st["rows"] == T
    assert (token_slot[:T - 3] <= 5).sum() > 20 and len(set(token_slot[:T - 3].tolist())) >= 6


@pytest.mark.parametrize("rows_per_set", [(100, 200, 256, 300), (130, 40, 0, 0), (256, 256, 0, 0), (512, 100, 300, 0),
                                          (129, 1, 1, 1), (0, 384, 0, 130)])
def test_weight_sets_dealt_between_single_ctas_and_cta_pairs(rows_per_set):
    """A context of more than 128 rows has two encode kernels (single CTAs, CTA pairs) and the front kernel deals
    the call's weight sets between them by their number of 128-row tiles: two sets of two tiles and one of three
    beside a one-tile set (both kernels work), one two-tile set beside a one-tile set (single CTAs only), two
    full pairs (pairs only), four tiles + one + three (both), ... -- one captured graph, a new map per replay,
    every row against the oracle."""
    mixlib = _mixlib()
    w = W.make_replay(DEV, d=256, T_max=1024, d_sae=2048, k=16, G=4, n_probe=4, n_steer=2, n_sae_slots=8, n_edit=4)
    m = W.make_context(mixlib.Mix, w)
    T, k_max = w.T_max, w.k_max
    h_static = w.hidden.clone()
    scores = torch.empty((T, 1), dtype=torch.float32, device=DEV)
    tk_idx = torch.empty((T, k_max), dtype=torch.int32, device=DEV)
    tk_val = torch.empty((T, k_max), dtype=torch.float32, device=DEV)
    n_act = torch.empty((T,), dtype=torch.int32, device=DEV)
    m.set_feature_out(tk_idx, tk_val, n_act)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h_static, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply(h_static, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    sae_slots = {gi: [sl for sl, a in w.apps.items() if a.kind == W.KIND_SAE and a.group == gi] for gi in range(4)}
    other = [sl for sl, a in w.apps.items() if a.kind != W.KIND_SAE]
    token_slot = np.full(T, -1, dtype=np.int32)
    t = 0
    for gi, n in enumerate(rows_per_set):                      # the sets' rows interleaved with a few other rows
        for j in range(n):
            token_slot[t] = sae_slots[gi][(j // 37) % len(sae_slots[gi])]
            t += 1
        token_slot[t:t + 3] = [other[gi % len(other)], -1, other[(gi + 1) % len(other)]]
        t += 3
    n_live = t
    for rep in range(2):                                       # twice: the second replay starts from the first one's state
        m.set_slot_map(token_slot, n_live)
        h_static.copy_(w.hidden)
        scores.copy_(torch.from_numpy(np.full((T, 1), CANARY_F32, dtype=np.uint32).view(np.float32)))
        tk_idx.fill_(-559038737); n_act.fill_(-559038737)
        g.replay()
        torch.cuda.synchronize()
        w.token_slot, w.T_live = token_slot, n_live
        out = dict(hidden=W.bits(h_static), scores=scores.cpu().numpy(), topk_idx=tk_idx.cpu().numpy(),
                   topk_val=tk_val.cpu().numpy(), n_active=n_act.cpu().numpy(), status=m.get_status())
        check_parity(W.host(w), out)
    m.destroy()
