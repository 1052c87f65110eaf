"""GPU: 8-bit (E4M3 codes x per-feature scale) encoder weights with the hidden state kept in bf16 (each row goes
to the 8-bit tcgen05 contraction as the exact sum of two E4M3 operands), against the oracle evaluated on the same
codes and scales."""
import numpy as np
import pytest
import torch

import workloads as W

from parity import check_parity, oracle_edit_hint, run_gpu, sample_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


@pytest.mark.parametrize("graph", [False, True])
def test_fp8_sae_heavy_small(graph):
    # TopK sets, two row tiles with a ragged tail per weight set, 3 k-blocks of 128, 4 feature tiles
    w = W.make_sae_heavy(DEV, d=384, d_sae=1024, k=16, T=400, R=12, G=2, n_edit=6, edit_hint=oracle_edit_hint, fp8=True)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_FP8_W_ENC, graph=graph)
    st = check_parity(W.host(w), out)
    assert st["rows"] == 400


def test_fp8_mixed_small_jumprelu_and_probes():
    w = W.make_mixed(DEV, d=512, T=900, R=20, d_sae=2048, C=4, n_probe=3, n_steer=3, G=2, n_edit=5, cap=300, mu=3.5,
                     edit_hint=oracle_edit_hint, fp8=True)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_FP8_W_ENC, graph=True)
    check_parity(W.host(w), out)


def test_fp8_wide_rows_many_stages():
    # d = 4096: 32 k-blocks per tile, so every stage of the ring is reused 10 times per tile
    w = W.make_sae_heavy(DEV, d=4096, d_sae=512, k=8, T=130, R=5, G=1, n_edit=4, edit_hint=oracle_edit_hint, fp8=True)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_FP8_W_ENC)
    check_parity(W.host(w), out)


def test_fp8_every_code_contracts_exactly():
    """One-hot rows read single encoder entries back: every one of the 254 finite codes, subnormal ones
    included, must come out of the contraction with exactly its value."""
    from oracle import mi_hook as O
    mixlib = _mixlib()
    d = S = T = 256
    j, i = np.meshgrid(np.arange(S), np.arange(d), indexing="ij")
    codes = ((j * 7 + i * 3) % 256).astype(np.uint8)          # every column holds every code once (7 is odd)
    codes[(codes & 0x7F) == 0x7F] = 0x00                        # no NaN codes
    g = torch.Generator(device=DEV); g.manual_seed(0)
    W_dec = torch.randn((S, d), generator=g, device=DEV).to(torch.bfloat16)
    sae = W.SaeWeights(S, W.SAE_TOPK, S, torch.from_numpy(codes).to(DEV), torch.zeros(S, device=DEV), W_dec,
                       w_scale=torch.ones(S, device=DEV))
    hidden = torch.eye(T, d, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    app = W.SaeApp(0, np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.uint8), True)
    w = W.Workload("codes", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=S, r_max=1, d_sae_max=S)
    out = run_gpu(w, flags=mixlib.MIX_FLAG_FP8_W_ENC)
    want = O.e4m3_to_f64(codes)                                 # [S, d]; row t of the batch reads column t
    for t in range(T):
        idx = out["topk_idx"][t]
        assert sorted(idx.tolist()) == list(range(S))
        got = np.empty(S); got[idx] = out["topk_val"][t].astype(np.float64)
        assert np.array_equal(got, want[:, t]), "row %d: %s" % (t, np.nonzero(got != want[:, t])[0][:8])
    assert np.array_equal(out["hidden"], W.bits(hidden))        # no edits: bit-exact rows


def test_fp8_duplicate_features_take_the_flagged_path_with_the_tie_rule():
    # identical code rows and scales give exactly equal pre-activations: the lower feature id must win,
    # through the candidate merge or (when a tile hides more than 8 of them) the exact fallback encode
    mixlib = _mixlib()
    d, S, k, T = 128, 512, 8, 40
    g = torch.Generator(device=DEV); g.manual_seed(2)
    sae = W.make_sae_weights(g, DEV, d, S, W.SAE_TOPK, k=k, fp8=True)
    sae.W_enc[1:12] = sae.W_enc[0]
    sae.w_scale[0:12] = sae.w_scale[0] * 4.0          # make the duplicated feature win
    sae.b_enc[0:12] = 0.25
    hidden = torch.randn((T, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    app = W.SaeApp(0, np.array([0], np.int32), np.array([1.0], np.float32), np.array([0], np.uint8), True)
    w = W.Workload("dup8", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=k, r_max=1, d_sae_max=S)
    out = run_gpu(w, flags=mixlib.MIX_FLAG_FP8_W_ENC)
    check_parity(W.host(w), out, expect_status=None)
    assert out["status"] & ~mixlib.MIX_STATUS_TOPK_GENERAL == 0


def test_fp8_api_errors():
    mixlib = _mixlib()
    for bad in (mixlib.MIX_FLAG_ENCODE_SIMT, mixlib.MIX_FLAG_SAE_EDIT_ONLY):
        with pytest.raises(mixlib.MixError) as e:
            mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256,
                       flags=mixlib.MIX_FLAG_FP8_W_ENC | bad)
        assert e.value.code == -1
    with pytest.raises(mixlib.MixError) as e:          # k-blocks of 128 codes: d_model must be a multiple of 128
        mixlib.Mix(d_model=192, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256,
                   flags=mixlib.MIX_FLAG_FP8_W_ENC)
    assert e.value.code == -3
    m = mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256,
                   flags=mixlib.MIX_FLAG_FP8_W_ENC)
    g = torch.Generator(device=DEV); g.manual_seed(0)
    sae = W.make_sae_weights(g, DEV, 128, 256, W.SAE_TOPK, k=4, fp8=True)
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_weights(0, 256, sae.act, 4, sae.W_enc, sae.b_enc, sae.W_dec)             # no scale
    assert e.value.code == -1
    b_dec = torch.zeros(128, device=DEV)
    with pytest.raises(mixlib.MixError) as e:
        m.register_sae_weights(0, 256, sae.act, 4, sae.W_enc, sae.b_enc, sae.W_dec, b_dec=b_dec, center_input=True,
                               w_scale=sae.w_scale)
    assert e.value.code == -1
    m.register_sae_weights(0, 256, sae.act, 4, sae.W_enc, sae.b_enc, sae.W_dec, w_scale=sae.w_scale)
    m.destroy()


def test_fp8_sae_heavy_full_size_sampled_rows():
    w = W.make_sae_heavy(DEV, edit_hint=oracle_edit_hint, fp8=True)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_FP8_W_ENC, graph=True)
    wh = W.host(w, only_groups=[1])                            # decoding 268 M codes per set on the host is slow
    rows = [t for t in sample_rows(wh, per_kind=6) if w.apps[int(w.token_slot[t])].group == 1][:8]
    assert len(rows) >= 4
    check_parity(wh, out, rows=rows)


def test_fp8_bf16_rows_reach_the_encoder_exactly():
    """The hidden state is NOT quantised by MIX_FLAG_FP8_W_ENC alone: with an identity encoder (code 0x38 = 1 on the
    diagonal) the TopK list of a row is the row itself, to the last bit for entries of at least 2^-10 of the row's
    largest magnitude (hi + lo is exact there) and within 2^-10 of the row scale below that."""
    from oracle import mi_hook as O
    d = 256
    codes = np.zeros((d, d), dtype=np.uint8)
    codes[np.arange(d), np.arange(d)] = 0x38
    g = torch.Generator(device=DEV); g.manual_seed(0)
    W_dec = torch.randn((d, d), generator=g, device=DEV).to(torch.bfloat16)
    sae = W.SaeWeights(d, W.SAE_TOPK, d, torch.from_numpy(codes).to(DEV), torch.zeros(d, device=DEV), W_dec,
                       w_scale=torch.ones(d, device=DEV))
    rng = np.random.default_rng(9)
    rows = [rng.standard_normal(d), rng.standard_normal(d) * 2.0 ** 30, rng.standard_normal(d) * 2.0 ** -40, np.zeros(d),
            rng.standard_normal(d) * np.exp(rng.uniform(-12, 12, d))]
    X = O.bf16_to_f64(O.f64_to_bf16_bits(np.stack(rows)))
    T = X.shape[0]
    hidden = W.from_bits(O.f64_to_bf16_bits(X), DEV)
    app = W.SaeApp(0, np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.uint8), True)
    w = W.Workload("rows", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=d, r_max=1, d_sae_max=d)
    out = run_gpu(w, flags=_mixlib().MIX_FLAG_FP8_W_ENC)
    for t in range(T):
        idx = out["topk_idx"][t]
        assert sorted(idx.tolist()) == list(range(d))
        got = np.empty(d); got[idx] = out["topk_val"][t].astype(np.float64)
        amax = np.abs(X[t]).max()
        s = O.act_row_scale(X[t])                       # the same power-of-two scale the split uses
        big = np.abs(X[t]) >= 0.25 * s
        assert np.array_equal(got[big], X[t][big]), "row %d" % t
        assert np.all(np.abs(got - X[t]) <= 2.0 ** -10 * s), "row %d" % t
        assert amax == 0 or np.abs(got - X[t]).max() <= 4.5e-6 * amax
