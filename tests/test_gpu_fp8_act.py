"""GPU: 8-bit encoder input (MIX_FLAG_FP8_ACT: rows quantised to E4M3 with a power-of-two scale when they are
packed, E4M3 x E4M3 tcgen05 contraction) against the oracle evaluated on the same definition."""
import numpy as np
import pytest
import torch

import workloads as W

from parity import check_parity, oracle_edit_hint, run_gpu, sample_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _flags():
    import paper_2607_22595_b200 as mixlib
    return mixlib.MIX_FLAG_FP8_W_ENC | mixlib.MIX_FLAG_FP8_ACT


@pytest.mark.parametrize("graph", [False, True])
def test_fp8_act_sae_heavy_small(graph):
    # TopK sets, two row tiles with a ragged tail per weight set, 3 k-blocks of 128, 4 feature tiles
    w = W.make_sae_heavy(DEV, d=384, d_sae=1024, k=16, T=400, R=12, G=2, n_edit=6, edit_hint=oracle_edit_hint,
                         fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags(), graph=graph)
    st = check_parity(W.host(w), out)
    assert st["rows"] == 400


def test_fp8_act_mixed_small_jumprelu_and_probes():
    w = W.make_mixed(DEV, d=512, T=900, R=20, d_sae=2048, C=4, n_probe=3, n_steer=3, G=2, n_edit=5, cap=300, mu=3.5,
                     edit_hint=oracle_edit_hint, fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags(), graph=True)
    check_parity(W.host(w), out)


def test_fp8_act_wide_rows_many_stages():
    # d = 8192: 64 k-blocks per tile, so every stage of the ring is reused 16 times per tile
    w = W.make_sae_heavy(DEV, d=8192, d_sae=512, k=8, T=130, R=5, G=1, n_edit=4, edit_hint=oracle_edit_hint,
                         fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags())
    check_parity(W.host(w), out)


def _identity_sae(d, act=W.SAE_TOPK):
    """Feature j reads input column j: code 0x38 (= 1) on the diagonal, scale 1, no bias."""
    codes = np.zeros((d, d), dtype=np.uint8)
    codes[np.arange(d), np.arange(d)] = 0x38
    g = torch.Generator(device=DEV); g.manual_seed(0)
    W_dec = torch.randn((d, d), generator=g, device=DEV).to(torch.bfloat16)
    return W.SaeWeights(d, act, d, torch.from_numpy(codes).to(DEV), torch.zeros(d, device=DEV), W_dec,
                        w_scale=torch.ones(d, device=DEV))


def test_fp8_act_quantiser_is_bit_exact_on_edge_rows():
    """With an identity encoder the TopK list of a row IS its quantised copy s * e4m3(code_i): ties, subnormal
    codes, rows scaled by powers of two, a row of zeros, the scale's edges and its floor."""
    from oracle import mi_hook as O
    d = 256
    rng = np.random.default_rng(7)
    rows = []
    base = rng.standard_normal(d)
    rows.append(base)                                                   # ordinary row
    rows.append(base * 2.0 ** 40)
    rows.append(base * 2.0 ** -60)
    rows.append(np.zeros(d))                                            # zero row: scale 1, all codes 0
    r = np.zeros(d); r[0] = 3.0; r[1:9] = np.array([54, 58, 53, 2.5 * 2.0 ** -2, 2.0 ** -3, 3 * 2.0 ** -3, -54, 432 / 1.0]) / 128
    rows.append(r)                                                      # s = 2^-7: ties 54 -> 56, 58 -> 56, subnormal ties
    r = np.zeros(d); r[5] = 448.0; r[6] = -1.0; r[7] = 2.0 ** -9; r[8] = 2.0 ** -10
    rows.append(r)                                                      # largest magnitude exactly 448: s = 1
    r = np.zeros(d); r[5] = 452.0; r[6] = 3.0
    rows.append(r)                                                      # just above: s = 2
    r = np.zeros(d); r[9] = -1.75; r[10] = 1.7421875
    rows.append(r)                                                      # 1.75 -> exactly 448 after scaling
    r = np.zeros(d); r[3] = 2.0 ** -120; r[4] = -2.0 ** -108
    rows.append(r)                                                      # below the scale's floor 2^-100: codes 0 / subnormal
    rows.append(rng.standard_normal(d) * np.exp(rng.uniform(-8, 8, d)))  # wide dynamic range inside one row
    X = O.bf16_to_f64(O.f64_to_bf16_bits(np.stack(rows)))
    T = X.shape[0]
    hidden = W.from_bits(O.f64_to_bf16_bits(X), DEV)
    app = W.SaeApp(0, np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.uint8), True)
    w = W.Workload("edges", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: _identity_sae(d)}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=d, r_max=1, d_sae_max=d, fp8_act=True)
    out = run_gpu(w, flags=_flags())
    assert out["status"] & ~_mixlib().MIX_STATUS_TOPK_GENERAL == 0
    want = O.quantize_rows_e4m3(X)
    for t in range(T):
        idx = out["topk_idx"][t]
        assert sorted(idx.tolist()) == list(range(d))
        got = np.empty(d); got[idx] = out["topk_val"][t].astype(np.float64)
        bad = np.nonzero(got != want[t])[0]
        assert bad.size == 0, "row %d: columns %s got %s want %s" % (t, bad[:6], got[bad[:6]], want[t][bad[:6]])
    assert np.array_equal(out["hidden"], W.bits(hidden))               # no edits: rows bit-exact


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


def test_fp8_act_every_code_pair_contracts_exactly():
    """One-hot rows (value 1 -> code 0x78 = 256 at scale 2^-8) read single encoder entries back: every finite
    code of the encoder must come out of the 8-bit contraction with exactly its value."""
    from oracle import mi_hook as O
    d = S = T = 256
    j, i = np.meshgrid(np.arange(S), np.arange(d), indexing="ij")
    codes = ((j * 7 + i * 3) % 256).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x00
    g = torch.Generator(device=DEV); g.manual_seed(0)
    W_dec = torch.randn((S, d), generator=g, device=DEV).to(torch.bfloat16)
    sae = W.SaeWeights(S, W.SAE_TOPK, S, torch.from_numpy(codes).to(DEV), torch.zeros(S, device=DEV), W_dec,
                       w_scale=torch.ones(S, device=DEV))
    hidden = torch.eye(T, d, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    app = W.SaeApp(0, np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.uint8), True)
    w = W.Workload("codes", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=S, r_max=1, d_sae_max=S, fp8_act=True)
    out = run_gpu(w, flags=_flags())
    want = O.e4m3_to_f64(codes)
    for t in range(T):
        idx = out["topk_idx"][t]
        assert sorted(idx.tolist()) == list(range(S))
        got = np.empty(S); got[idx] = out["topk_val"][t].astype(np.float64)
        assert np.array_equal(got, want[:, t]), "row %d: %s" % (t, np.nonzero(got != want[:, t])[0][:8])


def test_fp8_act_api_errors():
    mixlib = _mixlib()
    with pytest.raises(mixlib.MixError) as e:          # needs the 8-bit encoder
        mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256,
                   flags=mixlib.MIX_FLAG_FP8_ACT)
    assert e.value.code == -1
    with pytest.raises(mixlib.MixError) as e:          # d_model must be a multiple of 128
        mixlib.Mix(d_model=192, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256, flags=_flags())
    assert e.value.code == -3
    m = mixlib.Mix(d_model=128, T_max=8, n_slots_max=1, n_groups_max=1, k_max=4, r_max=1, d_sae_max=256, flags=_flags())
    m.destroy()


def test_fp8_act_time_out_path_leaves_the_context_usable():
    mixlib = _mixlib()
    w = W.make_sae_heavy(DEV, d=256, d_sae=512, k=8, T=200, R=6, G=2, n_edit=3, fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags() | mixlib.MIX_FLAG_TEST_STALL_ENCODE)
    assert out["status"] & mixlib.MIX_STATUS_WAIT_TIMEOUT
    out["mix"].destroy()
    out = run_gpu(w, flags=_flags())
    check_parity(W.host(w), out)


def test_fp8_act_sae_heavy_full_size_sampled_rows():
    w = W.make_sae_heavy(DEV, edit_hint=oracle_edit_hint, fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags(), graph=True)
    wh = W.host(w, only_groups=[1])
    rows = [t for t in sample_rows(wh, per_kind=6) if w.apps[int(w.token_slot[t])].group == 1][:8]
    assert len(rows) >= 4
    check_parity(wh, out, rows=rows)


def test_fp8_act_mixed_full_size_sampled_rows():
    # config 3 in the launch configuration bench.py times (JumpReLU sets: the plain-store epilogue, four warps)
    w = W.make_mixed(DEV, edit_hint=oracle_edit_hint, fp8=True, fp8_act=True)
    out = run_gpu(w, flags=_flags() | _mixlib().MIX_FLAG_RETILE_W_ENC, graph=True)
    wh = W.host(w)
    unh = np.nonzero(wh.token_slot < 0)[0]
    assert np.array_equal(out["hidden"][unh], wh.hidden[unh])        # every unhooked row is bit-identical
    rows = sample_rows(wh, per_kind=12, seed=5)
    check_parity(wh, out, rows=rows)
