"""CPU pins of the oracle's 8-bit encoder INPUT (rows quantised to E4M3 with a power-of-two scale): the
quantiser against a library conversion, brute force and hand-worked ties; the row scale against its
definition; the hook against an explicitly quantised input."""
import json
import math
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _all_bf16_up_to_448():
    bits = np.arange(1 << 16, dtype=np.uint32).astype(np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]                 # no infinities, no NaNs
    v = O.bf16_to_f64(bits)
    return v[np.abs(v) <= 448.0]


def test_quantiser_matches_the_library_conversion_on_every_bf16_value_in_range():
    v = _all_bf16_up_to_448()
    assert v.size > 30000
    lib = torch.from_numpy(v).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_quantize(v)
    # +0 / -0 carry the sign on both sides; compare the codes bit for bit
    assert np.array_equal(got, lib)


def test_quantiser_is_the_nearest_code_by_brute_force():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.uniform(-448, 448, 4000), rng.uniform(-1, 1, 4000) * 2.0 ** -5, rng.standard_normal(4000)])
    grid = O.e4m3_to_f64(np.arange(127, dtype=np.uint8))
    got = O.e4m3_to_f64(O.e4m3_quantize(x))
    best = np.min(np.abs(np.abs(x)[:, None] - grid[None, :]), axis=1)
    assert np.array_equal(np.abs(np.abs(got) - np.abs(x)), best)
    assert np.array_equal(np.signbit(got), np.signbit(x))


def test_quantiser_ties_go_to_the_even_code():
    # between 52 (0x65, odd) and 56 (0x66): 54 -> 56;  between 56 (0x66) and 60 (0x67): 58 -> 56
    # between 1 (0x38) and 1.125 (0x39): 1.0625 -> 1;  subnormals: 2^-9 * 2.5 -> 2 * 2^-9 (0x02); 2^-10 -> 0
    x = np.array([54.0, 58.0, 1.0625, 2.5 * 2.0 ** -9, 2.0 ** -10, -54.0, 3 * 2.0 ** -10, 448.0, 432.0])
    want = np.array([0x66, 0x66, 0x38, 0x02, 0x00, 0xE6, 0x02, 0x7E, 0x7E], dtype=np.uint8)
    # 3 * 2^-10 = 1.5 * 2^-9: tie between codes 1 and 2 -> 2;  432 is the tie between 416 (0x7D) and 448 (0x7E) -> 0x7E
    assert O.e4m3_quantize(x).tolist() == want.tolist()
    with pytest.raises(ValueError):
        O.e4m3_quantize(np.array([449.0]))


def test_row_scale_definition_and_edges():
    assert O.act_row_scale(np.zeros(8)) == 1.0
    assert O.act_row_scale(np.array([448.0, -3.0])) == 1.0
    assert O.act_row_scale(np.array([452.0])) == 2.0                    # next bf16 above 448
    assert O.act_row_scale(np.array([-1.0, 0.5])) == 2.0 ** -8          # 256 <= 448 < 512
    assert O.act_row_scale(np.array([1.75])) == 2.0 ** -8               # exactly 448 after scaling
    assert O.act_row_scale(np.array([1.7578125])) == 2.0 ** -7
    assert O.act_row_scale(np.array([2.0 ** -120])) == 2.0 ** -100      # floor of the scale
    assert O.act_row_scale(np.array([2.0 ** 127])) == 2.0 ** 119
    # definition, by search over exponents, on every positive bf16 value
    v = O.bf16_to_f64(np.arange(1, 0x7F80, 37, dtype=np.uint32).astype(np.uint16))
    for a in v:
        s = O.act_row_scale(np.array([a]))
        e = int(round(math.log2(s)))
        assert s == 2.0 ** e and e >= -100
        assert a / s <= 448.0
        assert e == -100 or a / (s / 2) > 448.0


def test_quantised_rows_properties():
    rng = np.random.default_rng(5)
    X = O.bf16_to_f64(O.f64_to_bf16_bits(rng.standard_normal((6, 96)) * np.array([1e-3, 0.1, 1, 7, 300, 4e4])[:, None]))
    Q = O.quantize_rows_e4m3(X)
    for x, q in zip(X, Q):
        s = O.act_row_scale(x)
        # normal codes: relative error <= 2^-4; subnormal codes: absolute error <= s * 2^-10
        err = np.abs(q - x)
        assert np.all(err <= np.maximum(np.abs(x) * 2.0 ** -4, s * 2.0 ** -10))
        i = int(np.argmax(np.abs(x)))
        assert abs(q[i]) >= 224 * s                 # the largest entry uses the top binade or the one below
        assert np.array_equal(O.quantize_rows_e4m3(q[None, :])[0], q)          # idempotent
        assert np.array_equal(O.quantize_rows_e4m3(4 * x[None, :])[0], 4 * q)  # equivariant to powers of two
        assert np.array_equal(O.quantize_rows_e4m3(-x[None, :])[0], -q)
    assert np.array_equal(O.quantize_rows_e4m3(np.zeros((1, 8)))[0], np.zeros(8))


def test_hand_worked_row():
    with open(os.path.join(GOLDEN, "hand_worked_fp8_act_d4.json")) as f:
        gold = json.load(f)
    x = np.array(gold["x"])
    assert O.act_row_scale(x) == gold["scale"]
    assert O.e4m3_quantize(x / gold["scale"]).tolist() == gold["codes"]
    assert O.quantize_rows_e4m3(x[None, :])[0].tolist() == gold["x_seen_by_encoder"]
    codes = np.array(gold["W_enc_codes"], dtype=np.uint8)
    z = O.sae_preact(O.quantize_rows_e4m3(x[None, :]), codes, np.array(gold["b_enc"], dtype=np.float32),
                     w_scale=np.array(gold["W_enc_scale"], dtype=np.float32))[0]
    assert z.tolist() == gold["z"]


def test_hook_with_8bit_input_equals_hook_on_explicitly_quantised_encoder_input():
    g = torch.Generator().manual_seed(4)
    d, S, T = 64, 256, 12
    sae = W.make_sae_weights(g, "cpu", d, S, W.SAE_JUMPRELU, theta_range=(0.05, 0.3), fp8=True)
    hidden = (torch.randn((T, d), generator=g) * 3).to(torch.bfloat16)
    idx = np.array([3, 77, 200], dtype=np.int32)
    app = W.SaeApp(0, idx, np.array([5.0, 0.0, 2.0], np.float32),
                   np.array([W.EDIT_CLAMP, W.EDIT_ABLATE, W.EDIT_CLAMP], np.uint8), True)
    w = W.Workload("q", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                   n_groups_max=1, C_max=1, k_max=1, r_max=3, d_sae_max=S)
    wh = W.host(w)
    wh.fp8_act = True
    res = O.apply_hook(wh, keep_z=True)
    X = O.bf16_to_f64(W.bits(hidden))
    Wf = O.encoder_rows_f64(W.bits(sae.W_enc), W.bits(sae.w_scale))
    for t in range(T):
        s = O.act_row_scale(X[t])
        xq = O.e4m3_to_f64(O.e4m3_quantize(X[t] / s)) * s
        z = Wf @ xq + W.bits(sae.b_enc).astype(np.float64)
        # the error-term form: only the edited features move the row, and by (f' - f) W_dec[j] on the UNQUANTISED row
        f = np.where(z > W.bits(sae.theta).astype(np.float64), z, 0.0)
        y = X[t].copy()
        for j, f_new in zip(idx, [5.0, 0.0, 2.0]):          # clamp to 5, ablate, clamp to 2
            y += (f_new - f[j]) * O.bf16_to_f64(W.bits(sae.W_dec)[j])
        assert np.allclose(res.y[t], y, rtol=1e-12, atol=1e-12)
    # and it differs from the unquantised hook (the option is not a no-op)
    wh.fp8_act = False
    res0 = O.apply_hook(wh)
    assert any(not np.array_equal(res0.y[t], res.y[t]) for t in range(T))
