"""CPU pins of the oracle's 8-bit (E4M3) encoder: the decode against the format's definition, known
codes and a library conversion; the pre-activations against an explicitly dequantised matrix."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import mi_hook as O


def test_e4m3_known_codes():
    # sign.eeee.mmm, bias 7: 0x38 = 0.0111.000 = 1; 0x3C = 1.5; 0x40 = 2; 0x7E = 0.1111.110 = 2^8 * 1.75 = 448 (largest);
    # 0x08 = 2^-6 (smallest normal); 0x01 = 2^-9 (smallest subnormal); 0x07 = 7 * 2^-9; 0x00 / 0x80 = +-0
    codes = np.array([0x38, 0x3C, 0x40, 0x7E, 0x08, 0x01, 0x07, 0x00, 0x80, 0xB8, 0xFE, 0x30], dtype=np.uint8)
    want = [1.0, 1.5, 2.0, 448.0, 2.0 ** -6, 2.0 ** -9, 7 * 2.0 ** -9, 0.0, -0.0, -1.0, -448.0, 0.5]
    got = O.e4m3_to_f64(codes)
    assert got.tolist() == want
    assert np.signbit(got[8]) and not np.signbit(got[7])
    assert np.isnan(O.e4m3_to_f64(np.array([0x7F, 0xFF], dtype=np.uint8))).all()


def test_e4m3_all_codes_match_the_library_conversion():
    codes = torch.arange(256, dtype=torch.int64).to(torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = O.e4m3_to_f64(codes.numpy())
    finite = ~np.isnan(lib)
    assert finite.sum() == 254
    assert np.array_equal(got[finite], lib[finite]) and np.isnan(got[~finite]).all()
    # monotone in the code within each sign, spacing doubles every 8 codes
    pos = got[:0x7F]
    assert (np.diff(pos) > 0).all()
    assert np.allclose(np.diff(pos)[8:16], 2.0 ** -9) and np.allclose(np.diff(pos)[16:24], 2.0 ** -8)


def test_fp8_preact_equals_explicit_dequantised_matmul_and_term_sum():
    rng = np.random.default_rng(3)
    S, d, n = 40, 24, 5
    codes = rng.integers(0, 256, size=(S, d)).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x30                      # no NaN codes
    scale = rng.uniform(1e-3, 1e-2, size=S).astype(np.float32)
    b = rng.standard_normal(S).astype(np.float32)
    X = rng.standard_normal((n, d))
    Wd = codes.copy()
    Wf = torch.from_numpy(Wd).view(torch.float8_e4m3fn).to(torch.float64).numpy() * scale.astype(np.float64)[:, None]
    Z = O.sae_preact(X, codes, b, w_scale=scale)
    assert np.allclose(Z, X @ Wf.T + b.astype(np.float64), rtol=1e-13, atol=1e-13)
    # one entry term by term (a transposed operand or a scale applied to the wrong axis fails here)
    j, r = 17, 3
    z = float(b[j]) + float(scale[j]) * sum(float(O.e4m3_to_f64(codes[j, i:i + 1])[0]) * X[r, i] for i in range(d))
    assert Z[r, j] == pytest.approx(z, rel=1e-13)
    # scaling one feature's scale scales only that pre-activation (minus its bias)
    scale2 = scale.copy(); scale2[j] *= 2
    Z2 = O.sae_preact(X, codes, b, w_scale=scale2)
    assert np.allclose(Z2[:, j] - b[j], 2 * (Z[:, j] - b[j]), rtol=1e-13)
    assert np.array_equal(np.delete(Z2, j, axis=1), np.delete(Z, j, axis=1))


def test_fp8_generator_roundtrip_and_hook():
    g = torch.Generator().manual_seed(1)
    sae = W.make_sae_weights(g, "cpu", 64, 256, W.SAE_TOPK, k=8, fp8=True)
    assert sae.W_enc.dtype == torch.uint8 and sae.w_scale.shape == (256,)
    Wq = O.encoder_rows_f64(W.bits(sae.W_enc), W.bits(sae.w_scale))
    # the largest entry of every row sits at the format's maximum: |w| max = 448 * scale
    assert np.allclose(np.abs(Wq).max(axis=1), 448.0 * W.bits(sae.w_scale).astype(np.float64), rtol=1e-6)
    # a hook call on an 8-bit weight set runs end to end and keeps unhooked rows bit-exact
    hidden = torch.randn((6, 64), generator=g).to(torch.bfloat16)
    app = W.SaeApp(0, np.array([3], np.int32), np.array([2.0], np.float32), np.array([0], np.uint8), True)
    w = W.host(W.Workload("f", 64, 6, 6, hidden, np.array([0, -1, 0, 0, -1, 0], np.int32), {0: app}, {0: sae},
                          n_slots_max=1, n_groups_max=1, k_max=8, r_max=1, d_sae_max=256))
    r = O.apply_hook(w)
    assert np.array_equal(r.out_bits[1], w.hidden[1]) and len(r.topk[0]) == 8
    # single clamp with the error term: displacement along decoder row 3 only
    disp = r.y[0] - O.bf16_to_f64(w.hidden[0])
    dec = O.bf16_to_f64(w.groups[0].W_dec[3])
    coef = disp @ dec / (dec @ dec)
    assert np.allclose(disp, coef * dec, atol=1e-12)
