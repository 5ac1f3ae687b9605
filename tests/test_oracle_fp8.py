"""Pins of the FP8 latent-cache part of the oracle (CPU only).

The paper only names FP8 quantisation (abstract); the stored format is this library's own (parity unpinned by the
paper).  What can be pinned is pinned: the e4m3 number format against the values its published definition gives and
against torch's float8_e4m3fn conversion (an independent implementation), the quantiser's error bound, and that the
attention over an FP8 cache is Eq. 9 over the dequantised rows.
"""
import numpy as np
import torch

from oracle import mla_oracle as orc


def test_e4m3_values_of_the_format_definition():
    # 1 sign, 4 exponent bits (bias 7), 3 mantissa bits; subnormals below 2^-6; no infinities; S.1111.111 is NaN
    d = lambda c: float(orc.e4m3_decode(np.array([c], dtype=np.uint8))[0])
    assert d(0x00) == 0.0 and d(0x01) == 2.0 ** -9 and d(0x07) == 7 * 2.0 ** -9
    assert d(0x08) == 2.0 ** -6 and d(0x38) == 1.0 and d(0x39) == 1.125 and d(0x40) == 2.0
    assert d(0x7E) == 448.0 and d(0xFE) == -448.0 and d(0xC0) == -2.0
    assert np.isnan(d(0x7F)) and np.isnan(d(0xFF))
    v = orc.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    assert np.all(np.diff(v) > 0)                                   # codes order the non-negative values


def test_e4m3_agrees_with_torch_float8():
    codes = torch.arange(256, dtype=torch.uint8)
    want = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = orc.e4m3_decode(codes.numpy())
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000) * 50, rng.standard_normal(20000) * 0.01, [0.0, 448.0, -448.0, 2.0 ** -10]])
    x = x[np.abs(x) <= 448.0]                                        # torch does not saturate; the oracle does
    t = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = orc.e4m3_encode(x.astype(np.float32).astype(np.float64))
    nz = orc.e4m3_decode(mine) != 0                                  # +0 / -0 differ in the sign bit only
    assert np.array_equal(mine[nz], t[nz])


def test_e4m3_round_trip_ties_and_saturation():
    finite = np.array([c for c in range(256) if (c & 0x7F) != 0x7F and c != 0x80], dtype=np.uint8)
    assert np.array_equal(orc.e4m3_encode(orc.e4m3_decode(finite)), finite)
    e = lambda x: int(orc.e4m3_encode(np.array([x]))[0])
    assert e(1.0625) == 0x38 and e(1.1875) == 0x3A                   # ties go to the even mantissa
    assert e(2.0 ** -10) == 0x00 and e(3 * 2.0 ** -10) == 0x02
    assert e(1e9) == 0x7E and e(-1e9) == 0xFE and e(449.0) == 0x7E    # saturates, never NaN


def test_quantiser_error_bound_and_exact_rows():
    rng = np.random.default_rng(4)
    r, dR = 64, 16
    rows = rng.standard_normal((50, r + dR)) * rng.uniform(0.01, 30, size=(50, 1))
    codes, k_pe, scale = orc.quantize_latent_rows(rows, r)
    back = orc.dequantize_latent_rows(codes, k_pe, scale)
    amax = np.abs(rows[:, :r]).max(axis=1, keepdims=True)
    assert np.all(np.abs(back[:, :r] - rows[:, :r]) <= amax * 2.0 ** -4 / 1.75 + 1e-12)   # half an ulp at the top binade
    assert np.all(np.abs(back[:, r:] - rows[:, r:]) <= np.abs(rows[:, r:]) * 2.0 ** -8 + 1e-12)  # bf16 rounding
    assert np.all(np.abs(orc.e4m3_decode(codes)).max(axis=1) == 448.0)
    # rows made of representable numbers with maximum 448 come back bit for bit (scale = 1)
    grid = orc.e4m3_decode(rng.integers(0, 0x7F, size=(5, r)).astype(np.uint8)) * rng.choice([-1.0, 1.0], size=(5, r))
    grid[:, 0] = 448.0
    kp = orc._round_bf16(rng.standard_normal((5, dR)))
    codes, k_pe, scale = orc.quantize_latent_rows(np.concatenate([grid, kp], axis=1), r)
    assert np.all(scale == 1.0)
    assert np.array_equal(orc.dequantize_latent_rows(codes, k_pe, scale), np.concatenate([grid, kp], axis=1))
    z = orc.quantize_latent_rows(np.zeros((1, r + dR)), r)
    assert z[2][0] == 1.0 and not np.any(z[0])


def test_attention_over_an_fp8_cache_is_eq9_over_the_dequantised_rows():
    rng = np.random.default_rng(5)
    H, dn, dR, dv, r, P = 3, 4, 6, 5, 16, 4
    lens = [9, 4]
    table = np.array([[3, 0, 5], [2, -1, -1]], dtype=np.int32)
    rows = rng.standard_normal((6, P, r + dR))
    codes, k_pe, scale = orc.quantize_latent_rows(rows, r)
    codes[4] = 0x7F                                                  # an unowned page full of NaN codes is never touched
    qn, qp = rng.standard_normal((2, 1, H, dn)), rng.standard_normal((2, 1, H, dR))
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    out, lse = orc.mla_decode_fp8_cache(qn, qp, w_uk, w_uv, codes, k_pe, scale, table, lens, 0.3, page_size=P)
    deq = orc.dequantize_latent_rows(codes, k_pe, scale)
    deq[4] = 0.0
    want, want_lse = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, deq, table, lens, 0.3, page_size=P)
    assert np.array_equal(out, want) and np.array_equal(lse, want_lse)
    # and it stays within the quantiser's error of the unquantised attention
    exact, _ = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, rows, table, lens, 0.3, page_size=P)
    assert np.abs(out - exact).max() < 0.2 and np.abs(out - exact).max() > 0


def test_append_into_an_fp8_cache():
    rng = np.random.default_rng(6)
    r, dR, D, P = 16, 8, 12, 4
    w = rng.standard_normal((r + dR, D)) / 3
    x = rng.standard_normal((2, D))
    table = np.array([[1, 0], [2, -1]], dtype=np.int32)
    codes = np.full((3, P, r), 0x7F, dtype=np.uint8)
    k_pe, scale = np.full((3, P, dR), np.nan), np.full((3, P), np.nan)
    orc.latent_append_fp8(x, w, [5, 0], table, codes, k_pe, scale, r, page_size=P)
    plain = np.full((3, P, r + dR), np.nan)
    orc.latent_append(x, w, [5, 0], table, plain, r, page_size=P)
    for page, off in ((0, 1), (2, 0)):                               # position 5 -> page_table[0][1] = 0, offset 1
        c, k, s = orc.quantize_latent_rows(plain[page, off], r)
        assert np.array_equal(codes[page, off], c) and np.array_equal(k_pe[page, off], k) and scale[page, off] == s
    untouched = np.ones((3, P), bool); untouched[0, 1] = untouched[2, 0] = False
    assert np.all(codes[untouched] == 0x7F) and np.all(np.isnan(scale[untouched]))
