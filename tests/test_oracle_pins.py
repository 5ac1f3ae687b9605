"""Pins of the fp64 oracle against what the paper and the mathematics fix (CPU only).

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or index,
transposed operand, wrong group mapping, wrong scale) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import mla_oracle as orc
from tests import lifts

TOL = 1e-10


# ---------------------------------------------------------------- RoPE (Sec. 3.1, Eq. 1; App. B)
def test_rope_is_complex_multiplication():
    # Sec. 3.1: pair l is a complex number (odd index real, even index imaginary, 1-based);
    # rotating it to position t multiplies it by exp(i t theta_l).
    rng = np.random.default_rng(0)
    d, theta = 16, 10000.0
    x = rng.standard_normal((5, d))
    pos = np.array([0, 1, 7, 1000, 131071])
    z = (x[:, 0::2] + 1j * x[:, 1::2]) * np.exp(1j * pos[:, None] * theta ** (-2 * np.arange(d // 2) / d))
    got = orc.rope(x, pos, theta)
    assert np.allclose(got[:, 0::2], z.real, atol=1e-9) and np.allclose(got[:, 1::2], z.imag, atol=1e-9)


def test_rope_closed_forms():
    # position 0 is the identity; norms are preserved; the first pair turns at 1 rad per position
    # (theta_1 = 1) and the last at theta**(-(d-2)/d).
    x = np.arange(1.0, 9.0)
    assert np.array_equal(orc.rope(x, 0), x)
    y = orc.rope(x, 12345)
    assert abs(np.linalg.norm(y) - np.linalg.norm(x)) < 1e-9
    e = np.zeros(8); e[0] = 1.0
    y = orc.rope(e, 2.0)
    assert abs(y[0] - math.cos(2.0)) < 1e-15 and abs(y[1] - math.sin(2.0)) < 1e-15
    e = np.zeros(8); e[6] = 1.0
    y = orc.rope(e, 3.0, theta=10000.0)
    ang = 3.0 * 10000.0 ** (-6.0 / 8.0)
    assert abs(y[6] - math.cos(ang)) < 1e-15 and abs(y[7] - math.sin(ang)) < 1e-15


def test_rope_relative_position_identity():
    # App. B: S_l = cos((t-j)th_l)(qx.kx + qy.ky) + sin((t-j)th_l)(qx.ky - qy.kx).
    rng = np.random.default_rng(1)
    d, theta = 64, 10000.0
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    th = theta ** (-2 * np.arange(d // 2) / d)
    for t, j in [(5, 5), (9, 2), (8191, 17), (100, 131000)]:
        lhs = orc.rope(q, t, theta) @ orc.rope(k, j, theta)
        rhs = np.sum(np.cos((t - j) * th) * (q[0::2] * k[0::2] + q[1::2] * k[1::2])
                     + np.sin((t - j) * th) * (q[0::2] * k[1::2] - q[1::2] * k[0::2]))
        assert abs(lhs - rhs) < 1e-8
    # hence a common shift of both positions changes nothing
    assert abs(orc.rope(q, 40) @ orc.rope(k, 3) - orc.rope(q, 1040) @ orc.rope(k, 1003)) < 1e-8


def test_rope_inner_product_invariant_under_per_frequency_rotation_across_heads():
    # Eq. 18: the same orthogonal U_l applied to the real and to the imaginary parts of
    # frequency l across all heads leaves the RoPE-hat inner product unchanged.
    rng = np.random.default_rng(2)
    g, d = 4, 8
    q, k = rng.standard_normal(g * d), rng.standard_normal(g * d)
    base = lifts.rope_hat(q, 11, d) @ lifts.rope_hat(k, 4, d)

    def mix(v, us):
        v = v.reshape(g, d).copy()
        for l in range(d // 2):
            v[:, 2 * l] = us[l] @ v[:, 2 * l]
            v[:, 2 * l + 1] = us[l] @ v[:, 2 * l + 1]
        return v.reshape(-1)
    us = [np.linalg.qr(rng.standard_normal((g, g)))[0] for _ in range(d // 2)]
    assert abs(lifts.rope_hat(mix(q, us), 11, d) @ lifts.rope_hat(mix(k, us), 4, d) - base) < 1e-9


# ---------------------------------------------------------------- attention core, closed forms
def _one_seq(rows, P=64):
    rng = np.random.default_rng(99)
    return lifts.paged(np.asarray(rows, np.float64), P, rng)


def test_single_token_returns_its_value():
    rng = np.random.default_rng(3)
    H, dn, dR, dv, r = 3, 4, 2, 5, 6
    c = rng.standard_normal((1, r + dR))
    pg = _one_seq(c)
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    qn, qp = rng.standard_normal((1, 1, H, dn)), rng.standard_normal((1, 1, H, dR))
    out, lse = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, pg['cache'], pg['page_table'], pg['seqlens'], 0.3)
    for h in range(H):
        assert np.allclose(out[0, 0, h], w_uv[h] @ c[0, :r], atol=TOL)
        z = (qn[0, 0, h] @ (w_uk[h] @ c[0, :r]) + qp[0, 0, h] @ c[0, r:]) * 0.3
        assert abs(lse[0, 0, h] - z) < TOL


def test_zero_scale_is_uniform_mean_and_identical_rows_return_the_row():
    rng = np.random.default_rng(4)
    H, dn, dR, dv, r, L = 2, 4, 2, 3, 8, 150
    rows = rng.standard_normal((L, r + dR))
    pg = _one_seq(rows)
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    qn, qp = rng.standard_normal((1, 1, H, dn)), rng.standard_normal((1, 1, H, dR))
    out, lse = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, pg['cache'], pg['page_table'], pg['seqlens'], 0.0)
    for h in range(H):
        assert np.allclose(out[0, 0, h], w_uv[h] @ rows[:, :r].mean(0), atol=TOL)
        assert abs(lse[0, 0, h] - math.log(L)) < TOL
    same = np.repeat(rows[:1], L, axis=0)
    pg = _one_seq(same)
    out, _ = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, pg['cache'], pg['page_table'], pg['seqlens'], 0.7)
    for h in range(H):
        assert np.allclose(out[0, 0, h], w_uv[h] @ rows[0, :r], atol=TOL)


def test_two_token_softmax_with_exact_weights():
    # scores (0, ln 3) -> weights (1/4, 3/4); the rope part contributes ln 3 through q_pe.k_pe,
    # the latent part contributes 0 to the score but carries the values 10 and 20.
    w_uk = np.array([[[1.0, 0.0]]])             # H=1, dn=1, r=2: k^C = c[0]
    w_uv = np.array([[[0.0, 2.0]]])             # v = 2 * c[1]
    rows = np.array([[0.0, 10.0, 0.0], [0.0, 20.0, math.log(3.0)]])   # [c0, c1, k_pe]
    pg = _one_seq(rows)
    qn, qp = np.array([[[[5.0]]]]), np.array([[[[2.0]]]])
    out, lse = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, pg['cache'], pg['page_table'], pg['seqlens'], 0.5)
    assert abs(out[0, 0, 0, 0] - 2.0 * (0.25 * 10.0 + 0.75 * 20.0)) < 1e-12
    assert abs(lse[0, 0, 0] - math.log(4.0)) < 1e-12
    # and the no-RoPE term really enters the score: move the ln 3 into the latent
    rows = np.array([[0.0, 10.0, 0.0], [math.log(3.0), 20.0, 0.0]])
    pg = _one_seq(rows)
    out, _ = orc.mla_decode_mha_form(np.array([[[[2.0]]]]), qp, w_uk, w_uv, pg['cache'], pg['page_table'],
                                     pg['seqlens'], 0.5)
    assert abs(out[0, 0, 0, 0] - 2.0 * (0.25 * 10.0 + 0.75 * 20.0)) < 1e-12


def _tiny_case(seed=1, seqlens=(17, 64), S=1, shape=None):
    from paper_2502_07864_b200 import synth
    shape = shape or synth.TINY
    if S != shape.S:
        shape = synth.MLAShape(**{**shape.__dict__, 'S': S})
    return shape, lifts.case_f64(synth.make_decode_case(shape, list(seqlens), seed, nan_tails=True))


def test_brute_force_scalar_loops_on_tiny_config():
    # Eq. 8 and Eq. 9 (left) spelled out element by element in Python scalars.
    shape, c = _tiny_case()
    scale = 1.0 / math.sqrt(shape.dn + shape.dR)
    out, lse = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'],
                                       c['page_table'], c['seqlens'], scale)
    r, P = shape.r, shape.page_size
    for b in range(2):
        L = int(c['seqlens'][b])
        for h in (0, 3, 7):
            zs = []
            vs = []
            for j in range(L):
                row = c['cache'][int(c['page_table'][b][j // P])][j % P]
                z = 0.0
                for a in range(shape.dn):
                    kc = sum(c['w_uk'][h][a][m] * row[m] for m in range(r))
                    z += c['q_nope'][b][0][h][a] * kc
                for a in range(shape.dR):
                    z += c['q_pe'][b][0][h][a] * row[r + a]
                zs.append(z * scale)
                vs.append([sum(c['w_uv'][h][a][m] * row[m] for m in range(r)) for a in range(shape.dv)])
            den = sum(math.exp(z) for z in zs)
            for a in range(shape.dv):
                o = sum(math.exp(zs[j]) / den * vs[j][a] for j in range(L))
                assert abs(o - out[b, 0, h, a]) < 1e-10
            assert abs(math.log(den) - lse[b, 0, h]) < 1e-10


# ---------------------------------------------------------------- Absorb == MHA form (Eq. 9; App. A.2.2)
@pytest.mark.parametrize('G', [1, 2, 3, 7, 40])
def test_absorbed_form_equals_mha_form_for_any_partition(G):
    shape, c = _tiny_case(seed=5, seqlens=(17, 64, 200, 1, 129))
    scale = 1.0 / math.sqrt(shape.dn + shape.dR)
    a = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                c['seqlens'], scale)
    b = orc.mla_decode_absorbed_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'],
                                     c['page_table'], c['seqlens'], scale, G=G)
    assert np.abs(a[0] - b[0]).max() < TOL and np.abs(a[1] - b[1]).max() < TOL


# ---------------------------------------------------------------- GQA -> MLA lifts (Sec. 4.1; App. A.2.1)
def test_grouped_attention_matches_torch_sdpa():
    # pins the independent GQA routine (group index, scale, softmax, value sum) to a library routine
    rng = np.random.default_rng(6)
    h, g, T, dq, dv = 8, 2, 33, 12, 12
    q, k, v = rng.standard_normal((h, dq)), rng.standard_normal((T, g, dq)), rng.standard_normal((T, g, dv))
    mine = orc.grouped_attention(q, k, v, 0.37)
    tq = torch.tensor(q)[None, :, None, :]
    tk = torch.tensor(k).permute(1, 0, 2)[None]
    tv = torch.tensor(v).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.37, enable_gqa=True)
    assert np.abs(mine - ref[0, :, 0, :].numpy()).max() < 1e-12


def test_selector_lift_reproduces_gqa():
    rng = np.random.default_rng(7)
    ref, m = lifts.selector_lift(rng)
    out, _ = orc.mla_decode_mha_form(m['q_nope'], m['q_pe'], m['w_uk'], m['w_uv'], m['cache'],
                                     m['page_table'], m['seqlens'], m['scale'])
    assert np.abs(out[0, 0] - ref).max() < TOL
    out2, _ = orc.mla_decode_absorbed_form(m['q_nope'], m['q_pe'], m['w_uk'], m['w_uv'], m['cache'],
                                           m['page_table'], m['seqlens'], m['scale'], G=3)
    assert np.abs(out2[0, 0] - ref).max() < TOL
    # Eq. 12: the paper rotates after absorbing; the selector moves whole d-blocks, so both orders agree
    q_hat = orc.absorb(m['q_nope'], m['q_pe'], m['w_uk'])[0, 0]
    g, d = m['g'], m['d']
    for i in range(q_hat.shape[0]):
        absorbed_first = m['w_uk'][i].T @ m['q_raw'][i]
        rotated = lifts.rope_hat(absorbed_first[:g * d], m['t'], d)
        assert np.abs(rotated - q_hat[i, :g * d]).max() < TOL


def test_replicated_lift_reproduces_grouped_attention():
    rng = np.random.default_rng(8)
    ref, m = lifts.replicated_lift(rng)
    out, _ = orc.mla_decode_mha_form(m['q_nope'], m['q_pe'], m['w_uk'], m['w_uv'], m['cache'],
                                     m['page_table'], m['seqlens'], m['scale'])
    assert np.abs(out[0, 0] - ref).max() < TOL
    # a wrong head->group map must be visible: rolling the heads' weights by one breaks the match
    bad, _ = orc.mla_decode_mha_form(m['q_nope'], m['q_pe'], np.roll(m['w_uk'], 1, 0), m['w_uv'], m['cache'],
                                     m['page_table'], m['seqlens'], m['scale'])
    assert np.abs(bad[0, 0] - ref).max() > 1e-3


# ---------------------------------------------------------------- invariances (App. D.2; Eq. 19)
def test_orthogonal_rebasing_of_the_latent_changes_nothing():
    # App. D.2 with a square orthogonal R: c -> R^T c, W_UK -> W_UK R, W_UV -> W_UV R.
    shape, c = _tiny_case(seed=9)
    scale = 0.2
    base = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                   c['seqlens'], scale)
    rng = np.random.default_rng(9)
    R = np.linalg.qr(rng.standard_normal((shape.r, shape.r)))[0]
    cache = np.nan_to_num(c['cache'].copy())
    cache[..., :shape.r] = cache[..., :shape.r] @ R            # rows: (R^T c)^T = c^T R
    for fn in (orc.mla_decode_mha_form, orc.mla_decode_absorbed_form):
        got = fn(c['q_nope'], c['q_pe'], c['w_uk'] @ R, c['w_uv'] @ R, cache, c['page_table'], c['seqlens'], scale)
        assert np.abs(got[0] - base[0]).max() < 1e-9 and np.abs(got[1] - base[1]).max() < 1e-9


def test_key_value_balancing_changes_nothing():
    # Eq. 19: divide the key part of the latent by alpha and multiply W_UK by alpha.
    rng = np.random.default_rng(10)
    ref, m = lifts.selector_lift(rng)
    gd = m['g'] * m['d']
    alpha = 3.7
    cache = m['cache'].copy()
    cache[..., :gd] /= alpha
    out, _ = orc.mla_decode_mha_form(m['q_nope'], m['q_pe'], m['w_uk'] * alpha, m['w_uv'], cache,
                                     m['page_table'], m['seqlens'], m['scale'])
    assert np.abs(out[0, 0] - ref).max() < TOL


# ---------------------------------------------------------------- paging / index path
def test_page_permutation_is_bit_invariant():
    shape, c = _tiny_case(seed=11, seqlens=(130, 64, 5))
    scale = 0.1
    base = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                   c['seqlens'], scale)
    rng = np.random.default_rng(11)
    n = c['cache'].shape[0]
    perm = rng.permutation(n)                       # new index of old page p is perm[p]
    cache2 = np.empty_like(c['cache'])
    cache2[perm] = c['cache']
    table2 = np.where(c['page_table'] >= 0, perm[np.maximum(c['page_table'], 0)], -1)
    got = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], cache2, table2, c['seqlens'], scale)
    assert np.array_equal(got[0], base[0]) and np.array_equal(got[1], base[1])


def test_gather_and_slot_follow_the_page_table():
    P = 4
    cache = np.arange(5 * P * 2, dtype=np.float64).reshape(5, P, 2)
    rows = orc.gather_latent(cache, [3, 0, 4], 10, P)
    want = [cache[3, 0], cache[3, 1], cache[3, 2], cache[3, 3], cache[0, 0], cache[0, 1], cache[0, 2],
            cache[0, 3], cache[4, 0], cache[4, 1]]
    assert np.array_equal(rows, np.array(want))
    assert orc.append_slot([3, 0, 4], 9, P) == (4, 1) and orc.append_slot([3, 0, 4], 4, P) == (0, 0)


# ---------------------------------------------------------------- S > 1, empty sequences (library definitions)
def test_two_query_positions_are_causal_within_the_pair():
    shape, c = _tiny_case(seed=12, seqlens=(70, 65), S=2)
    scale = 0.15
    out, lse = orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                       c['seqlens'], scale)
    for s, drop in ((0, 1), (1, 0)):
        o1, l1 = orc.mla_decode_mha_form(c['q_nope'][:, s:s + 1], c['q_pe'][:, s:s + 1], c['w_uk'], c['w_uv'],
                                         c['cache'], c['page_table'], c['seqlens'] - drop, scale)
        assert np.array_equal(o1[:, 0], out[:, s]) and np.array_equal(l1[:, 0], lse[:, s])
    b = orc.mla_decode_absorbed_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                     c['seqlens'], scale, G=3)
    assert np.abs(b[0] - out).max() < TOL


def test_empty_sequence_gives_zero_and_minus_inf():
    shape, c = _tiny_case(seed=13, seqlens=(0, 5))
    for fn in (orc.mla_decode_mha_form, orc.mla_decode_absorbed_form):
        out, lse = fn(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'], c['seqlens'], 0.1)
        assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0])) and np.all(np.isfinite(lse[1]))


# ---------------------------------------------------------------- split plan (index path)
@pytest.mark.parametrize('seqlens,G', [((17, 64), 1), ((17, 64), 5), ((8192,) * 16, 148), ((0, 5, 0, 700, 64, 65), 7),
                                       ((1,), 4), ((0, 0), 3), ((1000, 3, 3, 3, 9000), 33)])
def test_split_plan_properties_and_closed_form(seqlens, G):
    P, c = 64, orc.SEGMENT_COST_PAGES
    cum, plan = orc.split_plan(seqlens, P, G)
    n = [(L + P - 1) // P for L in seqlens]
    v = [x + c if x > 0 else 0 for x in n]
    assert list(cum) == [sum(v[:b]) for b in range(len(n) + 1)]
    T = sum(v)
    # partitions tile [0, T) in order with sizes differing by at most one
    assert plan[0, 0] == 0 and plan[-1, 1] == T and all(plan[i, 1] == plan[i + 1, 0] for i in range(G - 1))
    sizes = plan[:, 1] - plan[:, 0]
    assert sizes.max() - sizes.min() <= 1
    # sequence fields by bisection on cum (a second route to the same integers)
    for i in range(G):
        p0, p1 = int(plan[i, 0]), int(plan[i, 1])
        if p1 > p0:
            assert plan[i, 2] == np.searchsorted(cum, p0, side='right') - 1
            assert plan[i, 3] == np.searchsorted(cum, p1 - 1, side='right') - 1
        else:
            assert plan[i, 2] == -1 and plan[i, 3] == -1
    # segments cover every page of every sequence exactly once, with distinct slots below G + B - 1
    segs = orc.plan_segments(cum, plan)
    seen = {b: [] for b in range(len(n))}
    for (i, b, lo, hi, slot) in segs:
        seen[b] += list(range(lo, hi))
        assert slot == i + b and 0 <= slot <= G + len(n) - 2
    assert all(seen[b] == list(range(n[b])) for b in seen)
    assert len({s[4] for s in segs}) == len(segs)
    # load per partition = pages + c per sequence opened after the first, never above the even share + c
    load = {}
    for (i, b, lo, hi, slot) in segs:
        load[i] = load.get(i, -c) + (hi - lo) + c
    assert all(x <= -(-T // G) + c for x in load.values())


# ---------------------------------------------------------------- append (Eq. 7 left)
def test_append_writes_projection_and_rotated_key_into_the_right_row_only():
    rng = np.random.default_rng(14)
    D, r, dR, P = 12, 6, 4, 4
    x = rng.standard_normal((2, D))
    w = rng.standard_normal((r + dR, D))
    table = np.array([[2, 0, -1], [1, 3, 4]], dtype=np.int32)
    pos = np.array([5, 8])
    cache = np.full((5, P, r + dR), 7.0)
    got = orc.latent_append(x, w, pos, table, cache.copy(), r, theta=100.0, page_size=P)
    touched = np.zeros((5, P), bool)
    for b, (pg, off) in enumerate([(0, 1), (4, 0)]):
        touched[pg, off] = True
        assert np.allclose(got[pg, off, :r], w[:r] @ x[b], atol=1e-12)
        k = w[r:] @ x[b]
        z = (k[0::2] + 1j * k[1::2]) * np.exp(1j * pos[b] * 100.0 ** (-2 * np.arange(dR // 2) / dR))
        assert np.allclose(got[pg, off, r::2], z.real, atol=1e-12) and np.allclose(got[pg, off, r + 1::2], z.imag, atol=1e-12)
    assert np.all(got[~touched] == 7.0)


def test_append_then_decode_equals_decode_over_the_full_sequence():
    # building the cache token by token with append gives the attention of Eq. 8-9 over x_0..x_t
    rng = np.random.default_rng(15)
    D, H, dn, dR, dv, r, P, T = 10, 2, 3, 4, 3, 5, 4, 11
    x = rng.standard_normal((T, D))
    w = rng.standard_normal((r + dR, D)) / 3
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    table = np.array([[2, 0, 1]], dtype=np.int32)
    cache = np.full((3, P, r + dR), np.nan)
    for t in range(T):
        orc.latent_append(x[t:t + 1], w, [t], table, cache, r, page_size=P)
    qn, qp = rng.standard_normal((1, 1, H, dn)), rng.standard_normal((1, 1, H, dR))
    out, _ = orc.mla_decode_mha_form(qn, qp, w_uk, w_uv, cache, table, [T], 0.3, page_size=P)
    c = x @ w[:r].T
    kr = orc.rope(x @ w[r:].T, np.arange(T))
    for h in range(H):
        z = ((c @ w_uk[h].T) @ qn[0, 0, h] + kr @ qp[0, 0, h]) * 0.3
        p = np.exp(z - z.max()); p /= p.sum()
        assert np.allclose(out[0, 0, h], p @ (c @ w_uv[h].T), atol=1e-10)


# ---------------------------------------------------------------- whole layer (Eq. 6 vs Eq. 10-14; App. A.2.2)
def test_lifted_layer_reproduces_the_gqa_layer_output_token_by_token():
    # A GQA layer decoded token by token through the MLA layer routine (cache built by its own appends) gives
    # y_t = W_O [o_t,1; ...; o_t,h] of Eq. 6.  The lift keeps d^R = d rope dims for ALL key dims of one "rope
    # head" per group is not available in the decoupled form, so the exact lift used here is g = 1 (MQA):
    # W_KR = W_K (the single key head carries RoPE), the latent holds only the value head, W_UK is empty.
    rng = np.random.default_rng(21)
    h, d, D, T, P = 4, 8, 24, 9, 4
    xs = rng.standard_normal((T, D))
    w_q = rng.standard_normal((h * d, D)) / 5
    w_k = rng.standard_normal((d, D)) / 5
    w_v = rng.standard_normal((d, D)) / 5
    w_o = rng.standard_normal((D, h * d)) / 5
    # MLA weights: latent c = W_V x (r = d), rope key = RoPE(W_K x) (dR = d), no no-RoPE key part (dn = 0 is not
    # representable, so one zero no-RoPE dim is carried: dn = 1 with zero W_UQ rows)
    r, dR, dn = d, d, 1
    w_dkv_kr = np.concatenate([w_v, w_k], axis=0)
    w_uk = np.zeros((h, dn, r))
    w_uv = np.tile(np.eye(d)[None], (h, 1, 1))
    w_uq = np.zeros((h * dn, D))
    table = np.array([[2, 0, 1]], dtype=np.int32)
    cache = np.full((3, P, r + dR), np.nan)
    for t in range(T):
        y = orc.mla_layer_decode(xs[t][None, None], w_uq, w_q, w_dkv_kr, w_uk, w_uv, w_o, cache, table, [t + 1],
                                 1.0 / np.sqrt(d), r, page_size=P)
        ref = orc.gqa_attention_last_token(xs[:t + 1], w_q, w_k, w_v, h, 1)
        assert np.abs(y[0, 0] - ref.reshape(-1) @ w_o.T).max() < 1e-10


def test_layer_step_with_two_new_tokens_equals_two_single_token_steps():
    # S = 2: token (b, s) sits at position L_b - S + s, the S latent rows are appended in that order and query
    # s sees everything up to its own token.  One call with x[B, 2, D] must therefore give, token by token,
    # what two successive single-token calls give on a cache that grows by one token per call.
    rng = np.random.default_rng(23)
    H, dn, dR, dv, r, D, P = 3, 4, 6, 5, 7, 12, 4
    lens = [9, 4, 2]                                       # after the step; the last sequence starts empty
    B = len(lens)
    w = dict(w_uq=rng.standard_normal((H * dn, D)) / 3, w_qr=rng.standard_normal((H * dR, D)) / 3,
             w_dkv_kr=rng.standard_normal((r + dR, D)) / 3, w_uk=rng.standard_normal((H, dn, r)) / 3,
             w_uv=rng.standard_normal((H, dv, r)) / 3, w_o=rng.standard_normal((D, H * dv)) / 3)
    table = np.array([[5, 1, 3], [0, 6, -1], [2, -1, -1]], dtype=np.int32)
    base = np.full((7, P, r + dR), np.nan)
    for b, L in enumerate(lens):                           # the L_b - 2 tokens cached before the step
        for j in range(L - 2):
            base[table[b, j // P], j % P] = rng.standard_normal(r + dR)
    x = rng.standard_normal((B, 2, D))
    args = lambda: (w['w_uq'], w['w_qr'], w['w_dkv_kr'], w['w_uk'], w['w_uv'], w['w_o'])
    both = base.copy()
    y2 = orc.mla_layer_decode(x, *args(), both, table, lens, 0.4, r, page_size=P)
    one = base.copy()
    y_first = orc.mla_layer_decode(x[:, :1], *args(), one, table, [L - 1 for L in lens], 0.4, r, page_size=P)
    y_second = orc.mla_layer_decode(x[:, 1:], *args(), one, table, lens, 0.4, r, page_size=P)
    assert np.abs(y2[:, 0] - y_first[:, 0]).max() < 1e-10
    assert np.abs(y2[:, 1] - y_second[:, 0]).max() < 1e-10
    assert np.array_equal(np.isnan(both), np.isnan(one)) and np.abs(np.nan_to_num(both - one)).max() < 1e-12
    # the two tokens really differ in what they see: swapping the pair changes the result
    swapped = orc.mla_layer_decode(x[:, ::-1], *args(), base.copy(), table, lens, 0.4, r, page_size=P)
    assert np.abs(swapped[:, ::-1] - y2).max() > 1e-3


def test_decompressed_keys_and_values_under_ordinary_attention_give_the_mha_form():
    # Eq. 8 + Eq. 9 left: per head the key is [W_UK_h c ; k^R] and the value W_UV_h c; ordinary multi-head
    # attention (grouped_attention with g = h, itself pinned to torch) over them is the definition
    rng = np.random.default_rng(41)
    H, dn, dR, dv, r, P = 4, 8, 4, 6, 10, 4
    L = 11
    cache = rng.standard_normal((5, P, r + dR))
    table = np.array([[3, 0, 4, 1]])
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    q_nope, q_pe = rng.standard_normal((1, 1, H, dn)), rng.standard_normal((1, 1, H, dR))
    k_c, v, k_r = orc.decompress_kv(cache, table[0], L, w_uk, w_uv, P)
    assert k_c.shape == (L, H, dn) and v.shape == (L, H, dv) and k_r.shape == (L, dR)
    # token 6 lives in page table[0][1] = 0, row 2
    assert np.allclose(k_c[6, 2], w_uk[2] @ cache[0, 2, :r], atol=TOL) and np.array_equal(k_r[6], cache[0, 2, r:])
    k = np.concatenate([k_c, np.repeat(k_r[:, None, :], H, axis=1)], axis=2)
    got = orc.grouped_attention(np.concatenate([q_nope[0, 0], q_pe[0, 0]], axis=1), k, v, 0.3)
    want, _ = orc.mla_decode_mha_form(q_nope, q_pe, w_uk, w_uv, cache, table, [L], 0.3, page_size=P)
    assert np.allclose(got, want[0, 0], atol=TOL)


def test_a_chunk_of_query_positions_equals_single_positions_over_the_growing_prefix():
    # chunked prefill: position s of S sees the prefix that a one-token step at length L - S + 1 + s sees
    rng = np.random.default_rng(42)
    H, dn, dR, dv, r, P = 3, 8, 4, 6, 10, 4
    S, L = 7, 13
    cache = rng.standard_normal((6, P, r + dR))
    table = np.array([[5, 2, 0, 3]])
    w_uk, w_uv = rng.standard_normal((H, dn, r)), rng.standard_normal((H, dv, r))
    q_nope, q_pe = rng.standard_normal((1, S, H, dn)), rng.standard_normal((1, S, H, dR))
    out, lse = orc.mla_decode_mha_form(q_nope, q_pe, w_uk, w_uv, cache, table, [L], 0.4, page_size=P)
    for s in range(S):
        o1, l1 = orc.mla_decode_mha_form(q_nope[:, s:s + 1], q_pe[:, s:s + 1], w_uk, w_uv, cache, table,
                                         [L - S + 1 + s], 0.4, page_size=P)
        assert np.allclose(out[0, s], o1[0, 0], atol=TOL) and np.allclose(lse[0, s], l1[0, 0], atol=TOL)


def test_low_rank_queries_and_folded_output_projection():
    # Eq. 8 right: low-rank queries equal full-rank ones with W = W_U{Q,R} W_DQ; App. A.2.2: folding the block
    # diagonal of W_UV into W_O gives the same y from the latent-space outputs.
    rng = np.random.default_rng(22)
    H, dn, dR, dv, r, D, rq, T = 3, 4, 6, 5, 7, 16, 8, 5
    x = rng.standard_normal((T, D))
    w_dq, w_uq, w_qr = rng.standard_normal((rq, D)), rng.standard_normal((H * dn, rq)), rng.standard_normal((H * dR, rq))
    pos = np.array([0, 3, 3, 100, 7])
    a = orc.mla_queries(x, pos, w_uq, w_qr, H, w_dq)
    b = orc.mla_queries(x, pos, w_uq @ w_dq, w_qr @ w_dq, H)
    assert np.abs(a[0] - b[0]).max() < 1e-9 and np.abs(a[1] - b[1]).max() < 1e-9
    # RoPE really sits on the rope part, per head, at the token's position
    raw = (x @ (w_qr @ w_dq).T).reshape(T, H, dR)
    assert np.abs(a[1][3, 1] - orc.rope(raw[3, 1], 100)).max() < 1e-9 and np.abs(a[1][0] - raw[0]).max() < 1e-12
    o_lat = rng.standard_normal((T, H, r))
    w_uv, w_o = rng.standard_normal((H, dv, r)), rng.standard_normal((D, H * dv))
    o = np.einsum('hvr,thr->thv', w_uv, o_lat)
    folded = np.concatenate([w_o[:, i * dv:(i + 1) * dv] @ w_uv[i] for i in range(H)], axis=1)      # W'O [D, H*r]
    assert np.abs(orc.output_projection(o, w_o) - o_lat.reshape(T, -1) @ folded.T).max() < 1e-9


# ---------------------------------------------------------------- numbers the paper prints
def test_kv_cache_ratio_printed_in_the_paper():
    here = os.path.dirname(os.path.abspath(__file__))
    vals = {}
    for line in open(os.path.join(here, 'golden', 'kv_cache_ratio.txt')):
        if line.strip() and not line.startswith('#'):
            k, v = line.split('=')
            vals[k.strip()] = float(v)
    from paper_2502_07864_b200 import synth
    s = synth.LLAMA2_7B
    original = 2 * 32 * 128                                   # 2 g d per token and layer (Sec. 4.1)
    assert round(100.0 * s.row / original, 2) == vals['latent_percent_of_original']
    assert round(100.0 * (1 - s.row / original), 2) == vals['kv_reduction_percent']
