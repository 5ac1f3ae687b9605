"""Pins of the conversion oracle (RoRoPE, FreqFold, key/value balancing, joint PCA) on the CPU."""
import numpy as np
import pytest

from oracle import conversion_oracle as cv
from oracle import mla_oracle as orc

TOL = 1e-9


def _random_orthogonal(rng, m):
    q, r = np.linalg.qr(rng.standard_normal((m, m)))
    return q * np.sign(np.diag(r))


def test_segment_index_follows_the_worked_example_of_the_paper():
    # App. C's example: g = 2 heads of d = 8; the group of phi_1 holds dimensions {1,2} of head 1 and {9,10} of
    # head 2 (1-based), 2D-FreqFold merges phi_1 with phi_2: {1,2,3,4} and {9,10,11,12}
    re, im = cv.segment_index(2, 8, 1)
    assert sorted(np.concatenate([re[0], im[0]]) + 1) == [1, 2, 9, 10]
    assert sorted(np.concatenate([re[1], im[1]]) + 1) == [3, 4, 11, 12]
    re, im = cv.segment_index(2, 8, 2)
    assert re.shape == (2, 4)
    assert sorted(np.concatenate([re[0], im[0]]) + 1) == [1, 2, 3, 4, 9, 10, 11, 12]
    assert sorted(np.concatenate([re[1], im[1]]) + 1) == [5, 6, 7, 8, 13, 14, 15, 16]


@pytest.mark.parametrize('fold', [1, 2])
def test_covariances_by_scalar_loops(fold):
    rng = np.random.default_rng(0)
    n, g, d = 7, 3, 8
    K = rng.standard_normal((n, g * d))
    got = cv.rorope_covariances(K, g, d, fold)
    for G in range(d // 2 // fold):
        for a in range(g * fold):
            for b in range(g * fold):
                (pa, ja), (pb, jb) = divmod(a, g), divmod(b, g)
                ca, cb = 2 * (G * fold + pa), 2 * (G * fold + pb)
                want = sum(K[t, ja * d + ca] * K[t, jb * d + cb] + K[t, ja * d + ca + 1] * K[t, jb * d + cb + 1] for t in range(n))
                assert abs(got[G, a, b] - want) < TOL


def test_rotation_leaves_the_rope_inner_product_unchanged():
    # Eq. 18: with the same orthogonal U_l on the real and on the imaginary parts of frequency l across heads,
    # rope(q', t) . rope(k', j) == rope(q, t) . rope(k, j), where rope rotates every head's d dimensions alike
    rng = np.random.default_rng(1)
    g, d = 4, 8
    q, k = rng.standard_normal(g * d), rng.standard_normal(g * d)
    U = np.stack([_random_orthogonal(rng, g) for _ in range(d // 2)])
    qr, kr = cv.rorope_apply(q[:, None], U, g, d)[:, 0], cv.rorope_apply(k[:, None], U, g, d)[:, 0]

    def merged_rope(x, pos):
        return orc.rope(x.reshape(g, d), pos).reshape(-1)

    for t, j in [(0, 0), (5, 2), (1000, 3), (17, 4000)]:
        want = merged_rope(q, t) @ merged_rope(k, j)
        got = merged_rope(qr, t) @ merged_rope(kr, j)
        assert abs(got - want) < 1e-9 * max(1.0, abs(want))
    # a different matrix on the imaginary parts breaks it (the constraint App. B derives)
    V = U.copy()
    V[0] = _random_orthogonal(rng, g)
    kb = cv.rorope_apply(k[:, None], U, g, d)[:, 0]
    idx_re, idx_im = cv.segment_index(g, d, 1)
    for qq in range(g):
        kb[qq * d + 1] = V[0][:, qq] @ k[idx_im[0]]
    assert abs(merged_rope(qr, 5) @ merged_rope(kb, 2) - merged_rope(q, 5) @ merged_rope(k, 2)) > 1e-3


@pytest.mark.parametrize('fold', [1, 2])
def test_rotation_is_orthogonal_and_puts_the_most_energy_into_the_first_heads(fold):
    rng = np.random.default_rng(2)
    n, g, d = 200, 4, 8
    K = rng.standard_normal((n, g * d)) @ rng.standard_normal((g * d, g * d))
    cov = cv.rorope_covariances(K, g, d, fold)
    vals, U = cv.rorope_rotations(cov)
    m = g * fold
    for G in range(cov.shape[0]):
        assert np.allclose(U[G].T @ U[G], np.eye(m), atol=1e-10)
        assert np.all(np.diff(vals[G]) <= 1e-9) and np.allclose(U[G].T @ cov[G] @ U[G], np.diag(vals[G]), atol=1e-8 * vals[G][0])
        for keep in (1, 2):   # Ky Fan: no orthogonal matrix keeps more in its first columns
            best = np.trace((U[G].T @ cov[G] @ U[G])[:keep, :keep])
            assert abs(best - vals[G][:keep].sum()) < 1e-8 * vals[G][0]
            for _ in range(20):
                W = _random_orthogonal(rng, m)
                assert np.trace((W.T @ cov[G] @ W)[:keep, :keep]) <= best + 1e-9
    # the rotated activations carry that energy in head 0: (K rotated)^T second moments
    Kr = cv.rorope_apply(K.T, U, g, d, fold).T
    cov_r = cv.rorope_covariances(Kr, g, d, fold)
    for G in range(cov.shape[0]):
        # component q sits at segment index (q % fold) * g + q // fold after the rotation
        pos = [(q % fold) * g + q // fold for q in range(m)]
        assert np.allclose(np.diag(cov_r[G])[pos], vals[G], atol=1e-8 * vals[G][0])
    assert abs((Kr ** 2).sum() - (K ** 2).sum()) < 1e-8 * (K ** 2).sum()


def test_freqfold_keeps_at_least_what_separate_rotations_keep():
    # Prop. 2 (App. C): the M largest eigenvalues of the merged group's covariance sum to at least the sum of the
    # largest eigenvalue of each of its M members
    rng = np.random.default_rng(3)
    n, g, d, M = 300, 4, 16, 4
    K = rng.standard_normal((n, g * d)) @ rng.standard_normal((g * d, g * d))
    v1, _ = cv.rorope_rotations(cv.rorope_covariances(K, g, d, 1))
    vM, _ = cv.rorope_rotations(cv.rorope_covariances(K, g, d, M))
    for G in range(d // 2 // M):
        V1 = v1[G * M:(G + 1) * M, 0].sum()
        V2 = vM[G, :M].sum()
        assert V2 >= V1 - 1e-9
    # the merged covariance has the members' covariances as its diagonal blocks
    c1, cM = cv.rorope_covariances(K, g, d, 1), cv.rorope_covariances(K, g, d, M)
    for p in range(M):
        assert np.allclose(cM[1][p * g:(p + 1) * g, p * g:(p + 1) * g], c1[M + p], atol=1e-9)


def test_alpha_closed_forms():
    rng = np.random.default_rng(4)
    v = rng.standard_normal((50, 6))
    assert abs(cv.bkv_alpha(3.0 * v, v) - 3.0) < 1e-12
    k = np.zeros((2, 4)); k[0, 0] = 3.0; k[0, 1] = 4.0; k[1, 2] = 1.0     # norms 5 and 1 -> mean 3
    vv = np.zeros((2, 2)); vv[0, 0] = 2.0; vv[1, 1] = 4.0                  # norms 2 and 4 -> mean 3
    assert abs(cv.bkv_alpha(k, vv) - 1.0) < 1e-12


def test_joint_pca_reconstructs_low_rank_data_and_everything_at_full_rank():
    rng = np.random.default_rng(5)
    n, m, D, r = 80, 12, 20, 5
    w_dkv = rng.standard_normal((m, r)) @ rng.standard_normal((r, D))          # rank r: activations live in r dims
    x = rng.standard_normal((n, D))
    Z = x @ w_dkv.T
    vals, R = cv.joint_pca(Z, r)
    assert np.allclose(R.T @ R, np.eye(r), atol=1e-10) and np.all(vals[r:] < 1e-8 * vals[0])
    assert np.allclose(Z @ R @ R.T, Z, atol=1e-8)
    w_ukv = rng.standard_normal((9, m))
    d2, u2 = cv.low_rank_rewrite(w_dkv, w_ukv, R)
    assert d2.shape == (r, D) and u2.shape == (9, r)
    assert np.allclose(u2 @ d2, w_ukv @ R @ R.T @ w_dkv, atol=1e-9)
    assert np.allclose(u2 @ (d2 @ x.T), w_ukv @ (w_dkv @ x.T), atol=1e-7)        # nothing lost on rank-r data
    full = rng.standard_normal((m, D))
    _, Rf = cv.joint_pca(x @ full.T, m)
    d3, u3 = cv.low_rank_rewrite(full, w_ukv, Rf)
    assert np.allclose(u3 @ d3, w_ukv @ full, atol=1e-9)
    # captured energy grows with r and equals the eigenvalue sum
    C = Z.T @ Z
    assert abs(cv.captured_energy(C, R) - vals[:r].sum()) < 1e-8 * vals[0]
    assert cv.captured_energy(C, R[:, :3]) <= cv.captured_energy(C, R) + 1e-9
