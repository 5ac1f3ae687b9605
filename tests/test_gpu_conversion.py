"""Conversion steps (Sec. 4.2, 4.3; App. B, C, D) through the C ABI against the fp64 conversion oracle.

Every step is compared with the oracle's same step on the same inputs.  Eigenvectors are unique only up to sign
(and up to rotation inside a repeated eigenvalue), so they are checked through what is unique: the eigenvalues,
orthonormality, the residual A V - V diag(w), and the energy a leading block captures."""
import numpy as np
import pytest
import torch

from oracle import conversion_oracle as cv
from oracle import mla_oracle as orc
from paper_2502_07864_b200 import binding, synth
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.tensor(np.ascontiguousarray(a), dtype=torch.float32, device='cuda')


def _f64(t):
    return t.detach().cpu().numpy().astype(np.float64)


def _rel(got, want):
    return np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)


@pytest.mark.parametrize('ta,tb', [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_all_storage_orders_with_ragged_edges(ta, tb):
    gu.ensure_built()
    rng = np.random.default_rng(10 + 2 * ta + tb)
    M, N, K = 261, 130, 77
    a = rng.standard_normal((K, M) if ta else (M, K)).astype(np.float32)
    b = rng.standard_normal((N, K) if tb else (K, N)).astype(np.float32)
    c = torch.full((M, N), float('nan'), device='cuda')
    binding.transmla_conv_gemm(_dev(a), _dev(b), c, ta=bool(ta), tb=bool(tb), alpha=0.5)
    want = 0.5 * (a.astype(np.float64).T if ta else a.astype(np.float64)) @ (b.astype(np.float64).T if tb else b.astype(np.float64))
    assert _rel(_f64(c), want) < 1e-6


@pytest.mark.parametrize('g,d,fold', [(4, 16, 1), (4, 16, 2), (32, 128, 4), (3, 8, 4)])
def test_rorope_covariance_matches_the_oracle(g, d, fold):
    gu.ensure_built()
    rng = np.random.default_rng(20)
    n = 300
    K = rng.standard_normal((n, g * d)).astype(np.float32)
    groups, m = d // 2 // fold, g * fold
    scratch = torch.empty(binding.transmla_conv_rorope_scratch_bytes(n, g, d, fold) // 4, device='cuda')
    cov = torch.full((groups, m, m), float('nan'), device='cuda')
    binding.transmla_conv_rorope_covariance(_dev(K), g, d, fold, scratch, cov)
    want = cv.rorope_covariances(K, g, d, fold)
    assert _rel(_f64(cov), want) < 1e-5


@pytest.mark.parametrize('m,batch', [(7, 3), (32, 64), (128, 4), (1, 2), (2, 1)])
def test_symmetric_eigendecomposition(m, batch):
    gu.ensure_built()
    rng = np.random.default_rng(30 + m)
    x = rng.standard_normal((batch, 3 * m + 2, m)) * (np.arange(1, m + 1) ** -0.7)
    a = np.einsum('bni,bnj->bij', x, x).astype(np.float32)
    w = torch.empty(batch, m, device='cuda'); v = torch.empty(batch, m, m, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    binding.transmla_conv_sym_eig(_dev(a), w, v, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    w, v = _f64(w), _f64(v)
    for b in range(batch):
        want, _ = cv.sorted_eigh(a[b])
        top = want[0]
        assert np.abs(w[b] - want).max() < 2e-5 * top                       # eigenvalues, descending
        assert np.all(np.diff(w[b]) <= 1e-6 * top)
        # orthonormal columns: a column takes part in at most sweeps * (m - 1) fp32 rotations, each off by at most
        # 2^-24 relative; 10 sweeps at m = 128 bound the drift by 8e-5
        assert np.abs(v[b].T @ v[b] - np.eye(m)).max() < 1e-4
        assert np.abs(a[b].astype(np.float64) @ v[b] - v[b] * w[b]).max() < 1e-4 * top
        for keep in (1, max(1, m // 4)):                                     # Ky Fan: the leading block is optimal
            assert abs(cv.captured_energy(a[b], v[b][:, :keep]) - want[:keep].sum()) < 1e-4 * top


@pytest.mark.parametrize('fold', [1, 2])
def test_rorope_apply_matches_the_oracle_and_keeps_the_rope_inner_product(fold):
    gu.ensure_built()
    rng = np.random.default_rng(40)
    g, d, C = 4, 16, 70
    X = rng.standard_normal((g * d, C)).astype(np.float32)
    U = np.stack([np.linalg.qr(rng.standard_normal((g * fold, g * fold)))[0] for _ in range(d // 2 // fold)]).astype(np.float32)
    Y = torch.full((g * d, C), float('nan'), device='cuda')
    binding.transmla_conv_rorope_apply(_dev(X), _dev(U), g, d, fold, Y)
    want = cv.rorope_apply(X, U, g, d, fold)
    assert _rel(_f64(Y), want) < 1e-6
    if fold == 1:   # Eq. 18 on the CUDA result: columns 0 and 1 as a query and a key
        def merged_rope(x, pos):
            return orc.rope(x.reshape(g, d), pos).reshape(-1)
        y = _f64(Y)
        for t, j in [(3, 1), (900, 17)]:
            want_ip = merged_rope(X[:, 0].astype(np.float64), t) @ merged_rope(X[:, 1].astype(np.float64), j)
            got_ip = merged_rope(y[:, 0], t) @ merged_rope(y[:, 1], j)
            assert abs(got_ip - want_ip) < 1e-4 * max(1.0, abs(want_ip))


def test_alpha_and_balanced_concatenation():
    gu.ensure_built()
    rng = np.random.default_rng(50)
    n, mk, mv = 1000, 48, 64
    k = (3.0 * rng.standard_normal((n, mk))).astype(np.float32)
    v = rng.standard_normal((n, mv)).astype(np.float32)
    alpha = torch.zeros(1, device='cuda')
    scratch = torch.empty(2 * n, device='cuda')
    binding.transmla_conv_alpha(_dev(k), _dev(v), scratch, alpha)
    want = cv.bkv_alpha(k, v)
    assert abs(float(alpha.item()) - want) < 1e-5 * want
    Z = torch.full((n, mk + mv), float('nan'), device='cuda')
    binding.transmla_conv_balance_concat(_dev(k), _dev(v), alpha, Z)
    z = _f64(Z)
    assert _rel(z[:, :mk], k.astype(np.float64) / float(alpha.item())) < 1e-6 and np.array_equal(z[:, mk:], v.astype(np.float64))


@pytest.mark.parametrize('m,r', [(96, 24), (300, 64)])
def test_top_subspace_captures_what_the_leading_eigenvectors_capture(m, r):
    gu.ensure_built()
    rng = np.random.default_rng(60 + m)
    basis = np.linalg.qr(rng.standard_normal((m, m)))[0]
    lam = np.concatenate([np.linspace(50.0, 10.0, r), np.linspace(4.0, 0.01, m - r)])   # a clear gap after r
    Cm = ((basis * lam) @ basis.T).astype(np.float32)
    Q = _dev(rng.standard_normal((m, r)))
    scratch = torch.empty(binding.transmla_conv_subspace_scratch_bytes(m, r), dtype=torch.uint8, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    binding.transmla_conv_top_subspace(_dev(Cm), Q, 25, scratch, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    q = _f64(Q)
    assert np.abs(q.T @ q - np.eye(r)).max() < 1e-4
    vals, R = cv.joint_pca(np.linalg.cholesky(Cm.astype(np.float64) + 1e-9 * np.eye(m)).T, r)   # Z with Z^T Z = C
    assert cv.captured_energy(Cm, q) >= (1 - 1e-4) * vals[:r].sum()
    assert np.linalg.norm(q @ q.T - R @ R.T) < 1e-2 * np.sqrt(r)      # the same subspace (projectors agree)


def test_whole_conversion_step_by_step_against_the_oracle():
    # activations -> per-group covariances -> rotations -> rotated W_K -> alpha -> joint second moment -> basis -> rewrite
    gu.ensure_built()
    n, D, g, d, fold, r = 600, 96, 4, 16, 2, 40
    case = synth.make_conversion_case(n, D, g, d, seed=70, device='cuda')
    x, w_k, w_v = case['x'], case['w_k'], case['w_v']
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    k_act = torch.empty(n, g * d, device='cuda')
    binding.transmla_conv_gemm(x, w_k, k_act, tb=True)                       # k_t = W_K x_t
    assert _rel(_f64(k_act), _f64(x) @ _f64(w_k).T) < 1e-5
    groups, m = d // 2 // fold, g * fold
    cov = torch.empty(groups, m, m, device='cuda')
    scratch = torch.empty(binding.transmla_conv_rorope_scratch_bytes(n, g, d, fold) // 4, device='cuda')
    binding.transmla_conv_rorope_covariance(k_act, g, d, fold, scratch, cov)
    assert _rel(_f64(cov), cv.rorope_covariances(_f64(k_act), g, d, fold)) < 1e-5
    vals = torch.empty(groups, m, device='cuda'); U = torch.empty(groups, m, m, device='cuda')
    binding.transmla_conv_sym_eig(cov.clone(), vals, U, status)
    want_vals, _ = cv.rorope_rotations(_f64(cov))
    assert np.abs(_f64(vals) - want_vals).max() < 2e-5 * want_vals.max()
    # Prop. 2 on the CUDA eigenvalues: folding keeps at least what separate rotations keep
    cov1 = torch.empty(d // 2, g, g, device='cuda')
    s1 = torch.empty(binding.transmla_conv_rorope_scratch_bytes(n, g, d, 1) // 4, device='cuda')
    binding.transmla_conv_rorope_covariance(k_act, g, d, 1, s1, cov1)
    v1 = torch.empty(d // 2, g, device='cuda'); u1 = torch.empty(d // 2, g, g, device='cuda')
    binding.transmla_conv_sym_eig(cov1, v1, u1, status)
    for G in range(groups):
        assert float(vals[G, :fold].sum()) >= float(v1[G * fold:(G + 1) * fold, 0].sum()) * (1 - 1e-5)
    # rotate W_K with the CUDA rotations; the oracle does the same step with the same U
    w_k_rot = torch.empty_like(w_k)
    binding.transmla_conv_rorope_apply(w_k, U, g, d, fold, w_k_rot)
    assert _rel(_f64(w_k_rot), cv.rorope_apply(_f64(w_k), _f64(U), g, d, fold)) < 1e-5
    # head 0 keeps RoPE; heads 1.. are the NoPE keys (Sec. 4.3)
    w_k_nope = w_k_rot[d:].contiguous()
    k_nope = torch.empty(n, (g - 1) * d, device='cuda'); v_act = torch.empty(n, g * d, device='cuda')
    binding.transmla_conv_gemm(x, w_k_nope, k_nope, tb=True)
    binding.transmla_conv_gemm(x, w_v, v_act, tb=True)
    alpha = torch.zeros(1, device='cuda'); ns = torch.empty(2 * n, device='cuda')
    binding.transmla_conv_alpha(k_nope, v_act, ns, alpha)
    want_alpha = cv.bkv_alpha(_f64(k_nope), _f64(v_act))
    assert abs(float(alpha.item()) - want_alpha) < 1e-5 * want_alpha
    mz = (2 * g - 1) * d
    Z = torch.empty(n, mz, device='cuda')
    binding.transmla_conv_balance_concat(k_nope, v_act, alpha, Z)
    Cm = torch.empty(mz, mz, device='cuda')
    binding.transmla_conv_gemm(Z, Z, Cm, ta=True)
    assert _rel(_f64(Cm), _f64(Z).T @ _f64(Z)) < 1e-5
    gen = torch.Generator(device='cuda'); gen.manual_seed(71)
    Q = torch.randn(mz, r, generator=gen, device='cuda')
    ws = torch.empty(binding.transmla_conv_subspace_scratch_bytes(mz, r), dtype=torch.uint8, device='cuda')
    binding.transmla_conv_top_subspace(Cm, Q, 60, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    w_top, R = cv.joint_pca(_f64(Z), r)
    assert cv.captured_energy(_f64(Cm), _f64(Q)) >= (1 - 2e-3) * w_top[:r].sum()
    # rewrite (App. D.2 step 3) with the CUDA basis, against the oracle's rewrite with the same basis
    w_dkv = torch.cat([w_k_nope / alpha, w_v], dim=0).contiguous()           # [mz, D]
    w_ukv = torch.randn(50, mz, generator=gen, device='cuda')
    d2 = torch.empty(r, D, device='cuda'); u2 = torch.empty(50, r, device='cuda')
    binding.transmla_conv_gemm(Q, w_dkv, d2, ta=True)
    binding.transmla_conv_gemm(w_ukv, Q, u2)
    want_d, want_u = cv.low_rank_rewrite(_f64(w_dkv), _f64(w_ukv), _f64(Q))
    assert _rel(_f64(d2), want_d) < 1e-5 and _rel(_f64(u2), want_u) < 1e-5
    # what the compressed layer loses is what the oracle's own basis loses, to within the iteration's tolerance
    full = _f64(w_ukv) @ _f64(w_dkv) @ _f64(x).T
    err_cuda = np.linalg.norm(_f64(u2) @ (_f64(d2) @ _f64(x).T) - full)
    od, ou = cv.low_rank_rewrite(_f64(w_dkv), _f64(w_ukv), R)
    err_orc = np.linalg.norm(ou @ (od @ _f64(x).T) - full)
    assert err_cuda <= 1.05 * err_orc + 1e-6 * np.linalg.norm(full)
