"""fp64 CPU oracle of the GQA -> MLA conversion steps on calibration activations (numpy).

TEST INFRASTRUCTURE ONLY, like mla_oracle.py: nothing in the product package imports this module and
it shares no code with the CUDA path.  Library primitives used as steps: ``@`` and
``numpy.linalg.eigh``.  Each function names the passage of the TransMLA paper it follows.

Index conventions (0-based).  The merged key of Sec. 4.1 is a vector of g*d entries, entry (j, c) =
j*d + c for original head j and dimension c.  RoPE pair l of a head is (c = 2l, 2l+1): real and
imaginary part (Sec. 3.1).  FreqFold with M consecutive frequencies per group (App. C): group G holds
l = G*M .. G*M+M-1; within a group the segment index of (frequency p = l - G*M, head j) is p*g + j.
After the rotation, component q of group G is stored at head q // M, frequency G*M + q % M, so that the
M strongest components of every group land in head 0 - the head that keeps RoPE.

Readings where the paper leaves room (all listed in the design doc): the covariance is the plain second
moment K^T K (App. B writes sigma = K^T K with no centring); with FreqFold the real parts of all M
frequencies of a group rotate together, and the imaginary parts by the same matrix (App. B's
constraint carried over to App. C's concatenated segments); alpha is a ratio of mean L2 norms
(Eq. 19); the PCA of App. D.2 is on the second moment of [k_nope / alpha ; v], not centred.

Pins (tests/test_oracle_conversion.py): brute-force loops for the covariances, Eq. 18 (the RoPE'd inner
product is unchanged by the rotation, with the RoPE of mla_oracle.py), Ky Fan optimality of the
rotation against random orthogonal matrices, Prop. 2 (V2 >= V1), closed forms of alpha, exact
reconstruction of rank-r data by the joint PCA and of any data at full rank, and equality of the
rewritten low-rank product with the projector form.
"""
import numpy as np


def segment_index(g, d, fold):
    """idx_re, idx_im [groups, g*fold]: positions in the merged key of every group's real / imaginary parts."""
    groups = d // 2 // fold
    idx_re = np.empty((groups, g * fold), dtype=np.int64)
    idx_im = np.empty((groups, g * fold), dtype=np.int64)
    for G in range(groups):
        for p in range(fold):
            for j in range(g):
                l = G * fold + p
                idx_re[G, p * g + j] = j * d + 2 * l
                idx_im[G, p * g + j] = j * d + 2 * l + 1
    return idx_re, idx_im


def rorope_covariances(K, g, d, fold=1):
    """App. B: sigma_x + sigma_y = K_x^T K_x + K_y^T K_y per frequency group.  K [n, g*d] -> [groups, g*fold, g*fold]."""
    K = np.asarray(K, np.float64)
    idx_re, idx_im = segment_index(g, d, fold)
    out = np.empty((idx_re.shape[0], g * fold, g * fold))
    for G in range(idx_re.shape[0]):
        kx, ky = K[:, idx_re[G]], K[:, idx_im[G]]
        out[G] = kx.T @ kx + ky.T @ ky
    return out


def sorted_eigh(a):
    """Eigenvalues in descending order and the matching eigenvectors as columns."""
    w, v = np.linalg.eigh(np.asarray(a, np.float64))
    order = np.argsort(-w, kind='stable')
    return w[order], v[:, order]


def rorope_rotations(cov):
    """App. B: U_l = eigenvectors of the summed covariance, columns by descending eigenvalue.  -> (eigvals, U)."""
    vals = np.empty(cov.shape[:2])
    U = np.empty_like(np.asarray(cov, np.float64))
    for G in range(cov.shape[0]):
        vals[G], U[G] = sorted_eigh(cov[G])
    return vals, U


def rorope_apply(X, U, g, d, fold=1):
    """Eq. 18 / Sec. 4.2: rotate the rows of X [g*d, C] (a W^K, or a merged query/key written as a column).

    Component q of group G, real part:  Y[(q // M, 2(G*M + q % M))] = sum_i U_G[i, q] X[idx_re[G, i]],
    and the imaginary part with the same U_G.
    """
    X = np.asarray(X, np.float64)
    idx_re, idx_im = segment_index(g, d, fold)
    Y = np.empty_like(X)
    for G in range(idx_re.shape[0]):
        for q in range(g * fold):
            row = (q // fold) * d + 2 * (G * fold + q % fold)
            Y[row] = U[G][:, q] @ X[idx_re[G]]
            Y[row + 1] = U[G][:, q] @ X[idx_im[G]]
    return Y


def bkv_alpha(k_nope, v):
    """Eq. 19: alpha = E_t ||k_nope,t||_2 / E_t ||v_t||_2 over the calibration tokens (rows)."""
    k_nope, v = np.asarray(k_nope, np.float64), np.asarray(v, np.float64)
    return np.sqrt((k_nope ** 2).sum(axis=1)).mean() / np.sqrt((v ** 2).sum(axis=1)).mean()


def joint_pca(Z, r):
    """App. D.2 step 2: the r leading eigenvectors of Z^T Z (Z [n, m] = rows [k_nope / alpha ; v]) -> (eigvals, R [m, r])."""
    Z = np.asarray(Z, np.float64)
    w, v = sorted_eigh(Z.T @ Z)
    return w, v[:, :r]


def low_rank_rewrite(w_dkv, w_ukv, R):
    """App. D.2 step 3: W_DKV' = R^T W_DKV [r, D] and W_UKV' = W_UKV R [p, r]."""
    R = np.asarray(R, np.float64)
    return R.T @ np.asarray(w_dkv, np.float64), np.asarray(w_ukv, np.float64) @ R


def captured_energy(C, Q):
    """trace(Q^T C Q) for an orthonormal Q: the second moment kept by projecting onto span(Q)."""
    Q = np.asarray(Q, np.float64)
    return float(np.trace(Q.T @ np.asarray(C, np.float64) @ Q))
