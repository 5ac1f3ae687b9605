"""Test fixtures: a GQA layer rewritten as an MLA layer (paper Sec. 4.1, App. A.2.1), and small helpers.

Both lifts return (gqa_reference [h, dv], mla_inputs dict in float64).  The reference is computed
by the GQA routines alone; the MLA inputs are what the decode path (oracle or CUDA) consumes.
"""
import numpy as np

from oracle import mla_oracle as orc


def rope_hat(x, pos, d, theta=10000.0):
    """The merged RoPE of Sec. 4.1: the same RoPE applied to every consecutive d-block."""
    x = np.asarray(x, np.float64)
    blocks = x.reshape(x.shape[:-1] + (x.shape[-1] // d, d))
    return orc.rope(blocks, np.asarray(pos)[..., None], theta).reshape(x.shape)


def selector_lift(rng, h=8, g=2, d=32, D=48, T=37, theta=10000.0, P=64):
    """Paper-exact lift: W_DKV = [W_K; W_V], r = 2gd, dR = 0, selector W_UK_i / W_UV_i (Eq. 10-14).

    The cached latent is [RoPE-hat(c^K_j, j) ; c^V_j]; the absorbed query is
    RoPE-hat(W_UK_i^T q_i, t), which equals W_UK_i^T RoPE(q_i, t) because the selector moves whole
    d-blocks; so q_nope := RoPE(q_i, t) with the unrotated selector as W_UK.
    """
    x = rng.standard_normal((T, D))
    w_q = rng.standard_normal((h * d, D)) / np.sqrt(D)
    w_k = rng.standard_normal((g * d, D)) / np.sqrt(D)
    w_v = rng.standard_normal((g * d, D)) / np.sqrt(D)
    ref = orc.gqa_attention_last_token(x, w_q, w_k, w_v, h, g, theta)

    r = 2 * g * d
    w_dkv = np.concatenate([w_k, w_v], axis=0)                  # [2gd, D]
    c = x @ w_dkv.T                                             # [T, 2gd]
    c[:, :g * d] = rope_hat(c[:, :g * d], np.arange(T), d, theta)
    w_uk = np.zeros((h, d, r))
    w_uv = np.zeros((h, d, r))
    for i in range(h):
        j = i // (h // g)
        w_uk[i, :, j * d:(j + 1) * d] = np.eye(d)
        w_uv[i, :, (g + j) * d:(g + j + 1) * d] = np.eye(d)
    q = (x[T - 1] @ w_q.T).reshape(h, d)
    q_nope = orc.rope(q, T - 1, theta)
    mla = paged(c, P, rng)
    mla.update(q_nope=q_nope[None, None], q_pe=np.zeros((1, 1, h, 0)), w_uk=w_uk, w_uv=w_uv,
               scale=1.0 / np.sqrt(d), q_raw=q, t=T - 1, d=d, g=g)
    return ref, mla


def replicated_lift(rng, h=8, g=2, dn=32, dR=16, dv=32, r=64, T=50, theta=10000.0, P=64):
    """A grouped layer acting on an r-dim latent with one shared RoPE key, lifted by replication.

    Group j has K/V up-projections A_j [dn, r], B_j [dv, r]; every query head i of the group gets
    W_UK_i = A_j, W_UV_i = B_j (App. A.2.1: W'^K_i = W^K_{ceil(i/(h/g))}).  The reference runs
    grouped attention with keys [A_j c ; k^R] and values B_j c.
    """
    c = rng.standard_normal((T, r))
    k_pe = orc.rope(rng.standard_normal((T, dR)), np.arange(T), theta)
    a = rng.standard_normal((g, dn, r)) / np.sqrt(r)
    b = rng.standard_normal((g, dv, r)) / np.sqrt(r)
    q_nope = rng.standard_normal((h, dn))
    q_pe = orc.rope(rng.standard_normal((h, dR)), T - 1, theta)
    scale = 1.0 / np.sqrt(dn + dR)
    k = np.concatenate([np.einsum('gnr,tr->tgn', a, c), np.repeat(k_pe[:, None, :], g, axis=1)], axis=-1)
    v = np.einsum('gvr,tr->tgv', b, c)
    ref = orc.grouped_attention(np.concatenate([q_nope, q_pe], axis=-1), k, v, scale)
    grp = np.arange(h) // (h // g)
    mla = paged(np.concatenate([c, k_pe], axis=-1), P, rng)
    mla.update(q_nope=q_nope[None, None], q_pe=q_pe[None, None], w_uk=a[grp], w_uv=b[grp], scale=scale)
    return ref, mla


def paged(rows, P, rng, extra=3):
    """Scatter one sequence's rows [T, w] into a shuffled page pool; tails and spare pages are NaN."""
    T, w = rows.shape
    n = (T + P - 1) // P
    perm = rng.permutation(n + extra)
    cache = np.full((n + extra, P, w), np.nan)
    for j in range(T):
        cache[perm[j // P], j % P] = rows[j]
    table = np.full((1, n), -1, dtype=np.int32)
    table[0, :n] = perm[:n]
    return dict(cache=cache, page_table=table, seqlens=np.array([T], dtype=np.int32))


def f64(t):
    """torch tensor (any float dtype) -> float64 numpy; integer tensors -> numpy as they are."""
    import torch
    if t.dtype in (torch.bfloat16, torch.float16, torch.float32, torch.float64):
        return t.detach().cpu().to(torch.float64).numpy()
    return t.detach().cpu().numpy()


def case_f64(case):
    return {k: f64(v) for k, v in case.items()}


def rel_l2(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))
