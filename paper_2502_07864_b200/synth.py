"""Seeded synthetic inputs for absorbed-MLA decode and latent append.

This module only draws random numbers and lays out index tables.  It contains none of the
method's arithmetic (no RoPE, no projections, no attention), so that it can serve both the
CUDA path and an independent checker without coupling them.

Value recipe: activations and cache rows are N(0,1); weights are N(0, 1/sqrt(fan_in)) with
fan_in the contracted dimension (r for W_UK and W_UV, D for the append weight); everything is
rounded to bf16 once, and those bf16 bits are the inputs.  A rotation applied to i.i.d. N(0,1)
pairs leaves them i.i.d. N(0,1), so the RoPE'd parts of the cache and of the queries are drawn
directly from N(0,1).  Pages of each sequence are scattered over the pool by a seeded
permutation; unused page-table entries hold -1.
"""
from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class MLAShape:
    """Dimensions of one converted attention layer (paper Sec. 3.3 symbols)."""
    H: int          # query heads h
    dn: int         # per-head no-RoPE key dim d
    dR: int         # decoupled RoPE dim d^R (may be 0)
    dv: int         # per-head value dim
    r: int          # latent rank r_kv
    D: int = 4096   # hidden size
    S: int = 1      # new query tokens per sequence
    page_size: int = 64

    @property
    def row(self):
        return self.r + self.dR


TINY = MLAShape(H=8, dn=32, dR=16, dv=32, r=64, D=256)
LLAMA2_7B = MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096)
QWEN25_72B = MLAShape(H=64, dn=128, dR=64, dv=128, r=512, D=8192, S=2)


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn_bf16(shape, std, g, device):
    """N(0, std) in bf16, drawn in chunks so that no large fp32 temporary is held."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for i in range(0, flat.numel(), step):
        n = min(step, flat.numel() - i)
        flat[i:i + n] = (torch.randn(n, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def uniform_seqlens(B, lo, hi, seed):
    """B lengths uniform in [lo, hi], seeded (CPU generator, so the same on every machine)."""
    g = _gen(seed, 'cpu')
    return torch.randint(lo, hi + 1, (B,), generator=g, dtype=torch.int64).tolist()


def make_decode_case(shape, seqlens, seed, pool_factor=1.2, device='cpu', nan_tails=False,
                     extra_pages=0):
    """Inputs of one decode step.  Returns a dict of tensors on ``device``.

    q_nope [B,S,H,dn], q_pe [B,S,H,dR], w_uk [H,dn,r], w_uv [H,dv,r], cache
    [num_pages, P, r+dR] (bf16); page_table [B, max_pages], seqlens [B] (int32).
    With ``nan_tails`` every cache row that no sequence owns (page tails and unowned pages) is
    NaN, to show that such rows never reach a result.
    """
    P = shape.page_size
    B = len(seqlens)
    g = _gen(seed, device)
    gc = _gen(seed, 'cpu')
    n_pages = [(int(L) + P - 1) // P for L in seqlens]
    total = sum(n_pages)
    num_pages = max(int(total * pool_factor + 0.999), total, 1) + extra_pages
    max_pages = max(max(n_pages), 1)
    perm = torch.randperm(num_pages, generator=gc)
    page_table = torch.full((B, max_pages), -1, dtype=torch.int32)
    k = 0
    for b in range(B):
        page_table[b, :n_pages[b]] = perm[k:k + n_pages[b]].to(torch.int32)
        k += n_pages[b]
    case = {
        'q_nope': _randn_bf16((B, shape.S, shape.H, shape.dn), 1.0, g, device),
        'q_pe': _randn_bf16((B, shape.S, shape.H, shape.dR), 1.0, g, device),
        'w_uk': _randn_bf16((shape.H, shape.dn, shape.r), shape.r ** -0.5, g, device),
        'w_uv': _randn_bf16((shape.H, shape.dv, shape.r), shape.r ** -0.5, g, device),
        'cache': _randn_bf16((num_pages, P, shape.row), 1.0, g, device),
        'page_table': page_table.to(device),
        'seqlens': torch.tensor([int(L) for L in seqlens], dtype=torch.int32, device=device),
    }
    if nan_tails:
        owned = torch.zeros(num_pages, P, dtype=torch.bool)
        for b in range(B):
            for j in range(n_pages[b]):
                owned[page_table[b, j], :min(P, int(seqlens[b]) - j * P)] = True
        case['cache'][~owned.to(device)] = float('nan')
    return case


FP8_ROW_BYTES = 656   # 512 e4m3 codes, 64 bf16, one fp32 scale, 12 bytes unused


def make_fp8_cache(shape, num_pages, seed, device='cpu'):
    """A latent cache in the library's FP8 row format, [num_pages, P, 656] uint8, filled with seeded N(0,1) rows that
    are rounded once to the storage format (as the bf16 cache is rounded once to bf16): per row scale = max|c| / 448,
    codes = e4m3(c / scale) by torch's float8 cast, k_pe / scale in bf16.  r = 512, dR = 64."""
    assert shape.r == 512 and shape.dR == 64
    g = _gen(seed, device)
    P = shape.page_size
    out = torch.zeros((num_pages, P, FP8_ROW_BYTES), dtype=torch.uint8, device=device)
    step = 2048
    for i in range(0, num_pages, step):
        n = min(step, num_pages - i)
        rows = torch.randn((n, P, shape.row), generator=g, device=device, dtype=torch.float32)
        scale = rows[..., :shape.r].abs().amax(dim=-1, keepdim=True) / 448.0
        out[i:i + n, :, :shape.r] = (rows[..., :shape.r] / scale).to(torch.float8_e4m3fn).view(torch.uint8)
        out[i:i + n, :, shape.r:shape.r + 2 * shape.dR] = (rows[..., shape.r:] / scale).to(torch.bfloat16).view(torch.uint8).view(n, P, -1)
        out[i:i + n, :, 640:644] = scale.contiguous().view(torch.uint8).view(n, P, 4)
    return out


def make_append_case(shape, positions, seed, device='cpu'):
    """Inputs of one append step: x [B, S, D] ~ N(0,1), w_dkv_kr [r+dR, D] ~ N(0, 1/sqrt(D)), bf16;
    positions [B] = position of each sequence's first new token."""
    g = _gen(seed, device)
    B = len(positions)
    return {
        'x': _randn_bf16((B, shape.S, shape.D), 1.0, g, device),
        'w_dkv_kr': _randn_bf16((shape.row, shape.D), shape.D ** -0.5, g, device),
        'positions': torch.tensor([int(p) for p in positions], dtype=torch.int32, device=device),
    }


def make_layer_weights(shape, seed, q_lora_rank=0, device='cpu'):
    """Weights of the linear maps either side of the attention: w_uq [H*dn, Dq], w_qr [H*dR, Dq], w_o [D, H*dv] and,
    for low-rank queries, w_dq [r_q, D]; N(0, 1/sqrt(fan_in)), bf16."""
    g = _gen(seed, device)
    Dq = q_lora_rank if q_lora_rank else shape.D
    w = {
        'w_uq': _randn_bf16((shape.H * shape.dn, Dq), Dq ** -0.5, g, device),
        'w_qr': _randn_bf16((shape.H * shape.dR, Dq), Dq ** -0.5, g, device),
        'w_o': _randn_bf16((shape.D, shape.H * shape.dv), (shape.H * shape.dv) ** -0.5, g, device),
    }
    if q_lora_rank:
        w['w_dq'] = _randn_bf16((q_lora_rank, shape.D), shape.D ** -0.5, g, device)
    return w


def make_conversion_case(n, D, g, d, seed, device='cpu', key_gain=3.0):
    """Calibration inputs of the conversion (Sec. 4.2, 4.3), fp32: hidden states x [n, D] whose coordinates decay like
    i**-0.5 (a few strong directions, as the hidden states of a trained model have), key and value projections
    w_k, w_v [g*d, D] ~ N(0, 1/sqrt(D)) with the keys `key_gain` times larger (the imbalance Eq. 19 is there for), and
    a start basis for the subspace iteration is left to the caller.  No arithmetic of the method happens here."""
    gen = _gen(seed, device)
    scale = torch.arange(1, D + 1, dtype=torch.float32, device=device) ** -0.5
    x = torch.randn(n, D, generator=gen, device=device) * scale * (D ** 0.5 / scale.norm())
    w_k = torch.randn(g * d, D, generator=gen, device=device) * (key_gain * D ** -0.5)
    w_v = torch.randn(g * d, D, generator=gen, device=device) * D ** -0.5
    return {'x': x, 'w_k': w_k, 'w_v': w_v}
