"""fp64 CPU oracle for absorbed-MLA decode over a paged latent cache.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this module; it is used
by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no code,
table or helper with the CUDA path and never calls it.

Everything here is numpy float64 and written for reading, not speed.  The only library
primitives used as steps are ``@`` (matmul), ``exp``, ``log``, ``cos`` and ``sin``.  Each
function names the passage of the TransMLA paper (arXiv 2502.07864) it follows.

Notation (paper, Sec. 3): D hidden size, h query heads, g GQA groups, d head dim, r = r_kv latent
rank, dR decoupled-RoPE dim, dn / dv per-head no-RoPE key dim and value dim.  B sequences, S new
query tokens per sequence, L_b cached length of sequence b (the S new tokens included), P tokens
per cache page.

Pins (tests/test_oracle_*.py): closed forms (one token, zero scale, identical rows, a two-token
softmax with exact weights), RoPE as complex multiplication and its relative-position identity
(App. B), Absorb == MHA form (Eq. 9), GQA lifted to MLA == an independent GQA routine that is
itself pinned to torch's scaled_dot_product_attention (Sec. 4.1, App. A.2.1), orthogonal
re-basing of the latent (App. D.2), key/value balancing (Eq. 19), page-permutation invariance,
partition invariance of split + combine, brute-force restatement of the split plan.

Prefill (decompress_kv): ordinary multi-head attention (the routine pinned to torch) over its output
equals mla_decode_mha_form, and a chunk of S query positions equals S single-position calls over the
growing prefix.

FP8 latent cache (end of the file): the e4m3 format is pinned to the values of its published
definition and to torch's float8_e4m3fn conversions, the quantiser to its error bound and to exact
round trips of representable rows, the attention over an FP8 cache to Eq. 9 over the dequantised rows
(tests/test_oracle_fp8.py).

Parity unpinned (no statement in the paper to pin against; fixed by this library's own
definition): the causal reading for S > 1 (query s sees tokens [0, L_b - S + s]), the result for
L_b = 0 (zeros and lse = -inf), that page tails are ignored, and the stored format of the FP8 cache
(per-token scale, e4m3 codes of c / scale, k^R / scale in bf16): the paper only names FP8.
"""
import numpy as np


# --------------------------------------------------------------------------------------------
# RoPE, Sec. 3.1, Eq. 1
# --------------------------------------------------------------------------------------------
def rope(x, pos, theta=10000.0):
    """Rotate the last axis of ``x`` (even length d) to position ``pos`` (Eq. 1).

    Elements (2l, 2l+1) (0-based) are the real and imaginary part of pair l, whose angle is
    pos * theta**(-2l/d).  ``pos`` is a scalar or an array broadcastable to ``x[..., 0]``.
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    if d == 0:
        return x.copy()
    assert d % 2 == 0
    l = np.arange(d // 2, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta ** (-2.0 * l / d)
    c, s = np.cos(ang), np.sin(ang)
    re, im = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x)
    out[..., 0::2] = re * c - im * s
    out[..., 1::2] = im * c + re * s
    return out


# --------------------------------------------------------------------------------------------
# GQA attention, Sec. 3.2, Eq. 2-6 (used only to pin the GQA -> MLA lift)
# --------------------------------------------------------------------------------------------
def grouped_attention(q, k, v, scale):
    """Eq. 5 for one query token: head i attends to key/value group i // (h/g).

    q [h, dq]; k [T, g, dq]; v [T, g, dv] (RoPE already applied where it belongs).  Returns [h, dv].
    """
    q, k, v = (np.asarray(a, dtype=np.float64) for a in (q, k, v))
    h, g = q.shape[0], k.shape[1]
    out = np.zeros((h, v.shape[2]))
    for i in range(h):
        grp = i // (h // g)
        z = (k[:, grp, :] @ q[i]) * scale
        p = np.exp(z - z.max())
        p /= p.sum()
        out[i] = p @ v[:, grp, :]
    return out


def gqa_attention_last_token(x, w_q, w_k, w_v, h, g, theta=10000.0):
    """Output o_{t,i} of Eq. 5 for the last token t of one sequence, before W_O (Eq. 2-5).

    x [T, D]; w_q [h*d, D]; w_k, w_v [g*d, D].  Positions are 0..T-1.  Returns [h, d].
    """
    x = np.asarray(x, dtype=np.float64)
    T = x.shape[0]
    d = w_q.shape[0] // h
    q = (x[T - 1] @ w_q.T).reshape(h, d)
    k = (x @ w_k.T).reshape(T, g, d)
    v = (x @ w_v.T).reshape(T, g, d)
    q_r = rope(q, T - 1, theta)
    k_r = rope(k, np.arange(T)[:, None], theta)
    return grouped_attention(q_r, k_r, v, 1.0 / np.sqrt(d))


# --------------------------------------------------------------------------------------------
# Paged latent cache
# --------------------------------------------------------------------------------------------
def gather_latent(cache, page_row, n, page_size):
    """Rows of tokens 0..n-1 of one sequence: token j lives at cache[page_row[j // P], j % P]."""
    rows = np.empty((n, cache.shape[-1]))
    for j in range(n):
        rows[j] = cache[page_row[j // page_size], j % page_size]
    return rows


def visible_tokens(L_b, S, s):
    """Tokens query position s of S may see when the cache already holds all S new tokens."""
    return max(int(L_b) - (S - 1 - s), 0)


# --------------------------------------------------------------------------------------------
# MLA decode, MHA form = the definition of the result (Sec. 3.3, Eq. 8 and Eq. 9 left)
# --------------------------------------------------------------------------------------------
def mla_decode_mha_form(q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, scale, page_size=64,
                        only=None):
    """Per head: decompress k^C_j = W_UK_h c_j and v_j = W_UV_h c_j, then ordinary attention.

    q_nope [B,S,H,dn]; q_pe [B,S,H,dR] (already rotated); w_uk [H,dn,r]; w_uv [H,dv,r];
    cache [num_pages, P, r+dR] with c_j = row[:r] and k^R_j = row[r:]; page_table [B, max_pages];
    seqlens [B].  Returns out [B,S,H,dv] and lse [B,S,H] (natural log of the softmax
    denominator, max included).  ``only`` is an optional list of (b, s, h) to compute; other
    entries stay zero.  W_O is not applied.
    """
    q_nope = np.asarray(q_nope, np.float64)
    q_pe = np.asarray(q_pe, np.float64)
    B, S, H, _ = q_nope.shape
    r = w_uk.shape[2]
    dv = w_uv.shape[1]
    out = np.zeros((B, S, H, dv))
    lse = np.full((B, S, H), -np.inf)
    todo = only if only is not None else [(b, s, h) for b in range(B) for s in range(S) for h in range(H)]
    rows_of = {}                                # latent rows of the sequence being worked on
    for (b, s, h) in todo:
        if b not in rows_of:
            rows_of = {b: gather_latent(cache, page_table[b], int(seqlens[b]), page_size)}
        n = visible_tokens(seqlens[b], S, s)
        if n == 0:
            continue
        c = rows_of[b][:n, :r]
        k_r = rows_of[b][:n, r:]
        k_c = c @ w_uk[h].T                     # [n, dn]   k^C_{j,h} = W_UK_h c_j
        v = c @ w_uv[h].T                       # [n, dv]   v_{j,h}   = W_UV_h c_j
        z = (k_c @ q_nope[b, s, h] + k_r @ q_pe[b, s, h]) * scale
        m = z.max()
        e = np.exp(z - m)
        out[b, s, h] = (e / e.sum()) @ v
        lse[b, s, h] = m + np.log(e.sum())
    return out, lse


# --------------------------------------------------------------------------------------------
# Prefill in the MHA form (Sec. 3.3, Eq. 8 and Eq. 9 left): a chunk of S query positions per sequence is
# what mla_decode_mha_form computes for that S; the library materialises the decompressed keys and
# values first, which is this function.
# --------------------------------------------------------------------------------------------
def decompress_kv(cache, page_row, n, w_uk, w_uv, page_size=64):
    """k^C_{j,h} = W_UK_h c_j and v_{j,h} = W_UV_h c_j (Eq. 8) for tokens 0..n-1 of one sequence.

    Returns k_c [n, H, dn], v [n, H, dv] and the stored rotated keys k^R [n, dR] (shared by the heads).
    """
    r = w_uk.shape[2]
    rows = gather_latent(cache, page_row, n, page_size)
    c, k_r = rows[:, :r], rows[:, r:]
    k_c = np.stack([c @ np.asarray(w_uk[h], np.float64).T for h in range(w_uk.shape[0])], axis=1)
    v = np.stack([c @ np.asarray(w_uv[h], np.float64).T for h in range(w_uv.shape[0])], axis=1)
    return k_c, v, k_r


# --------------------------------------------------------------------------------------------
# MLA decode, Absorb form (Eq. 9 right), in the steps the library exposes
# --------------------------------------------------------------------------------------------
def absorb(q_nope, q_pe, w_uk):
    """q_hat[b,s,h] = [W_UK_h^T q_nope[b,s,h] ; q_pe[b,s,h]]  (Eq. 9 right, first line)."""
    q_lat = np.einsum('bshn,hnr->bshr', np.asarray(q_nope, np.float64), np.asarray(w_uk, np.float64))
    return np.concatenate([q_lat, np.asarray(q_pe, np.float64)], axis=-1)


SEGMENT_COST_PAGES = 2   # what opening one more sequence costs a partition, in page-equivalents


def split_plan(seqlens, page_size, G, seg_cost=SEGMENT_COST_PAGES):
    """Balanced split of all cache pages of a batch over G partitions (index path; the library's own rule).

    Sequence b owns n_b = ceil(L_b / P) pages.  Every non-empty sequence is given seg_cost extra
    "virtual" slots in front of its pages, so that a partition which has to open a second sequence
    (load its queries, write out another partial result) receives that many fewer pages.  Slots are
    numbered in sequence order: cum[b] = sum over b' < b of (n_b' + seg_cost if n_b' > 0 else 0),
    T = cum[B]; page j of sequence b is slot cum[b] + seg_cost + j.  Partition i owns slots
    [floor(i*T/G), floor((i+1)*T/G)).  Returned: cum [B+1] and plan [G,4] with rows (slot_begin,
    slot_end, sequence of the first slot, sequence of the last slot); an empty partition has sequence
    fields -1.  Written as a plain walk over every slot.
    """
    B = len(seqlens)
    cum = np.zeros(B + 1, dtype=np.int64)
    owner_seq = []
    for b in range(B):
        n = (int(seqlens[b]) + page_size - 1) // page_size
        v = n + seg_cost if n > 0 else 0
        cum[b + 1] = cum[b] + v
        owner_seq += [b] * v
    T = int(cum[B])
    plan = np.zeros((G, 4), dtype=np.int32)
    for i in range(G):
        p0, p1 = (i * T) // G, ((i + 1) * T) // G
        plan[i] = (p0, p1, owner_seq[p0] if p1 > p0 else -1, owner_seq[p1 - 1] if p1 > p0 else -1)
    return cum.astype(np.int32), plan


def plan_segments(cum, plan, seg_cost=SEGMENT_COST_PAGES):
    """Segments = maximal page ranges inside one partition and one sequence.

    Returns a list of (partition i, sequence b, first page in b, end page in b, slot) with
    slot = i + b, which is distinct for distinct segments because walking the slots in order
    moves to a new segment only by increasing i, b or both.
    """
    segs = []
    for i in range(plan.shape[0]):
        p0, p1, b0, b1 = (int(v) for v in plan[i])
        if p1 <= p0:
            continue
        for b in range(b0, b1 + 1):
            first = int(cum[b]) + seg_cost                     # slot of page 0 of sequence b
            lo, hi = max(p0, first), min(p1, int(cum[b + 1]))
            if hi > lo:
                segs.append((i, b, lo - first, hi - first, i + b))
    return segs


def decode_partial(q_hat_rows, n_vis, rows, r, scale, tok_begin, tok_end):
    """One split of Eq. 9 right, second line, over tokens [tok_begin, tok_end) of a sequence.

    q_hat_rows [R, r+dR]; n_vis [R] visible-token count of each row; rows [L, r+dR] the
    sequence's latent rows.  Returns o [R, r] = softmax-weighted mean of c_j over the visible
    part of the range and lse [R]; a row with nothing visible in the range gets o = 0,
    lse = -inf.
    """
    R = q_hat_rows.shape[0]
    o = np.zeros((R, r))
    lse = np.full(R, -np.inf)
    for i in range(R):
        hi = min(tok_end, int(n_vis[i]))
        if hi <= tok_begin:
            continue
        k_hat = rows[tok_begin:hi]
        z = (k_hat @ q_hat_rows[i]) * scale
        m = z.max()
        e = np.exp(z - m)
        o[i] = (e / e.sum()) @ k_hat[:, :r]
        lse[i] = m + np.log(e.sum())
    return o, lse


def combine(partial_o, partial_lse, w_uv_h):
    """Merge splits of one (b, s, h) by their lse and up-project (Eq. 9 right, last line, before W_O).

    partial_o [n, r], partial_lse [n], w_uv_h [dv, r].  Returns (out [dv], lse).
    """
    partial_lse = np.asarray(partial_lse, np.float64)
    m = partial_lse.max() if len(partial_lse) else -np.inf
    if not np.isfinite(m):
        return np.zeros(w_uv_h.shape[0]), -np.inf
    w = np.exp(partial_lse - m)
    o_lat = (w / w.sum()) @ np.asarray(partial_o, np.float64)
    return w_uv_h @ o_lat, m + np.log(w.sum())


def mla_decode_absorbed_form(q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, scale,
                             page_size=64, G=1):
    """Absorb -> per-segment partials under split_plan(G) -> combine.  Same outputs as the MHA form."""
    q_hat = absorb(q_nope, q_pe, w_uk)
    B, S, H, _ = q_hat.shape
    r = w_uk.shape[2]
    dv = w_uv.shape[1]
    cum, plan = split_plan(seqlens, page_size, G)
    segs = plan_segments(cum, plan)
    out = np.zeros((B, S, H, dv))
    lse = np.full((B, S, H), -np.inf)
    for b in range(B):
        rows = gather_latent(cache, page_table[b], int(seqlens[b]), page_size)
        n_vis = np.array([visible_tokens(seqlens[b], S, s) for s in range(S) for _ in range(H)])
        q_rows = q_hat[b].reshape(S * H, -1)
        parts = [decode_partial(q_rows, n_vis, rows, r, scale, pb * page_size, pe * page_size)
                 for (_, bb, pb, pe, _) in segs if bb == b]
        for s in range(S):
            for h in range(H):
                i = s * H + h
                po = np.array([p[0][i] for p in parts]).reshape(len(parts), r)
                pl = np.array([p[1][i] for p in parts])
                out[b, s, h], lse[b, s, h] = combine(po, pl, w_uv[h])
    return out, lse


# --------------------------------------------------------------------------------------------
# Latent append, Sec. 3.3, Eq. 7 left: c = W_DKV x, k^R = RoPE(W_KR x, t)
# --------------------------------------------------------------------------------------------
def append_slot(page_row, pos, page_size):
    """(page, offset) of the cache row of the token at 0-based position pos."""
    return int(page_row[pos // page_size]), int(pos % page_size)


def latent_append(x, w_dkv_kr, positions, page_table, cache, r, theta=10000.0, page_size=64):
    """Write [W_DKV x_b ; RoPE(W_KR x_b, pos_b)] into the cache row of each sequence's new token.

    x [B, D]; w_dkv_kr [r+dR, D] (rows 0..r-1 = W_DKV, the rest = W_KR); positions [B];
    cache [num_pages, P, r+dR] float64, modified in place and returned.
    """
    x = np.asarray(x, np.float64)
    w = np.asarray(w_dkv_kr, np.float64)
    for b in range(x.shape[0]):
        y = w @ x[b]
        y[r:] = rope(y[r:], int(positions[b]), theta)
        page, off = append_slot(page_table[b], int(positions[b]), page_size)
        cache[page, off] = y
    return cache


# --------------------------------------------------------------------------------------------
# The steps either side of the attention: queries (Eq. 8, right column) and output projection
# (Eq. 9, last line).  Used by the layer-level entry point.
# --------------------------------------------------------------------------------------------
def mla_queries(x, positions, w_uq, w_qr, H, w_dq=None, theta=10000.0):
    """q^C and q^R of Eq. 8 (right column) for tokens x [T, D] at 0-based positions [T].

    Low-rank queries: c^Q = W_DQ x, q^C = W_UQ c^Q, q^R = RoPE(W_QR c^Q, t).  With w_dq = None the
    compression is skipped (full-rank queries: c^Q = x), which is the other variant the paper runs.
    w_uq [H*dn, Dq], w_qr [H*dR, Dq].  Returns q_nope [T, H, dn] and q_pe [T, H, dR]; RoPE acts on each
    head's dR-vector with d := dR.
    """
    x = np.asarray(x, np.float64)
    c_q = x if w_dq is None else x @ np.asarray(w_dq, np.float64).T
    T = x.shape[0]
    q_nope = (c_q @ np.asarray(w_uq, np.float64).T).reshape(T, H, -1)
    q_r = (c_q @ np.asarray(w_qr, np.float64).T).reshape(T, H, -1)
    q_pe = rope(q_r, np.asarray(positions)[:, None], theta)
    return q_nope, q_pe


def output_projection(o, w_o):
    """y_t = W_O [o_{t,1}; ...; o_{t,h}]  (Eq. 9, last line).  o [..., H, dv], w_o [D, H*dv]."""
    o = np.asarray(o, np.float64)
    return o.reshape(o.shape[:-2] + (-1,)) @ np.asarray(w_o, np.float64).T


def mla_layer_decode(x, w_uq, w_qr, w_dkv_kr, w_uk, w_uv, w_o, cache, page_table, seqlens, scale, r,
                     w_dq=None, theta=10000.0, page_size=64):
    """One attention layer's decode step for the S newest tokens of every sequence, x [B, S, D] -> y [B, S, D].

    Token (b, s) has position L_b - S + s.  Its latent row is appended (Eq. 7 left), queries are formed
    (Eq. 8 right), attention runs in the MHA form over the cache (Eq. 8-9 left) and W_O is applied.  `cache` is
    modified in place (float64).
    """
    x = np.asarray(x, np.float64)
    B, S, _ = x.shape
    H = w_uk.shape[0]
    for s in range(S):
        latent_append(x[:, s], w_dkv_kr, [int(L) - S + s for L in seqlens], page_table, cache, r, theta, page_size)
    pos = np.array([[int(L) - S + s for s in range(S)] for L in seqlens])
    q_nope, q_pe = mla_queries(x.reshape(B * S, -1), pos.reshape(-1), w_uq, w_qr, H, w_dq, theta)
    o, _ = mla_decode_mha_form(q_nope.reshape(B, S, H, -1), q_pe.reshape(B, S, H, -1), w_uk, w_uv, cache, page_table,
                               seqlens, scale, page_size)
    return output_projection(o, w_o)


# --------------------------------------------------------------------------------------------
# FP8 latent cache (the paper's abstract names FP8 quantisation as combinable with the method and says no more;
# the stored format below is this library's own reading).
#
# A cache row of one token holds, instead of r + dR bf16 values:
#   codes  r bytes   e4m3 codes of c_t / scale_t
#   k_pe   dR bf16   k^R_t / scale_t, rounded to bf16   (stored pre-divided so that a score is scale_t times one sum)
#   scale  1 fp32    scale_t = max_i |c_t[i]| / 448, rounded to fp32 (1.0 for an all-zero row)
# The value the attention sees is the dequantised row: c~_t = scale_t * decode(codes), k~R_t = scale_t * k_pe, and the
# result is Eq. 9 (MHA form above) on those values.  e4m3 is the 8-bit format of the OCP 8-bit floating point
# specification: 1 sign, 4 exponent (bias 7), 3 mantissa bits, no infinities, S.1111.111 = NaN, largest finite 448.
# --------------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_decode(codes):
    """Value of each e4m3 code (uint8 array) as float64; the two NaN codes decode to NaN."""
    codes = np.asarray(codes, dtype=np.uint8)
    sign = np.where(codes & 0x80, -1.0, 1.0)
    e = ((codes >> 3) & 0xF).astype(np.int64)
    m = (codes & 0x7).astype(np.float64)
    normal = sign * np.exp2(e - 7.0) * (1.0 + m / 8.0)
    subnormal = sign * np.exp2(-6.0) * (m / 8.0)
    out = np.where(e == 0, subnormal, normal)
    return np.where((codes & 0x7F) == 0x7F, np.nan, out)


def e4m3_encode(x):
    """Nearest e4m3 code of each value (ties to the even code), saturating at +-448.  Written as a search over the
    126 non-negative finite codes, so that it shares nothing with the decoder but the table of values."""
    x = np.asarray(x, dtype=np.float64)
    grid = e4m3_decode(np.arange(0x7F, dtype=np.uint8))            # 0 .. 448, increasing with the code
    mag = np.minimum(np.abs(x), E4M3_MAX)
    hi = np.clip(np.searchsorted(grid, mag, side='left'), 0, len(grid) - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = mag - grid[lo], grid[hi] - mag
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))     # a tie goes to the code with an even mantissa
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(x), code | 0x80, code).astype(np.uint8)


def _round_bf16(x):
    """float64 -> nearest bf16 value (ties to even), returned as float64."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def quantize_latent_rows(rows, r):
    """rows [..., r+dR] float64 -> (codes uint8 [..., r], k_pe float64 [..., dR] (bf16 values), scale float64 [...])."""
    rows = np.asarray(rows, np.float64)
    c, k = rows[..., :r], rows[..., r:]
    amax = np.abs(c).max(axis=-1)
    scale = np.where(amax > 0, amax / E4M3_MAX, 1.0).astype(np.float32).astype(np.float64)
    codes = e4m3_encode(c / scale[..., None])
    return codes, _round_bf16(k / scale[..., None]), scale


def dequantize_latent_rows(codes, k_pe, scale):
    """The rows the attention sees: [scale * decode(codes) ; scale * k_pe], float64."""
    scale = np.asarray(scale, np.float64)[..., None]
    return np.concatenate([scale * e4m3_decode(codes), scale * np.asarray(k_pe, np.float64)], axis=-1)


def mla_decode_fp8_cache(q_nope, q_pe, w_uk, w_uv, codes, k_pe, scale, page_table, seqlens, softmax_scale, page_size=64,
                         only=None):
    """Eq. 9 over an FP8 latent cache: dequantise every row, then the MHA form above.

    codes [num_pages, P, r] uint8, k_pe [num_pages, P, dR], scale [num_pages, P].  Rows that no sequence owns may hold
    anything (NaN codes included): they are never gathered.
    """
    with np.errstate(invalid='ignore'):
        cache = dequantize_latent_rows(codes, k_pe, scale)
    return mla_decode_mha_form(q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, softmax_scale, page_size, only)


def latent_append_fp8(x, w_dkv_kr, positions, page_table, codes, k_pe, scale, r, theta=10000.0, page_size=64):
    """Eq. 7 left, then the quantisation above, into the FP8 cache arrays (modified in place)."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w_dkv_kr, np.float64)
    for b in range(x.shape[0]):
        y = w @ x[b]
        y[r:] = rope(y[r:], int(positions[b]), theta)
        page, off = append_slot(page_table[b], int(positions[b]), page_size)
        codes[page, off], k_pe[page, off], scale[page, off] = quantize_latent_rows(y, r)
    return codes, k_pe, scale
