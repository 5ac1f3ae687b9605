"""GPU parity of the FP8 latent-cache path (C ABI) against the fp64 oracle.

The cache bytes are produced by the oracle's quantiser on the CPU from seeded N(0,1) rows (scaled row by row so that
the scales differ), so that the CUDA path and the oracle read the same bytes; the append is the one case where the
CUDA path produces the bytes itself.
"""
import numpy as np
import pytest
import torch

from oracle import mla_oracle as orc
from paper_2502_07864_b200 import binding, synth
from tests import gpu_util as gu
from tests import lifts

pytestmark = pytest.mark.gpu
ROW = binding.FP8_ROW_BYTES


def pack_fp8_cache(codes, k_pe, scale):
    """Oracle arrays -> the byte layout of the library: [num_pages, P, 656] uint8."""
    n, P, r = codes.shape
    out = np.zeros((n, P, ROW), dtype=np.uint8)
    out[..., :r] = codes
    kb = torch.tensor(k_pe, dtype=torch.float64).to(torch.bfloat16).view(torch.int16).numpy()
    out[..., r:r + 128] = kb.view(np.uint8).reshape(n, P, 128)
    out[..., 640:644] = scale.astype(np.float32).view(np.uint8).reshape(n, P, 4)
    return out


def fp8_case(shape, seqlens, seed, poison=True):
    case = synth.make_decode_case(shape, seqlens, seed)
    rng = np.random.default_rng(seed)
    rows = lifts.f64(case['cache']) * rng.uniform(0.5, 2.0, size=case['cache'].shape[:2] + (1,))
    codes, k_pe, scale = orc.quantize_latent_rows(rows, shape.r)
    if poison:   # rows that no sequence owns: NaN codes, NaN k_pe, NaN scale
        owned = np.zeros(codes.shape[:2], bool)
        for b, L in enumerate(seqlens):
            for j in range((L + 63) // 64):
                owned[int(case['page_table'][b, j]), :min(64, L - 64 * j)] = True
        codes[~owned] = 0x7F
        k_pe[~owned] = np.nan
        scale[~owned] = np.nan
    case['fp8'] = (codes, k_pe, scale)
    case['cache_fp8'] = torch.tensor(pack_fp8_cache(codes, k_pe, scale))
    return case


def run_fp8(shape, case, scale, G=0):
    B = case['seqlens'].numel()
    params = binding.make_params(shape, B, case['cache_fp8'].shape[0], case['page_table'].shape[1], scale, num_partitions=G)
    ws, lay = binding.alloc_workspace(params)
    ws.view(torch.int32).fill_(0x7FC00000 - (1 << 32) if False else -4194304)   # NaN bit patterns in the workspace
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.full((B, shape.S, shape.H, shape.dv), float('nan'), dtype=torch.bfloat16, device='cuda')
    lse = torch.full((B, shape.S, shape.H), float('nan'), dtype=torch.float32, device='cuda')
    d = {k: case[k].cuda() for k in ('q_nope', 'q_pe', 'w_uk', 'w_uv', 'cache_fp8', 'page_table', 'seqlens')}
    binding.transmla_mla_decode_fp8(params, d['q_nope'], d['q_pe'], d['w_uk'], d['cache_fp8'], d['page_table'], d['seqlens'], ws,
                                    status)
    binding.transmla_mla_combine(params, ws, d['w_uv'], out, lse, status)
    torch.cuda.synchronize()
    return out, lse, int(status.item())


def oracle_fp8(shape, case, scale, only=None):
    c = lifts.case_f64({k: case[k] for k in ('q_nope', 'q_pe', 'w_uk', 'w_uv', 'page_table', 'seqlens')})
    codes, k_pe, sc = case['fp8']
    return orc.mla_decode_fp8_cache(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], codes, k_pe, sc, c['page_table'],
                                    c['seqlens'], scale, only=only)


@pytest.mark.parametrize('seqlens,G', [([200, 327, 1000], 0), ([64 * 9], 4), ([1, 2, 63, 0], 2), ([4096 + 17, 33], 13),
                                       ([8192], 0)])
def test_fp8_decode_llama_shape(seqlens, G):
    gu.ensure_built()
    shape = synth.LLAMA2_7B
    scale = gu.mla_scale(shape)
    case = fp8_case(shape, seqlens, seed=21)
    out, lse, status = run_fp8(shape, case, scale, G)
    assert status == 0
    only = None if sum(seqlens) < 3000 else [(b, 0, h) for b in range(len(seqlens)) for h in (0, 5, 31)]
    want, want_lse = oracle_fp8(shape, case, scale, only=only)
    got, got_lse = lifts.f64(out), lifts.f64(lse)
    if only is not None:
        idx = tuple(np.array(only).T)
        got, want, got_lse, want_lse = got[idx], want[idx], got_lse[idx], want_lse[idx]
    gu.assert_close(got, want, f'fp8 cache {seqlens}')
    gu.assert_lse_close(got_lse, want_lse, 'fp8 cache lse')


def test_fp8_decode_two_query_positions_and_many_rows():
    gu.ensure_built()
    shape = synth.QWEN25_72B
    scale = gu.mla_scale(shape)
    case = fp8_case(shape, [131, 700, 64], seed=22)
    out, lse, status = run_fp8(shape, case, scale, 0)
    assert status == 0
    only = [(b, s, h) for b in range(3) for s in range(2) for h in (0, 17, 63)]
    want, want_lse = oracle_fp8(shape, case, scale, only=only)
    idx = tuple(np.array(only).T)
    gu.assert_close(lifts.f64(out)[idx], want[idx], 'fp8 cache, S = 2')
    gu.assert_lse_close(lifts.f64(lse)[idx], want_lse[idx], 'fp8 cache lse, S = 2')


def test_fp8_append_writes_the_quantised_row():
    gu.ensure_built()
    shape = synth.LLAMA2_7B
    positions = [8191, 0, 77, 130]
    B = len(positions)
    seqlens = [p + 1 for p in positions]
    case = synth.make_decode_case(shape, seqlens, 23)
    ac = synth.make_append_case(shape, positions, 24)
    n_pages = case['cache'].shape[0]
    params = binding.make_params(shape, B, n_pages, case['page_table'].shape[1], 0.1)
    cache = torch.full((n_pages, 64, ROW), 0xA5, dtype=torch.uint8, device='cuda')
    scratch = torch.empty(B * shape.row, dtype=torch.float32, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    binding.transmla_latent_append_fp8(params, ac['x'].cuda(), ac['w_dkv_kr'].cuda(), ac['positions'].cuda(),
                                       case['page_table'].cuda(), cache, scratch, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = cache.cpu().numpy()
    codes = np.zeros((n_pages, 64, shape.r), np.uint8)
    k_pe, sc = np.zeros((n_pages, 64, shape.dR)), np.ones((n_pages, 64))
    orc.latent_append_fp8(lifts.f64(ac['x'][:, 0]), lifts.f64(ac['w_dkv_kr']), positions, case['page_table'].numpy(), codes, k_pe,
                          sc, shape.r)
    touched = np.zeros((n_pages, 64), bool)
    for b, pos in enumerate(positions):
        page, off = int(case['page_table'][b, pos // 64]), pos % 64
        touched[page, off] = True
        row = got[page, off]
        g_scale = float(row[640:644].view(np.float32)[0])
        assert abs(g_scale - sc[page, off]) <= 2e-3 * sc[page, off]          # fp32 sums against fp64 sums
        g_c = orc.e4m3_decode(row[:shape.r]) * g_scale
        w_c = orc.e4m3_decode(codes[page, off]) * sc[page, off]
        step = np.maximum(np.abs(w_c), sc[page, off] * 2.0 ** -6) * 2.0 ** -3   # one code step at that magnitude
        assert np.all(np.abs(g_c - w_c) <= step + 1e-6)
        assert np.mean(row[:shape.r] == codes[page, off]) > 0.97               # and nearly all codes are the same
        g_k = torch.tensor(row[512:640].copy()).view(torch.bfloat16).to(torch.float64).numpy() * g_scale
        assert np.all(np.abs(g_k - k_pe[page, off] * sc[page, off]) <= 2.0 ** -7 * np.abs(g_k) + 2e-3)
    assert np.all(got[~touched] == 0xA5)                                       # no other byte of the pool changed
