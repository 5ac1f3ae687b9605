"""Prefill in the MHA form (Sec. 3.3, Eq. 8 + Eq. 9 left) through the C ABI against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import mla_oracle as orc
from paper_2502_07864_b200 import binding, synth
from tests import gpu_util as gu
from tests import lifts

pytestmark = pytest.mark.gpu


def _prefill(shape, case, scale, poison=True):
    B = case['seqlens'].numel()
    params = binding.make_params(shape, B, case['cache'].shape[0], case['page_table'].shape[1], scale)
    n = binding.transmla_prefill_scratch_bytes(params)
    assert n == case['cache'].shape[0] * 64 * shape.H * (shape.dn + shape.dv) * 2
    scratch = torch.empty(n // 2, dtype=torch.bfloat16, device='cuda')
    if poison:
        scratch.view(torch.int16).fill_(0x7fc1)  # NaN pattern: nothing may be read that was not written
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.full((B, shape.S, shape.H, shape.dv), float('nan'), dtype=torch.bfloat16, device='cuda')
    lse = torch.full((B, shape.S, shape.H), float('nan'), dtype=torch.float32, device='cuda')
    binding.transmla_mla_prefill(params, case['q_nope'], case['q_pe'], case['w_uk'], case['w_uv'], case['cache'],
                                 case['page_table'], case['seqlens'], scratch, out, lse, status)
    torch.cuda.synchronize()
    return out, lse, int(status.item()), scratch.view(case['cache'].shape[0], 64, shape.H, shape.dn + shape.dv)


def test_decompressed_store_matches_the_oracle_row_by_row():
    gu.ensure_built()
    shape = synth.MLAShape(H=3, dn=128, dR=64, dv=128, r=512, D=4096, S=4)
    seqlens = [130, 64, 5, 300]
    case = synth.make_decode_case(shape, seqlens, seed=31, nan_tails=True)
    out, lse, status, store = _prefill(shape, gu.to_dev(case), gu.mla_scale(shape))
    assert status == 0
    c = lifts.case_f64(case)
    store = store.cpu()
    named = set()
    for b, L in enumerate(seqlens):
        k_c, v, _ = orc.decompress_kv(c['cache'], c['page_table'][b], L, c['w_uk'], c['w_uv'], 64)
        n_pages = (L + 63) // 64
        for j in range(n_pages):
            pg = int(case['page_table'][b, j])
            named.add(pg)
            rows = min(64, L - j * 64)
            got = lifts.f64(store[pg, :rows])
            want = np.concatenate([k_c[j * 64:j * 64 + rows], v[j * 64:j * 64 + rows]], axis=2)
            gu.assert_close(got, want, f'decompressed rows of sequence {b} page {j}')
            assert torch.all(store[pg, rows:].view(torch.int16) == 0), 'rows beyond the sequence must be zeros'
    for pg in range(store.shape[0]):
        if pg not in named:
            assert torch.all(store[pg].view(torch.int16) == 0x7fc1), 'a page nobody names was written'


@pytest.mark.parametrize('S,seqlens', [(130, [130, 257, 64, 1000]), (1, [1, 64, 65]), (64, [64, 200]), (300, [320, 1100])])
def test_prefill_all_outputs_small_head_count(S, seqlens):
    # every output and lse; S = 130 and 300 leave the last 128-row tile ragged, L = S is a pure prefill,
    # L = 64 < S = 130 leaves the first positions with nothing to see (zeros, lse = -inf)
    gu.ensure_built()
    shape = synth.MLAShape(H=2, dn=128, dR=64, dv=128, r=512, D=4096, S=S)
    case = synth.make_decode_case(shape, seqlens, seed=32 + S, nan_tails=True)
    out, lse, status, _ = _prefill(shape, gu.to_dev(case), gu.mla_scale(shape))
    assert status == 0
    want, want_lse = gu.oracle_decode(shape, case, gu.mla_scale(shape))
    gu.assert_close(lifts.f64(out), want, 'prefill out')
    gu.assert_lse_close(lse.cpu().numpy(), want_lse, 'prefill lse')
    for b, L in enumerate(seqlens):
        for s in range(S):
            if orc.visible_tokens(L, S, s) == 0:
                assert torch.all(out[b, s] == 0) and torch.all(torch.isneginf(lse[b, s]))


def test_prefill_llama_heads_sampled_outputs():
    gu.ensure_built()
    shape = synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=200)
    seqlens = [300, 200, 1100]
    case = synth.make_decode_case(shape, seqlens, seed=33)
    out, lse, status, _ = _prefill(shape, gu.to_dev(case), gu.mla_scale(shape))
    assert status == 0
    only = [(b, s, h) for b in range(3) for s in (0, 1, 63, 64, 127, 128, 199) for h in (0, 13, 31)]
    want, want_lse = gu.oracle_decode(shape, case, gu.mla_scale(shape), only=only)
    idx = tuple(np.array(only).T)
    gu.assert_close(lifts.f64(out)[idx], want[idx], 'prefill sampled')
    gu.assert_lse_close(lse.cpu().numpy()[idx], want_lse[idx], 'prefill sampled lse')


def test_prefill_agrees_with_the_oracle_where_the_absorbed_path_is_also_checked():
    # the same case through both forms: each is compared with the oracle (Eq. 9: left == right)
    gu.ensure_built()
    shape = synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=8)
    seqlens = [520, 8, 131]
    case = synth.make_decode_case(shape, seqlens, seed=34)
    dev = gu.to_dev(case)
    want, want_lse = gu.oracle_decode(shape, case, gu.mla_scale(shape))
    out_p, lse_p, st_p, _ = _prefill(shape, dev, gu.mla_scale(shape))
    out_a, lse_a, st_a, _, _ = gu.gpu_decode(shape, dev, gu.mla_scale(shape))
    assert st_p == 0 and st_a == 0
    gu.assert_close(lifts.f64(out_p), want, 'MHA form')
    gu.assert_close(lifts.f64(out_a), want, 'absorbed form')
    gu.assert_lse_close(lse_p.cpu().numpy(), want_lse, 'MHA form lse')


def test_prefill_reports_a_bad_page_index_and_stays_usable():
    gu.ensure_built()
    shape = synth.MLAShape(H=2, dn=128, dR=64, dv=128, r=512, D=4096, S=16)
    case = synth.make_decode_case(shape, [100, 200], seed=35)
    bad = {k: (v.clone() if isinstance(v, torch.Tensor) else v) for k, v in case.items()}
    bad['page_table'][1, 1] = 10 ** 6
    _, _, status, _ = _prefill(shape, gu.to_dev(bad), gu.mla_scale(shape))
    assert status & 1  # TRANSMLA_DEV_BAD_PAGE
    out, lse, status, _ = _prefill(shape, gu.to_dev(case), gu.mla_scale(shape))
    assert status == 0
    want, _ = gu.oracle_decode(shape, case, gu.mla_scale(shape))
    gu.assert_close(lifts.f64(out), want, 'after a bad call')


def test_prefill_rejects_shapes_it_is_not_built_for():
    gu.ensure_built()
    params = binding.make_params(synth.TINY, 2, 4, 2, 0.1)
    assert binding.transmla_prefill_scratch_bytes(params) == 0
    t = torch.zeros(1024, dtype=torch.bfloat16, device='cuda')
    i = torch.zeros(8, dtype=torch.int32, device='cuda')
    with pytest.raises(binding.TransMLAError):
        binding.transmla_mla_prefill(params, t, t, t, t, t, i, i, t, t)
