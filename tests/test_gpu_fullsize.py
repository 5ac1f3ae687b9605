"""GPU parity at the benchmark's full sizes, in the launch configuration the benchmark times.

The oracle cannot finish every output of these cases in seconds, so it computes a seeded sample of
(sequence, query position, head) outputs one by one; the CUDA results at those entries must meet the
same tolerances as everywhere else.  Inputs are generated on the device with a seeded generator and
only the sampled sequences' pages are copied back for the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import mla_oracle as orc
from paper_2502_07864_b200 import binding, synth
from tests import gpu_util as gu
from tests import lifts

pytestmark = pytest.mark.gpu


@pytest.fixture(scope='module', autouse=True)
def _lib():
    gu.ensure_built()


def sub_case(case, seqs, P=64):
    """The same inputs restricted to sequences `seqs`, with their pages packed into a small pool (CPU)."""
    seqlens = [int(case['seqlens'][b]) for b in seqs]
    n_pages = [(L + P - 1) // P for L in seqlens]
    table = torch.full((len(seqs), max(max(n_pages), 1)), -1, dtype=torch.int32)
    pages, k = [], 0
    for i, b in enumerate(seqs):
        idx = case['page_table'][b, :n_pages[i]].long()
        pages.append(case['cache'][idx].cpu())
        table[i, :n_pages[i]] = torch.arange(k, k + n_pages[i], dtype=torch.int32)
        k += n_pages[i]
    out = {k_: case[k_].cpu() for k_ in ('w_uk', 'w_uv')}
    out.update(q_nope=case['q_nope'][seqs].cpu(), q_pe=case['q_pe'][seqs].cpu(),
               cache=torch.cat(pages) if pages else case['cache'][:1].cpu(), page_table=table,
               seqlens=torch.tensor(seqlens, dtype=torch.int32))
    return out


def check_sampled(shape, seqlens, seed, n_seq=3, n_heads=3, extra_pages=0):
    scale = gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, seed, device='cuda', extra_pages=extra_pages)
    out, lse, status, _, _ = gu.gpu_decode(shape, case, scale, G=0)
    assert status == 0
    assert torch.all(torch.isfinite(out.float()))
    rng = np.random.default_rng(seed)
    B = len(seqlens)
    # always include the shortest and the longest sequence
    seqs = sorted(set([int(np.argmin(seqlens)), int(np.argmax(seqlens))] +
                      [int(b) for b in rng.choice(B, size=min(n_seq, B), replace=False)]))
    sub = sub_case(case, seqs)
    only = [(i, int(s), int(h)) for i in range(len(seqs)) for s in range(shape.S)
            for h in rng.choice(shape.H, size=n_heads, replace=False)]
    want, want_lse = gu.oracle_decode(shape, sub, scale, only=only)
    got = lifts.f64(out[seqs])
    got_lse = lifts.f64(lse[seqs])
    idx = tuple(np.array(only).T)
    gu.assert_close(got[idx], want[idx], f'sampled outputs B={B}')
    gu.assert_lse_close(got_lse[idx], want_lse[idx], 'sampled lse')
    return case


@pytest.mark.parametrize('B', [1, 4, 16, 64, 128])
def test_llama_shape_batch_sweep_at_8k(B):
    check_sampled(synth.LLAMA2_7B, [8192] * B, seed=3)


def test_ragged_long_context_batch32():
    seqlens = synth.uniform_seqlens(32, 1024, 32768, seed=4)
    check_sampled(synth.LLAMA2_7B, seqlens, seed=4)


def test_batch4_at_131072():
    check_sampled(synth.LLAMA2_7B, [131072] * 4, seed=4, n_seq=1, n_heads=2)


def test_qwen_like_two_query_positions_batch64():
    seqlens = synth.uniform_seqlens(64, 2048, 8192, seed=5)
    check_sampled(synth.QWEN25_72B, seqlens, seed=5)


def test_pool_larger_than_4_gib():
    """Byte offsets into the pool need more than 32 bits: 62 000 pages of 73 728 bytes are 4.57 GB, and the seeded
    permutation scatters the sequences' pages over all of it.  Decode is checked on sampled outputs, the append
    on every row it writes and on every byte it must leave alone."""
    shape, P = synth.LLAMA2_7B, synth.LLAMA2_7B.page_size
    seqlens = [8192, 8192, 3000, 70, 8192, 8192]
    case = check_sampled(shape, seqlens, seed=41, n_seq=2, n_heads=2, extra_pages=61000)
    num_pages = case['cache'].shape[0]
    assert num_pages * P * shape.row * 2 > 1 << 32
    table = case['page_table'].cpu()
    used = torch.cat([table[b, :(L + P - 1) // P] for b, L in enumerate(seqlens)])
    assert int(used.max()) * P * shape.row * 2 > 1 << 32, 'the draw must place some page beyond 4 GiB'
    # append the token at position L-1 of every sequence over what is there
    positions = [L - 1 for L in seqlens]
    ac = synth.make_append_case(shape, positions, 42, device='cuda')
    before = case['cache'].clone()
    params = binding.make_params(shape, len(seqlens), num_pages, table.shape[1], 1.0, num_partitions=1)
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    binding.transmla_latent_append(params, ac['x'], ac['w_dkv_kr'], ac['positions'], case['page_table'], case['cache'], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    slots = [orc.append_slot(table[b].numpy(), positions[b], P) for b in range(len(seqlens))]
    pg = torch.tensor([s[0] for s in slots]); off = torch.tensor([s[1] for s in slots])
    got = lifts.f64(case['cache'][pg.cuda(), off.cuda()].cpu())                      # [B, r + dR]
    small = np.zeros((len(seqlens), P, shape.row))                                 # one private page per sequence
    small_table = np.full((len(seqlens), table.shape[1]), -1, dtype=np.int32)
    for b_, pos in enumerate(positions):
        small_table[b_, pos // P] = b_
    orc.latent_append(lifts.f64(ac['x'][:, 0].cpu()), lifts.f64(ac['w_dkv_kr'].cpu()), positions, small_table, small,
                      shape.r, page_size=P)
    want = small[np.arange(len(seqlens)), off.numpy()]
    assert np.all(np.abs(got - want) <= 2.0 ** -7 * np.abs(want) + 1e-3)
    case['cache'][pg.cuda(), off.cuda()] = 0
    before[pg.cuda(), off.cuda()] = 0
    assert torch.equal(case['cache'].view(torch.int16), before.view(torch.int16))   # nothing else changed


# ------------------------------------------------------------------ every output at full size, by closed forms
@pytest.mark.parametrize('shape,B', [(synth.LLAMA2_7B, 16), (synth.QWEN25_72B, 8)])
def test_full_size_closed_forms_cover_every_output(shape, B):
    """Two properties that hold at any size and fix every output element of a full-size launch:
    identical cached rows give out = W_UV_h c whatever the queries are, and a zero softmax scale gives
    out = W_UV_h mean_j(c_j) with lse = ln(visible tokens)."""
    seqlens = [8192] * B
    case = synth.make_decode_case(shape, seqlens, seed=23, device='cuda')
    w_uv = lifts.f64(case['w_uv'])
    # (1) zero scale on the random cache
    out, lse, status, _, _ = gu.gpu_decode(shape, case, 0.0, G=0)
    assert status == 0
    got, got_lse = lifts.f64(out), lifts.f64(lse)
    for b in range(B):
        idx = case['page_table'][b, :8192 // 64].long()
        rows = case['cache'][idx].reshape(-1, shape.row)[:, :shape.r].double()
        for s in range(shape.S):
            n = 8192 - (shape.S - 1 - s)
            want = w_uv @ rows[:n].mean(0).cpu().numpy()                      # [H, dv]
            gu.assert_close(got[b, s], want, f'uniform mean b={b} s={s}')
            assert np.abs(got_lse[b, s] - np.log(n)).max() < 1e-3
    # (2) every row of a sequence equal to its first row, ordinary scale
    for b in range(B):
        idx = case['page_table'][b, :8192 // 64].long()
        first = case['cache'][idx[0], 0].clone()
        case['cache'][idx] = first
    out, _, status, _, _ = gu.gpu_decode(shape, case, gu.mla_scale(shape), G=0)
    assert status == 0
    got = lifts.f64(out)
    for b in range(B):
        c = lifts.f64(case['cache'][case['page_table'][b, 0].long(), 0, :shape.r])
        want = w_uv @ c
        for s in range(shape.S):
            gu.assert_close(got[b, s], want, f'identical rows b={b} s={s}')


def test_prefill_chunk_of_2048_positions_over_8192_tokens_sampled():
    # the prefill workload bench.py times (B = 4 x 8192 cached tokens, S = 2048): sampled (sequence, position, head)
    # outputs against the oracle, among them the first and last position of the chunk and both sides of a 128-row tile
    shape = synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=2048)
    seqlens = [8192] * 4
    scale = gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, 8, device='cuda')
    params = binding.make_params(shape, 4, case['cache'].shape[0], case['page_table'].shape[1], scale)
    scratch = torch.empty(binding.transmla_prefill_scratch_bytes(params) // 2, dtype=torch.bfloat16, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.full((4, 2048, 32, 128), float('nan'), dtype=torch.bfloat16, device='cuda')
    lse = torch.full((4, 2048, 32), float('nan'), dtype=torch.float32, device='cuda')
    binding.transmla_mla_prefill(params, case['q_nope'], case['q_pe'], case['w_uk'], case['w_uv'], case['cache'],
                                 case['page_table'], case['seqlens'], scratch, out, lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.all(torch.isfinite(out.float()))
    seqs = [0, 3]
    sub = sub_case(case, seqs)
    rng = np.random.default_rng(8)
    positions = [0, 1, 127, 128, 1000, 2047]
    only = [(i, s, int(h)) for i in range(len(seqs)) for s in positions for h in rng.choice(32, size=2, replace=False)]
    want, want_lse = gu.oracle_decode(shape, sub, scale, only=only)
    idx = tuple(np.array(only).T)
    gu.assert_close(lifts.f64(out[seqs])[idx], want[idx], 'prefill sampled outputs at the benchmark size')
    gu.assert_lse_close(lifts.f64(lse[seqs])[idx], want_lse[idx], 'prefill sampled lse')
