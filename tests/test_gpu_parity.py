"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded bytes.

Tolerances (bf16 storage, fp32 accumulation): max-abs 2e-2 and relative L2 5e-3 on outputs;
index paths (split plan, page slots, untouched cache bytes) bit-exact.
"""
import math

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


def _run_and_compare(shape, seqlens, seed, G=0, scale=None, nan_tails=True, check_internals=False):
    scale = scale if scale is not None else gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, seed, nan_tails=nan_tails)
    out, lse, status, views, lay = gu.gpu_decode(shape, gu.to_dev(case), scale, G=G, want_views=check_internals,
                                                 fixed_plan=check_internals)
    assert status == 0
    want_out, want_lse = gu.oracle_decode(shape, case, scale)
    gu.assert_close(lifts.f64(out), want_out, f'out seqlens={seqlens} G={G}')
    gu.assert_lse_close(lifts.f64(lse), want_lse, 'lse')
    if check_internals:
        c = lifts.case_f64(case)
        # index path: bit-exact
        cum, plan = orc.split_plan(seqlens, shape.page_size, lay.num_partitions)
        assert np.array_equal(views['cum_pages'].cpu().numpy(), cum)
        assert np.array_equal(views['plan'].cpu().numpy(), plan)
        want_parts = np.array([[0, -1]] * len(seqlens))
        for (i, b, _, _, _) in orc.plan_segments(cum, plan):
            want_parts[b] = (i, i) if want_parts[b][1] < 0 else (min(want_parts[b][0], i), max(want_parts[b][1], i))
        assert np.array_equal(views['seq_parts'].cpu().numpy(), want_parts)
        # absorbed queries: bf16 rounding of an fp32 sum
        q_hat = orc.absorb(c['q_nope'], c['q_pe'], c['w_uk'])
        got = lifts.f64(views['q_hat'])
        assert np.all(np.abs(got - q_hat) <= 2.0 ** -7 * np.abs(q_hat) + 1e-3)
        # per-segment partials against the oracle's own split of Eq. 9
        B, S, H, r = len(seqlens), shape.S, shape.H, shape.r
        po, pl = lifts.f64(views['partial_o']), lifts.f64(views['partial_lse'])
        for (i, b, pb, pe, slot) in orc.plan_segments(cum, plan):
            rows = orc.gather_latent(c['cache'], c['page_table'][b], int(seqlens[b]), shape.page_size)
            n_vis = np.array([orc.visible_tokens(seqlens[b], S, s) for s in range(S) for _ in range(H)])
            # the CUDA path rounds q_hat to bf16 before the contraction; the tolerance covers it
            o, l = orc.decode_partial(q_hat[b].reshape(S * H, -1), n_vis, rows, r, scale,
                                      pb * shape.page_size, pe * shape.page_size)
            gu.assert_close(po[slot], o, f'partial_o slot {slot}')
            gu.assert_lse_close(pl[slot], l, f'partial_lse slot {slot}')
    return out, lse


# ------------------------------------------------------------------ config 1: tiny, element by element
@pytest.mark.parametrize('G', [0, 1, 2, 3, 7])
def test_tiny_config_all_outputs_and_internals(G):
    _run_and_compare(synth.TINY, [17, 64], seed=1, G=G, check_internals=True)


def test_tiny_ragged_many_sequences():
    _run_and_compare(synth.TINY, [1, 63, 64, 65, 128, 129, 200, 5, 700], seed=21, G=5, check_internals=True)


@pytest.mark.parametrize('which', ['selector', 'replicated'])
def test_gqa_lifts_reproduce_gqa(which):
    # Sec. 4.1 / App. A.2.1: a GQA layer written as MLA gives the GQA output.
    rng = np.random.default_rng(31)
    if which == 'selector':
        ref, m = lifts.selector_lift(rng, T=150)
        shape = synth.MLAShape(H=8, dn=32, dR=0, dv=32, r=128, D=48)
    else:
        ref, m = lifts.replicated_lift(rng, T=150)
        shape = synth.TINY
    bf = lambda a: torch.tensor(np.nan_to_num(a, nan=0.0) if a.dtype.kind == 'f' else a)
    case = {k: bf(m[k]).to(torch.bfloat16) for k in ('q_nope', 'q_pe', 'w_uk', 'w_uv')}
    cache = torch.tensor(m['cache']).to(torch.bfloat16)        # NaN tails stay NaN
    case.update(cache=cache, page_table=torch.tensor(m['page_table']), seqlens=torch.tensor(m['seqlens']))
    out, lse, status, _, _ = gu.gpu_decode(shape, gu.to_dev(case), m['scale'], G=3)
    assert status == 0
    want, _ = gu.oracle_decode(shape, case, m['scale'])
    gu.assert_close(lifts.f64(out), want, which)
    # and, up to the bf16 rounding of the lifted inputs, the original GQA output
    assert np.abs(lifts.f64(out)[0, 0] - ref).max() < 5e-2


# ------------------------------------------------------------------ production shape, sizes spanning tiles + tails
@pytest.mark.parametrize('seqlens,G', [([200, 327, 1000], 0), ([64 * 9], 4), ([1, 2, 63], 2), ([4096 + 17, 33], 13)])
def test_llama_shape_medium(seqlens, G):
    _run_and_compare(synth.LLAMA2_7B, seqlens, seed=2, G=G, check_internals=(len(seqlens) == 3 and G == 0))


@pytest.mark.parametrize('H,S', [(8, 1), (40, 1), (24, 2)])
def test_production_latent_with_row_counts_that_do_not_fill_a_block(H, S):
    # r = 512, dR = 64 goes through the TMA/tcgen05 kernel; S*H = 8, 40, 48 leave the last 32-row block ragged
    shape = synth.MLAShape(H=H, dn=128, dR=64, dv=128, r=512, D=4096, S=S)
    _run_and_compare(shape, [300, 64, 2, 1100], seed=17, G=5, check_internals=True)


def test_wide_heads_and_many_sequences():
    # dn = dv = 256 (largest supported head dims) on the small latent; 5000 one-page sequences make the plan
    # block take its global-memory path (more sequences than its shared-memory buffer holds)
    shape = synth.MLAShape(H=4, dn=256, dR=16, dv=256, r=64, D=256)
    _run_and_compare(shape, [70, 5, 129], seed=18, G=3)
    many = [1 + (i * 7) % 60 for i in range(5000)]
    case = synth.make_decode_case(synth.TINY, many, seed=19)
    out, lse, status, views, lay = gu.gpu_decode(synth.TINY, gu.to_dev(case), gu.mla_scale(synth.TINY), G=0, want_views=True)
    assert status == 0
    cum, plan = orc.split_plan(many, 64, lay.num_partitions)
    assert np.array_equal(views['cum_pages'].cpu().numpy(), cum) and np.array_equal(views['plan'].cpu().numpy(), plan)
    only = [(b, 0, h) for b in (0, 1, 2499, 4999) for h in (0, 7)]
    want, want_lse = gu.oracle_decode(synth.TINY, case, gu.mla_scale(synth.TINY), only=only)
    idx = tuple(np.array(only).T)
    gu.assert_close(lifts.f64(out)[idx], want[idx], 'many sequences')


def test_qwen_shape_two_query_positions():
    shape = synth.QWEN25_72B
    _run_and_compare(shape, [130, 300, 2], seed=5, G=6, check_internals=True)


def test_empty_sequences_and_short_pairs():
    shape = synth.MLAShape(H=8, dn=32, dR=16, dv=32, r=64, D=256, S=2)
    out, lse = _run_and_compare(shape, [0, 1, 2, 70], seed=7, G=3)
    assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))
    assert torch.all(out[1, 0] == 0) and torch.all(torch.isneginf(lse[1, 0]))   # L=1, S=2: query 0 sees nothing


def test_results_are_bitwise_reproducible():
    shape = synth.LLAMA2_7B
    case = gu.to_dev(synth.make_decode_case(shape, [777, 1500], 8))
    a = gu.gpu_decode(shape, case, gu.mla_scale(shape), G=9)
    b = gu.gpu_decode(shape, case, gu.mla_scale(shape), G=9)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_page_permutation_gives_identical_bits():
    shape = synth.LLAMA2_7B
    case = synth.make_decode_case(shape, [500, 129], 9)
    a = gu.gpu_decode(shape, gu.to_dev(case), gu.mla_scale(shape), G=5)
    n = case['cache'].shape[0]
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(3))
    case2 = dict(case)
    case2['cache'] = torch.empty_like(case['cache'])
    case2['cache'][perm] = case['cache']
    pt = case['page_table'].long()
    case2['page_table'] = torch.where(pt >= 0, perm[pt.clamp(min=0)], pt).to(torch.int32)
    b = gu.gpu_decode(shape, gu.to_dev(case2), gu.mla_scale(shape), G=5)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_bad_page_index_is_reported_not_fatal():
    shape = synth.TINY
    case = synth.make_decode_case(shape, [100, 64], 10)
    case['page_table'][0, 1] = case['cache'].shape[0] + 5
    out, lse, status, _, _ = gu.gpu_decode(shape, gu.to_dev(case), 0.1, G=2)
    assert status & 1
    # the skipped page contributes nothing: same as a 64-token first sequence
    case['seqlens'][0] = 64
    want, _ = gu.oracle_decode(shape, case, 0.1)
    gu.assert_close(lifts.f64(out), want, 'bad page skipped')


@pytest.mark.parametrize('shape', [synth.TINY, synth.LLAMA2_7B])
def test_sequence_length_beyond_the_page_table_is_clamped_and_reported(shape):
    # a length for which the page table has no entries: clamped to max_pages * P (nothing is read outside the
    # table's row), reported through the status word, and the result is that of the clamped length
    case = synth.make_decode_case(shape, [130, 192], 12)          # 3 pages per sequence, all of them owned
    max_pages = case['page_table'].shape[1]
    case['seqlens'][1] = max_pages * 64 + 1000
    case['seqlens'][0] = -7
    scale = gu.mla_scale(shape)
    for G in (0, 3):
        out, lse, status, _, _ = gu.gpu_decode(shape, gu.to_dev(case), scale, G=G)
        assert status == 4
        want_case = dict(case)
        want_case['seqlens'] = torch.tensor([0, max_pages * 64], dtype=torch.int32)
        want, want_lse = gu.oracle_decode(shape, want_case, scale)
        gu.assert_close(lifts.f64(out), want, 'clamped length')
        gu.assert_lse_close(lifts.f64(lse), want_lse, 'clamped length lse')


def test_combine_alone_on_oracle_partials():
    # feed the oracle's per-segment partials to the CUDA combine and compare with the oracle's result
    shape = synth.TINY
    seqlens = [300, 64, 0, 129]
    scale = gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, 11)
    c = lifts.case_f64(case)
    G = 6
    params = binding.make_params(shape, len(seqlens), case['cache'].shape[0], case['page_table'].shape[1], scale, G)
    ws, lay = binding.alloc_workspace(params)
    ws.zero_()
    v = binding.workspace_views(params, ws, lay)
    cum, plan = orc.split_plan(seqlens, 64, G)
    v['cum_pages'].copy_(torch.tensor(cum))
    parts = np.array([[0, -1]] * len(seqlens), dtype=np.int32)
    for (i, b, _, _, _) in orc.plan_segments(cum, plan):
        parts[b] = (i, i) if parts[b][1] < 0 else (min(parts[b][0], i), max(parts[b][1], i))
    v['seq_parts'].copy_(torch.tensor(parts))
    v['partial_lse'].fill_(float('nan'))
    v['partial_o'].fill_(float('nan'))
    q_hat = orc.absorb(c['q_nope'], c['q_pe'], c['w_uk'])
    for (i, b, pb, pe, slot) in orc.plan_segments(cum, plan):
        rows = orc.gather_latent(c['cache'], c['page_table'][b], seqlens[b], 64)
        o, l = orc.decode_partial(q_hat[b].reshape(shape.H, -1), np.full(shape.H, seqlens[b]), rows, shape.r, scale,
                                  pb * 64, pe * 64)
        v['partial_o'][slot] = torch.tensor(o, dtype=torch.float32)
        v['partial_lse'][slot] = torch.tensor(l, dtype=torch.float32)
    out = torch.empty(len(seqlens), 1, shape.H, shape.dv, dtype=torch.bfloat16, device='cuda')
    lse = torch.empty(len(seqlens), 1, shape.H, dtype=torch.float32, device='cuda')
    binding.transmla_mla_combine(params, ws, case['w_uv'].cuda(), out, lse)
    torch.cuda.synchronize()
    want, want_lse = gu.oracle_decode(shape, case, scale)
    gu.assert_close(lifts.f64(out), want, 'combine')
    gu.assert_lse_close(lifts.f64(lse), want_lse, 'combine lse')


def test_a_wait_that_nothing_satisfies_ends_by_itself_and_leaves_the_context_usable():
    import time
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    cycles = torch.zeros(2, dtype=torch.int64, device='cuda')
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    binding.transmla_selftest_bounded_wait(status, cycles)
    torch.cuda.synchronize()
    took = time.perf_counter() - t0
    assert int(status.item()) & 2                    # TRANSMLA_DEV_TIMEOUT
    assert 0.05 < took < 2.0
    first, second = (int(v) for v in cycles.tolist())
    assert first > 100_000_000 and second < 100_000  # the second wait does not spin again
    _run_and_compare(synth.TINY, [17, 64], seed=1, G=2)   # and ordinary work still runs afterwards


# ------------------------------------------------------------------ append
@pytest.mark.parametrize('shape,positions', [(synth.TINY, [16, 63, 64, 0]), (synth.LLAMA2_7B, [8191, 0, 77, 131071]),
                                             (synth.QWEN25_72B, [126, 63, 4000]),
                                             (synth.TINY, [(7 * i) % 200 for i in range(150)]),       # several token splits
                                             (synth.LLAMA2_7B, [(64 * i + i) % 700 for i in range(70)])])
def test_append_values_slots_and_untouched_bytes(shape, positions):
    B, S, P = len(positions), shape.S, shape.page_size
    seqlens = [p + S for p in positions]
    dc = synth.make_decode_case(shape, seqlens, 12)
    ac = synth.make_append_case(shape, positions, 13)
    x = ac['x']
    params = binding.make_params(shape, B, dc['cache'].shape[0], dc['page_table'].shape[1], 1.0, num_partitions=1)
    cache0 = dc['cache'].clone()
    cache = dc['cache'].cuda()
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    binding.transmla_latent_append(params, x.cuda(), ac['w_dkv_kr'].cuda(), ac['positions'].cuda(),
                                   dc['page_table'].cuda(), cache, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = cache.cpu()
    want = lifts.f64(cache0)
    touched = torch.zeros(cache0.shape[:2], dtype=torch.bool)
    for s in range(S):
        pos = [p + s for p in positions]
        orc.latent_append(lifts.f64(x[:, s]), lifts.f64(ac['w_dkv_kr']), pos, dc['page_table'].numpy(), want, shape.r,
                          page_size=P)
        for b in range(B):
            pg, off = orc.append_slot(dc['page_table'][b].numpy(), pos[b], P)       # slot: bit-exact index path
            touched[pg, off] = True
    g64 = lifts.f64(got)
    t = touched.numpy()
    assert np.all(np.abs(g64[t] - want[t]) <= 2.0 ** -7 * np.abs(want[t]) + 1e-3)
    assert torch.equal(got.view(torch.int16)[~touched], cache0.view(torch.int16)[~touched])   # nothing else changed


# ------------------------------------------------------------------ whole step from host buffers
@pytest.mark.parametrize('pinned', [True, False])
def test_decode_step_from_host_buffers(pinned):
    shape = synth.LLAMA2_7B
    seqlens = [300, 65, 1024]
    B = len(seqlens)
    scale = gu.mla_scale(shape)
    dc = synth.make_decode_case(shape, seqlens, 15)
    ac = synth.make_append_case(shape, [L - 1 for L in seqlens], 16)
    params = binding.make_params(shape, B, dc['cache'].shape[0], dc['page_table'].shape[1], scale)
    ws, _ = binding.alloc_workspace(params)
    staging = torch.empty(binding.transmla_step_staging_bytes(params), dtype=torch.uint8, device='cuda')
    # pinned arrays go through the library's transfer kernels, pageable ones through cudaMemcpyAsync
    pin = (lambda t: t.contiguous().pin_memory()) if pinned else (lambda t: t.contiguous().clone())
    h_out = pin(torch.empty(B, 1, shape.H, shape.dv, dtype=torch.bfloat16))
    h_lse = pin(torch.empty(B, 1, shape.H, dtype=torch.float32))
    cache = dc['cache'].cuda()
    word = binding.transmla_decode_step_host(params, pin(ac['x']), pin(dc['q_nope']), pin(dc['q_pe']),
                                             pin(dc['page_table']), pin(dc['seqlens']), ac['w_dkv_kr'].cuda(),
                                             dc['w_uk'].cuda(), dc['w_uv'].cuda(), cache, staging, ws, h_out, h_lse)
    assert word == 0
    # oracle: append in fp64, round the new rows to bf16 as the cache stores them, then decode
    want_cache = lifts.f64(dc['cache'])
    orc.latent_append(lifts.f64(ac['x'][:, 0]), lifts.f64(ac['w_dkv_kr']), [L - 1 for L in seqlens], dc['page_table'].numpy(),
                      want_cache, shape.r)
    case = dict(dc)
    case['cache'] = torch.tensor(want_cache).to(torch.bfloat16)
    want, want_lse = gu.oracle_decode(shape, case, scale)
    gu.assert_close(lifts.f64(h_out), want, 'host step')
    gu.assert_lse_close(lifts.f64(h_lse), want_lse, 'host step lse')


def test_host_step_repeated_with_new_contents_in_the_same_buffers():
    # three consecutive steps through the same pinned buffers, staging and workspace: every call must read the
    # buffers' current contents (new queries, a new token, sequences one token longer)
    shape = synth.LLAMA2_7B
    B = 2
    scale = gu.mla_scale(shape)
    dc = synth.make_decode_case(shape, [300, 129], 25, extra_pages=2)
    params = binding.make_params(shape, B, dc['cache'].shape[0], dc['page_table'].shape[1], scale)
    ws, _ = binding.alloc_workspace(params)
    staging = torch.empty(binding.transmla_step_staging_bytes(params), dtype=torch.uint8, device='cuda')
    pin = lambda t: t.contiguous().pin_memory()
    h = {k: pin(dc[k]) for k in ('q_nope', 'q_pe', 'page_table', 'seqlens')}
    h_x = pin(torch.empty(B, 1, shape.D, dtype=torch.bfloat16))
    h_out = pin(torch.empty(B, 1, shape.H, shape.dv, dtype=torch.bfloat16))
    cache = dc['cache'].cuda()
    want_cache = lifts.f64(dc['cache'])
    w = synth.make_append_case(shape, [0, 0], 26)['w_dkv_kr']
    w_dev, w_uk, w_uv = w.cuda(), dc['w_uk'].cuda(), dc['w_uv'].cuda()
    seqlens = [300, 129]
    for it in range(3):
        ac = synth.make_append_case(shape, [L - 1 for L in seqlens], 30 + it)
        qn = synth.make_decode_case(shape, seqlens, 40 + it)
        h_x.copy_(ac['x']); h['q_nope'].copy_(qn['q_nope']); h['q_pe'].copy_(qn['q_pe'])
        h['seqlens'].copy_(torch.tensor(seqlens, dtype=torch.int32))
        word = binding.transmla_decode_step_host(params, h_x, h['q_nope'], h['q_pe'], h['page_table'], h['seqlens'], w_dev,
                                                 w_uk, w_uv, cache, staging, ws, h_out)
        assert word == 0
        orc.latent_append(lifts.f64(ac['x'][:, 0]), lifts.f64(w), [L - 1 for L in seqlens], dc['page_table'].numpy(),
                          want_cache, shape.r)
        want_cache = lifts.f64(torch.tensor(want_cache).to(torch.bfloat16))
        case = dict(dc, q_nope=qn['q_nope'], q_pe=qn['q_pe'], cache=torch.tensor(want_cache).to(torch.bfloat16),
                    seqlens=torch.tensor(seqlens, dtype=torch.int32))
        want, _ = gu.oracle_decode(shape, case, scale)
        gu.assert_close(lifts.f64(h_out), want, f'repeated host step {it}')
        seqlens = [L + 1 for L in seqlens]


# ------------------------------------------------------------------ whole layer: queries, attention, W_O
@pytest.mark.parametrize('shape,seqlens,rq', [(synth.TINY, [17, 64, 130], 0), (synth.TINY, [5, 70], 256),
                                               (synth.LLAMA2_7B, [300, 65, 1024], 0), (synth.LLAMA2_7B, [200, 64], 512),
                                               (synth.QWEN25_72B, [131, 700], 0),
                                               # 48 and more new tokens: the large maps run on the tcgen05 kernel
                                               (synth.LLAMA2_7B, [70 + 3 * i for i in range(50)], 0),
                                               (synth.LLAMA2_7B, [64 + i for i in range(130)], 512),
                                               (synth.QWEN25_72B, [66 + 5 * i for i in range(25)], 0),
                                               # more than 256 tokens: two token blocks per tile, the second nearly empty
                                               (synth.LLAMA2_7B, [64 + (i % 7) for i in range(259)], 0)])
def test_layer_decode_step(shape, seqlens, rq):
    B, S = len(seqlens), shape.S
    scale = gu.mla_scale(shape)
    dc = synth.make_decode_case(shape, seqlens, 31)
    ac = synth.make_append_case(shape, [L - S for L in seqlens], 32)
    lw = synth.make_layer_weights(shape, 33, q_lora_rank=rq)
    weights = {k: v.cuda() for k, v in lw.items()}
    weights.update(w_dkv_kr=ac['w_dkv_kr'].cuda(), w_uk=dc['w_uk'].cuda(), w_uv=dc['w_uv'].cuda())
    params = binding.make_params(shape, B, dc['cache'].shape[0], dc['page_table'].shape[1], scale)
    ws, _ = binding.alloc_workspace(params)
    scratch = torch.empty(binding.transmla_layer_scratch_bytes(params, rq), dtype=torch.uint8, device='cuda')
    y = torch.full((B, S, shape.D), float('nan'), dtype=torch.bfloat16, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    cache = dc['cache'].cuda()
    binding.transmla_layer_decode_step(params, weights, ac['x'].cuda(), dc['page_table'].cuda(), dc['seqlens'].cuda(), cache,
                                       ws, scratch, y, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = orc.mla_layer_decode(lifts.f64(ac['x']), lifts.f64(lw['w_uq']), lifts.f64(lw['w_qr']), lifts.f64(ac['w_dkv_kr']),
                                lifts.f64(dc['w_uk']), lifts.f64(dc['w_uv']), lifts.f64(lw['w_o']), lifts.f64(dc['cache']),
                                dc['page_table'].numpy(), seqlens, scale, shape.r,
                                w_dq=None if not rq else lifts.f64(lw['w_dq']))
    err, rel = gu.assert_close(lifts.f64(y), want, f'layer output rq={rq}')


@pytest.mark.parametrize('shape,seqlens', [(synth.QWEN25_72B, [131, 700]), (synth.LLAMA2_7B, [300, 65, 1024])])
def test_layer_step_repeated_on_a_poisoned_workspace(shape, seqlens):
    """Nothing may be read before the kernel that produces it has finished.  From the second call on every kernel is
    loaded and the launches overlap as far as they can, so a load issued ahead of its dependency wait meets whatever
    the workspace held: it is filled with NaN bytes before every call, and every call must give the bits of the first
    and meet the oracle."""
    B, S = len(seqlens), shape.S
    scale = gu.mla_scale(shape)
    dc = synth.make_decode_case(shape, seqlens, 31)
    ac = synth.make_append_case(shape, [L - S for L in seqlens], 32)
    lw = synth.make_layer_weights(shape, 33)
    weights = {k: v.cuda() for k, v in lw.items()}
    weights.update(w_dkv_kr=ac['w_dkv_kr'].cuda(), w_uk=dc['w_uk'].cuda(), w_uv=dc['w_uv'].cuda())
    params = binding.make_params(shape, B, dc['cache'].shape[0], dc['page_table'].shape[1], scale)
    ws, _ = binding.alloc_workspace(params)
    x, table, lens = ac['x'].cuda(), dc['page_table'].cuda(), dc['seqlens'].cuda()
    outs = []
    for it in range(6):
        ws.fill_(0xff)
        scratch = torch.full((binding.transmla_layer_scratch_bytes(params, 0),), 0xff, dtype=torch.uint8, device='cuda')
        y = torch.full((B, S, shape.D), float('nan'), dtype=torch.bfloat16, device='cuda')
        status = torch.zeros(1, dtype=torch.int32, device='cuda')
        cache = dc['cache'].cuda()
        torch.cuda.synchronize()
        binding.transmla_layer_decode_step(params, weights, x, table, lens, cache, ws, scratch, y, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append(y.cpu())
    for it in range(1, 6):
        assert torch.equal(outs[it].view(torch.int16), outs[0].view(torch.int16)), f'call {it} differs from the first'
    want = orc.mla_layer_decode(lifts.f64(ac['x']), lifts.f64(lw['w_uq']), lifts.f64(lw['w_qr']), lifts.f64(ac['w_dkv_kr']),
                                lifts.f64(dc['w_uk']), lifts.f64(dc['w_uv']), lifts.f64(lw['w_o']), lifts.f64(dc['cache']),
                                dc['page_table'].numpy(), seqlens, scale, shape.r)
    gu.assert_close(lifts.f64(outs[0]), want, 'layer output on a poisoned workspace')


# ------------------------------------------------------------------ pages claimed at run time (G = 0, many CTAs per sequence)
@pytest.mark.parametrize('shape,seqlens', [(synth.LLAMA2_7B, [4096 + 17, 2100]), (synth.LLAMA2_7B, [8192]),
                                           (synth.LLAMA2_7B, [64 * 40, 64 * 41 + 1, 3000]),
                                           (synth.QWEN25_72B, [4000]), (synth.QWEN25_72B, [3001, 2990])])
def test_dynamic_page_claims_match_the_oracle(shape, seqlens):
    # With G = 0 and at least 8 partitions per sequence the CTAs of a sequence take its pages from a counter, so
    # the grouping of pages into partials depends on timing: what is unique is the combined result.
    scale = gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, seed=23, nan_tails=True)
    dev = gu.to_dev(case)
    only = [(b, s, h) for b in range(len(seqlens)) for s in range(shape.S) for h in (0, 5, shape.H - 1)]
    want, want_lse = gu.oracle_decode(shape, case, scale, only=only)
    idx = tuple(np.array(only).T)
    for _ in range(3):
        out, lse, status, _, lay = gu.gpu_decode(shape, dev, scale, G=0)
        assert status == 0 and lay.num_partitions >= 8 * len(seqlens)
        gu.assert_close(lifts.f64(out)[idx], want[idx], f'dynamic claims {seqlens}')
        gu.assert_lse_close(lifts.f64(lse)[idx], want_lse[idx], 'dynamic claims lse')


@pytest.mark.parametrize('G', [0, 37])
def test_many_serialized_launches_never_time_out(G):
    # Launches bracketed by events start all CTAs at once with cold instruction caches, which is when the softmax
    # warps can get a whole page ahead of the MMA warp; every bounded wait must still be satisfied.
    shape = synth.LLAMA2_7B
    seqlens = [1024] * 4
    case = gu.to_dev(synth.make_decode_case(shape, seqlens, seed=24))
    B = len(seqlens)
    params = binding.make_params(shape, B, case['cache'].shape[0], case['page_table'].shape[1], gu.mla_scale(shape),
                                 num_partitions=G)
    ws, lay = binding.alloc_workspace(params)
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.empty(B, 1, shape.H, shape.dv, dtype=torch.bfloat16, device='cuda')
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for e in evs:
        e.record()
    first = None
    for i in range(3000):
        binding.transmla_profile_decode_kernel(evs[0], evs[1])
        binding.transmla_mla_decode(params, case['q_nope'], case['q_pe'], case['w_uk'], case['cache'], case['page_table'],
                                    case['seqlens'], ws, status)
        binding.transmla_mla_combine(params, ws, case['w_uv'], out, None, status)
        if i == 0:
            first = out.clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (out.float() - first.float()).abs().max().item() <= 2e-2


def test_dynamic_claims_when_some_partitions_find_nothing_left():
    # A wide page table (capacity for 8K tokens) with short sequences: the library still picks 32+ partitions, most
    # of the ones that own a page claim three at once, so the later ones find the sequence's counter past its end
    # and must leave an empty partial (lse = -inf) that the combine skips.
    shape = synth.LLAMA2_7B
    seqlens = [640, 300, 64 * 7 + 1]
    scale = gu.mla_scale(shape)
    case = synth.make_decode_case(shape, seqlens, seed=29, nan_tails=True)
    pad = torch.full((len(seqlens), 128 - case['page_table'].shape[1]), -1, dtype=torch.int32)
    case['page_table'] = torch.cat([case['page_table'], pad], dim=1)
    dev = gu.to_dev(case)
    want, want_lse = gu.oracle_decode(shape, case, scale)
    for _ in range(3):
        out, lse, status, _, lay = gu.gpu_decode(shape, dev, scale, G=0)
        assert status == 0 and lay.num_partitions >= 8 * len(seqlens)
        gu.assert_close(lifts.f64(out), want, 'sparse dynamic claims')
        gu.assert_lse_close(lifts.f64(lse), want_lse, 'sparse dynamic claims lse')
