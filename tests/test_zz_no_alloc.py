"""The workspace-free entry point against the ordinary decode + combine pair and the oracle (collected last on purpose).

transmla_mla_attention_static is for hosts that cannot give the library a device workspace (a fixed
memory budget, a callback in which allocating would stall the GPU, an allocator that is someone
else's).  It keeps its scratch in an array inside the library, so consecutive calls reuse the same
memory.  The test therefore calls it twice in a row, on different problems, and each result must
match what the caller-workspace path gives on the same inputs, and the fp64 oracle's definition
of the result, within the usual tolerances; outputs are allocated before the calls, so nothing is
allocated between or inside them.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2502_07864_b200 import binding, synth
from tests import gpu_util as gu
from tests import lifts

pytestmark = pytest.mark.gpu


def _problem(shape, seqlens, seed, G):
    case = gu.to_dev(synth.make_decode_case(shape, seqlens, seed, nan_tails=True))
    B = len(seqlens)
    scale = gu.mla_scale(shape)
    params = binding.make_params(shape, B, case['cache'].shape[0], case['page_table'].shape[1], scale, num_partitions=G)
    ref_out, ref_lse, status, _, _ = gu.gpu_decode(shape, case, scale, G=G)
    assert status == 0
    out = torch.full((B, shape.S, shape.H, shape.dv), float('nan'), dtype=torch.bfloat16, device='cuda')
    lse = torch.full((B, shape.S, shape.H), float('nan'), dtype=torch.float32, device='cuda')
    want, want_lse = gu.oracle_decode(shape, case, scale)
    return case, params, out, lse, ref_out, ref_lse, want, want_lse


def test_two_calls_in_a_row_match_the_workspace_path():
    gu.ensure_built()
    first = _problem(synth.LLAMA2_7B, [700, 64, 1300, 5], seed=41, G=0)
    second = _problem(synth.TINY, [17, 64, 300], seed=42, G=5)
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    for case, params, out, lse, *_ in (first, second):             # back to back, nothing in between
        q_pe = case['q_pe'] if params.qk_rope_dim > 0 else None
        binding.transmla_mla_attention_static(params, case['q_nope'], q_pe, case['w_uk'], case['w_uv'], case['cache'],
                                              case['page_table'], case['seqlens'], out, lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for _, _, out, lse, ref_out, ref_lse, want, want_lse in (first, second):
        gu.assert_close(lifts.f64(out), lifts.f64(ref_out), 'static workspace vs caller workspace')
        gu.assert_lse_close(lifts.f64(lse), lifts.f64(ref_lse), 'lse')
        gu.assert_close(lifts.f64(out), want, 'static workspace vs oracle')
        gu.assert_lse_close(lifts.f64(lse), want_lse, 'lse vs oracle')


def test_problem_larger_than_the_builtin_array_is_refused():
    gu.ensure_built()
    shape = synth.LLAMA2_7B
    params = binding.make_params(shape, 256, 10, 1, 0.1, num_partitions=148)
    assert binding.transmla_workspace_layout(params).total_bytes > binding.transmla_static_workspace_capacity()
    a = ctypes.c_void_p(4096)
    code = binding.lib().transmla_mla_attention_static(ctypes.byref(params), a, a, a, a, a, a, a, a, None, None, None)
    assert code == 5 and 'workspace' in binding.status_string(code)
