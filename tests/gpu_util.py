"""Helpers of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the same bytes."""
import math

import numpy as np
import torch

from oracle import mla_oracle as orc
from paper_2502_07864_b200 import binding, build
from tests import lifts

MAX_ABS = 2e-2     # bf16 storage, fp32 accumulation, against the fp64 oracle
REL_L2 = 5e-3


def ensure_built():
    build.build()
    return binding.lib()


def to_dev(case):
    return {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in case.items()}


def gpu_decode(shape, case, scale, G=0, want_views=False, fixed_plan=False):
    """decode + combine through the C ABI on device tensors.  Returns out, lse, status word, views.

    G = 0 lets the library choose the partition count; it then also hands pages to CTAs dynamically, so
    which pages end up in which partial depends on timing.  With ``fixed_plan`` the library's own count is
    passed back explicitly, which pins every partition to the page range of the plan.
    """
    B = case['seqlens'].numel()
    params = binding.make_params(shape, B, case['cache'].shape[0], case['page_table'].shape[1], scale,
                                 num_partitions=G)
    if G == 0 and fixed_plan:
        params.num_partitions = binding.transmla_workspace_layout(params).num_partitions
    ws, lay = binding.alloc_workspace(params)
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.full((B, shape.S, shape.H, shape.dv), float('nan'), dtype=torch.bfloat16, device='cuda')
    lse = torch.full((B, shape.S, shape.H), float('nan'), dtype=torch.float32, device='cuda')
    q_pe = case['q_pe'] if shape.dR > 0 else None
    binding.transmla_mla_decode(params, case['q_nope'], q_pe, case['w_uk'], case['cache'], case['page_table'],
                                case['seqlens'], ws, status)
    binding.transmla_mla_combine(params, ws, case['w_uv'], out, lse, status)
    torch.cuda.synchronize()
    views = binding.workspace_views(params, ws, lay) if want_views else None
    return out, lse, int(status.item()), views, lay


def oracle_decode(shape, case, scale, only=None):
    c = lifts.case_f64(case)
    return orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                   c['seqlens'], scale, page_size=shape.page_size, only=only)


def assert_close(got, want, what=''):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert np.all(np.isfinite(got)), f'{what}: non-finite values in the CUDA result'
    err = np.abs(got - want).max() if got.size else 0.0
    rel = lifts.rel_l2(got, want)
    assert err <= MAX_ABS, f'{what}: max-abs {err:.3e} > {MAX_ABS}'
    assert rel <= REL_L2, f'{what}: rel-L2 {rel:.3e} > {REL_L2}'
    return err, rel


def assert_lse_close(got, want, what=''):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    inf = np.isneginf(want)
    assert np.array_equal(np.isneginf(got), inf), f'{what}: -inf pattern of lse differs'
    assert np.abs(got[~inf] - want[~inf]).max(initial=0.0) <= 5e-3, f'{what}: lse differs'


def mla_scale(shape):
    return 1.0 / math.sqrt(shape.dn + shape.dR)
