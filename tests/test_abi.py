"""CPU-only checks of the boundary: the library builds, loads, exports every declared symbol, and
its host-side argument checks answer with codes without touching a GPU."""
import ctypes
import os
import re

import torch

from paper_2502_07864_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    build.build()
    L = binding.lib()
    header = open(os.path.join(ROOT, 'include', 'transmla.h')).read()
    declared = set(re.findall(r'\b(transmla_[a-z0-9_]+)\s*\(', header))
    assert declared, 'no declarations found'
    for name in declared:
        assert hasattr(L, name), f'{name} declared in transmla.h but not exported'
    assert declared == set(binding.EXPORTS)


def test_status_strings():
    assert binding.status_string(0) == 'ok'
    assert 'workspace' in binding.status_string(5)


def test_workspace_layout_is_host_arithmetic():
    s = synth.LLAMA2_7B
    p = binding.make_params(s, batch=16, num_pages=2500, max_pages_per_seq=128, softmax_scale=0.07, num_partitions=148)
    lay = binding.transmla_workspace_layout(p)
    assert lay.num_partitions == 148 and lay.num_slots == 148 + 16 - 1
    assert lay.q_hat_offset == 0 and lay.cum_pages_offset >= 16 * 32 * 576 * 2
    assert lay.partial_lse_offset - lay.partial_o_offset >= lay.num_slots * 32 * 512 * 4
    assert lay.total_bytes >= lay.partial_lse_offset + lay.num_slots * 32 * 4
    for off in (lay.cum_pages_offset, lay.plan_offset, lay.partial_o_offset, lay.partial_lse_offset, lay.total_bytes):
        assert off % 256 == 0


def test_byte_counts_beyond_4_gib_come_back_whole():
    # host arithmetic only; the counts are size_t and must not pass through a 32-bit return type
    build.build()
    shape = synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=16)
    params = binding.make_params(shape, 16, 4096, 128, 0.07)
    assert binding.transmla_prefill_scratch_bytes(params) == 4096 * 64 * 32 * 256 * 2
    assert binding.transmla_conv_rorope_scratch_bytes(1 << 20, 32, 128, 4) == 16 * 2 * (1 << 20) * 128 * 4
    assert binding.transmla_conv_subspace_scratch_bytes(100000, 1024) > (1 << 28)
    assert binding.transmla_prefill_scratch_bytes(binding.make_params(synth.TINY, 2, 4, 2, 0.1)) == 0


def test_shape_errors_are_codes():
    s = synth.LLAMA2_7B
    lay = binding.WorkspaceLayout()
    bad = binding.make_params(s, 1, 1, 1, 0.1, num_partitions=4)
    bad.page_size = 32
    assert binding.lib().transmla_workspace_layout(ctypes.byref(bad), ctypes.byref(lay)) == 3
    bad = binding.make_params(synth.MLAShape(H=32, dn=128, dR=32, dv=128, r=512), 1, 1, 1, 0.1, num_partitions=4)
    assert binding.lib().transmla_workspace_layout(ctypes.byref(bad), ctypes.byref(lay)) == 3
    assert binding.lib().transmla_workspace_layout(None, ctypes.byref(lay)) == 1


def test_null_and_alignment_errors_come_before_any_launch():
    s = synth.TINY
    p = binding.make_params(s, 2, 4, 1, 0.1, num_partitions=2)
    L = binding.lib()
    z = ctypes.c_void_p(0)
    assert L.transmla_mla_decode(ctypes.byref(p), z, z, z, z, z, z, z, 0, z, z) == 1
    assert L.transmla_mla_combine(ctypes.byref(p), z, 0, z, z, z, z, z) == 1
    assert L.transmla_latent_append(ctypes.byref(p), z, z, z, z, z, z, z) == 1
    a = ctypes.c_void_p(4096)
    odd = ctypes.c_void_p(4096 + 8)
    assert L.transmla_mla_decode(ctypes.byref(p), odd, a, a, a, a, a, a, 1 << 30, z, z) == 2
    assert L.transmla_mla_decode(ctypes.byref(p), a, a, a, ctypes.c_void_p(4096 + 64), a, a, a, 1 << 30, z, z) == 2
    assert L.transmla_mla_decode(ctypes.byref(p), a, a, a, a, a, a, a, 16, z, z) == 5


def test_validate_tables_on_host():
    s = synth.TINY
    p = binding.make_params(s, 2, 4, 2, 0.1, num_partitions=2)
    table = torch.tensor([[3, -1], [0, 2]], dtype=torch.int32)
    assert binding.transmla_validate_tables(p, table, torch.tensor([17, 128], dtype=torch.int32)) == 0
    assert binding.transmla_validate_tables(p, table, torch.tensor([17, 129], dtype=torch.int32)) == 4
    assert binding.transmla_validate_tables(p, table, torch.tensor([65, 64], dtype=torch.int32)) == 4     # -1 used
    dup = torch.tensor([[3, -1], [3, 2]], dtype=torch.int32)
    assert binding.transmla_validate_tables(p, dup, torch.tensor([17, 128], dtype=torch.int32)) == 4
    big = torch.tensor([[4, -1], [0, 2]], dtype=torch.int32)
    assert binding.transmla_validate_tables(p, big, torch.tensor([17, 128], dtype=torch.int32)) == 4
    assert binding.transmla_validate_tables(p, table, torch.tensor([-1, 0], dtype=torch.int32)) == 4


def test_only_weights_are_declared_restrict_in_the_kernels():
    """Every kernel starts before the kernel ahead of it in the stream has finished and waits later.  A pointer
    declared const __restrict__ lets the compiler issue its loads above that wait, so only weights (which no
    kernel of the stream writes) may carry the qualifier."""
    import pathlib
    import re
    weights = {'w', 'w_uk', 'w_uv', 'w_dkv_kr', 'wrow'}
    csrc = pathlib.Path(__file__).resolve().parent.parent / 'paper_2502_07864_b200' / 'csrc'
    offenders = []
    for f in sorted(csrc.iterdir()):
        if f.suffix not in ('.cu', '.cuh'):
            continue
        for name in re.findall(r'__restrict__\s+(\w+)', f.read_text()):
            if name not in weights:
                offenders.append(f'{f.name}: {name}')
    assert not offenders, offenders
