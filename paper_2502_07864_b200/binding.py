"""ctypes binding of libtransmla.so: argument marshalling only, same names as the C ABI.

Every computation runs in the library's CUDA kernels.  There is no CPU fallback: if the library
is missing or was not built, importing a function from here raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, 'libtransmla.so')

EXPORTS = ('transmla_workspace_layout', 'transmla_latent_append', 'transmla_mla_decode', 'transmla_mla_combine',
           'transmla_validate_tables', 'transmla_step_staging_bytes', 'transmla_decode_step_host',
           'transmla_decode_step', 'transmla_profile_decode_kernel', 'transmla_status_string',
           'transmla_static_workspace_capacity', 'transmla_mla_attention_static', 'transmla_selftest_bounded_wait',
           'transmla_layer_scratch_bytes', 'transmla_layer_decode_step', 'transmla_stream_probe', 'transmla_page_claims_at_run_time', 'transmla_latent_append_fp8',
           'transmla_mla_decode_fp8', 'transmla_prefill_scratch_bytes', 'transmla_prefill_decompress',
           'transmla_prefill_attention', 'transmla_mla_prefill', 'transmla_conv_gemm',
           'transmla_conv_rorope_scratch_bytes', 'transmla_conv_rorope_covariance', 'transmla_conv_sym_eig',
           'transmla_conv_rorope_apply', 'transmla_conv_alpha', 'transmla_conv_balance_concat',
           'transmla_conv_subspace_scratch_bytes', 'transmla_conv_top_subspace')


class Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        'hidden_dim', 'num_heads', 'q_len', 'qk_nope_dim', 'qk_rope_dim', 'v_dim', 'kv_lora_rank', 'page_size',
        'num_pages', 'max_pages_per_seq', 'batch', 'num_partitions')] + [
        ('softmax_scale', ctypes.c_float), ('rope_theta', ctypes.c_float)]


class WorkspaceLayout(ctypes.Structure):
    _fields_ = [('num_partitions', ctypes.c_int32), ('num_slots', ctypes.c_int32),
                ('q_hat_offset', ctypes.c_size_t), ('cum_pages_offset', ctypes.c_size_t),
                ('plan_offset', ctypes.c_size_t), ('partial_o_offset', ctypes.c_size_t),
                ('partial_lse_offset', ctypes.c_size_t), ('total_bytes', ctypes.c_size_t)]


class LayerWeights(ctypes.Structure):
    _fields_ = [('w_dq', ctypes.c_void_p), ('q_lora_rank', ctypes.c_int32), ('w_uq', ctypes.c_void_p),
                ('w_qr', ctypes.c_void_p), ('w_dkv_kr', ctypes.c_void_p), ('w_uk', ctypes.c_void_p),
                ('w_uv', ctypes.c_void_p), ('w_o', ctypes.c_void_p)]


class TransMLAError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f'{where}: {status_string(code)} (status {code})')


_lib = None


def lib():
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f'{_LIB_PATH} is missing: build it with `python -m paper_2502_07864_b200.build`')
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32p, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
        pp = ctypes.POINTER(Params)
        L.transmla_workspace_layout.argtypes = [pp, ctypes.POINTER(WorkspaceLayout)]
        L.transmla_latent_append.argtypes = [pp, vp, vp, i32p, i32p, vp, i32p, vp]
        L.transmla_mla_decode.argtypes = [pp, vp, vp, vp, vp, i32p, i32p, vp, sz, i32p, vp]
        L.transmla_mla_combine.argtypes = [pp, vp, sz, vp, vp, vp, i32p, vp]
        L.transmla_validate_tables.argtypes = [pp, i32p, i32p]
        L.transmla_step_staging_bytes.argtypes = [pp]
        L.transmla_step_staging_bytes.restype = sz
        L.transmla_decode_step_host.argtypes = [pp, vp, vp, vp, i32p, i32p, vp, vp, vp, vp, vp, sz, vp, sz, vp, vp,
                                                i32p, vp]
        L.transmla_decode_step.argtypes = [pp, vp, vp, vp, i32p, i32p, vp, vp, vp, vp, vp, sz, vp, vp, i32p, vp]
        L.transmla_profile_decode_kernel.argtypes = [vp, vp]
        L.transmla_profile_decode_kernel.restype = None
        L.transmla_static_workspace_capacity.argtypes = []
        L.transmla_static_workspace_capacity.restype = sz
        L.transmla_mla_attention_static.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, vp, vp, i32p, vp]
        L.transmla_selftest_bounded_wait.argtypes = [i32p, vp, vp]
        L.transmla_stream_probe.argtypes = [pp, vp, i32p, vp, sz, i32p, vp]
        L.transmla_page_claims_at_run_time.argtypes = [pp]
        L.transmla_latent_append_fp8.argtypes = [pp, vp, vp, i32p, i32p, vp, vp, sz, i32p, vp]
        L.transmla_mla_decode_fp8.argtypes = [pp, vp, vp, vp, vp, i32p, i32p, vp, sz, i32p, vp]
        L.transmla_prefill_scratch_bytes.argtypes = [pp]
        L.transmla_prefill_scratch_bytes.restype = sz
        L.transmla_prefill_decompress.argtypes = [pp, vp, i32p, i32p, vp, vp, vp, sz, i32p, vp]
        L.transmla_prefill_attention.argtypes = [pp, vp, vp, vp, vp, sz, i32p, i32p, vp, vp, i32p, vp]
        L.transmla_mla_prefill.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, vp, sz, vp, vp, i32p, vp]
        ci, cf = ctypes.c_int, ctypes.c_float
        L.transmla_conv_gemm.argtypes = [ci, ci, ci, ci, ci, cf, vp, ci, vp, ci, vp, ci, vp]
        L.transmla_conv_rorope_scratch_bytes.argtypes = [ci, ci, ci, ci]
        L.transmla_conv_rorope_scratch_bytes.restype = sz
        L.transmla_conv_rorope_covariance.argtypes = [vp, ci, ci, ci, ci, vp, sz, vp, vp]
        L.transmla_conv_sym_eig.argtypes = [vp, ci, ci, vp, vp, i32p, vp]
        L.transmla_conv_rorope_apply.argtypes = [vp, ci, vp, ci, ci, ci, vp, vp]
        L.transmla_conv_alpha.argtypes = [vp, ci, ci, vp, ci, vp, vp, vp]
        L.transmla_conv_balance_concat.argtypes = [vp, ci, ci, vp, ci, vp, vp, vp]
        L.transmla_conv_subspace_scratch_bytes.argtypes = [ci, ci]
        L.transmla_conv_subspace_scratch_bytes.restype = sz
        L.transmla_conv_top_subspace.argtypes = [vp, ci, ci, ci, vp, vp, sz, i32p, vp]
        L.transmla_layer_scratch_bytes.argtypes = [pp, ctypes.c_int32]
        L.transmla_layer_scratch_bytes.restype = sz
        L.transmla_layer_decode_step.argtypes = [pp, ctypes.POINTER(LayerWeights), vp, i32p, i32p, vp, vp, sz, vp, sz, vp,
                                                 i32p, vp]
        L.transmla_status_string.argtypes = [ctypes.c_int]
        L.transmla_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ('transmla_step_staging_bytes', 'transmla_status_string',
                            'transmla_profile_decode_kernel', 'transmla_static_workspace_capacity',
                            'transmla_layer_scratch_bytes', 'transmla_prefill_scratch_bytes',
                            'transmla_conv_rorope_scratch_bytes', 'transmla_conv_subspace_scratch_bytes'):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code):
    return lib().transmla_status_string(int(code)).decode()


def make_params(shape, batch, num_pages, max_pages_per_seq, softmax_scale, num_partitions=0, rope_theta=10000.0):
    """Params from an MLAShape-like object (attributes H, S, dn, dR, dv, r, D, page_size)."""
    return Params(hidden_dim=shape.D, num_heads=shape.H, q_len=shape.S, qk_nope_dim=shape.dn,
                  qk_rope_dim=shape.dR, v_dim=shape.dv, kv_lora_rank=shape.r, page_size=shape.page_size,
                  num_pages=num_pages, max_pages_per_seq=max_pages_per_seq, batch=batch,
                  num_partitions=num_partitions, softmax_scale=softmax_scale, rope_theta=rope_theta)


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(code, where):
    if code != 0:
        raise TransMLAError(code, where)


def transmla_workspace_layout(params):
    lay = WorkspaceLayout()
    _check(lib().transmla_workspace_layout(ctypes.byref(params), ctypes.byref(lay)), 'transmla_workspace_layout')
    return lay


def transmla_latent_append(params, x, w_dkv_kr, positions, page_table, cache, dev_status=None, stream=None):
    _check(lib().transmla_latent_append(ctypes.byref(params), _ptr(x), _ptr(w_dkv_kr), _ptr(positions),
                                        _ptr(page_table), _ptr(cache), _ptr(dev_status), _stream(stream)),
           'transmla_latent_append')


def transmla_mla_decode(params, q_nope, q_pe, w_uk, cache, page_table, seqlens, workspace, dev_status=None,
                        stream=None):
    _check(lib().transmla_mla_decode(ctypes.byref(params), _ptr(q_nope), _ptr(q_pe), _ptr(w_uk), _ptr(cache),
                                     _ptr(page_table), _ptr(seqlens), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
           'transmla_mla_decode')


def transmla_mla_combine(params, workspace, w_uv, out, lse_out=None, dev_status=None, stream=None):
    _check(lib().transmla_mla_combine(ctypes.byref(params), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _ptr(w_uv), _ptr(out),
                                      _ptr(lse_out), _ptr(dev_status), _stream(stream)),
           'transmla_mla_combine')


def transmla_validate_tables(params, page_table_host, seqlens_host):
    """Host tensors (int32, contiguous).  Returns the status code instead of raising."""
    return lib().transmla_validate_tables(ctypes.byref(params), _ptr(page_table_host), _ptr(seqlens_host))


def transmla_step_staging_bytes(params):
    return lib().transmla_step_staging_bytes(ctypes.byref(params))


def transmla_decode_step_host(params, h_x, h_q_nope, h_q_pe, h_page_table, h_seqlens, w_dkv_kr, w_uk, w_uv, cache,
                              staging, workspace, h_out, h_lse=None, stream=None):
    """Returns the device status word."""
    word = ctypes.c_int32(0)
    _check(lib().transmla_decode_step_host(
        ctypes.byref(params), _ptr(h_x), _ptr(h_q_nope), _ptr(h_q_pe), _ptr(h_page_table), _ptr(h_seqlens),
        _ptr(w_dkv_kr), _ptr(w_uk), _ptr(w_uv), _ptr(cache), _ptr(staging),
        staging.numel() * staging.element_size(), _ptr(workspace), workspace.numel() * workspace.element_size(),
        _ptr(h_out), _ptr(h_lse), ctypes.cast(ctypes.byref(word), ctypes.c_void_p), _stream(stream)),
        'transmla_decode_step_host')
    return word.value


def transmla_decode_step(params, x, q_nope, q_pe, page_table, seqlens, w_dkv_kr, w_uk, w_uv, cache,
                         workspace, out, lse_out=None, dev_status=None, stream=None):
    _check(lib().transmla_decode_step(
        ctypes.byref(params), _ptr(x), _ptr(q_nope), _ptr(q_pe), _ptr(page_table), _ptr(seqlens), _ptr(w_dkv_kr),
        _ptr(w_uk), _ptr(w_uv), _ptr(cache), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(out), _ptr(lse_out), _ptr(dev_status), _stream(stream)),
        'transmla_decode_step')


def transmla_static_workspace_capacity():
    return lib().transmla_static_workspace_capacity()


def transmla_mla_attention_static(params, q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, out, lse_out=None,
                                  dev_status=None, stream=None):
    """Decode + combine on the library's built-in workspace; no device buffer is created here or in the library."""
    _check(lib().transmla_mla_attention_static(
        ctypes.byref(params), _ptr(q_nope), _ptr(q_pe), _ptr(w_uk), _ptr(w_uv), _ptr(cache), _ptr(page_table),
        _ptr(seqlens), _ptr(out), _ptr(lse_out), _ptr(dev_status), _stream(stream)), 'transmla_mla_attention_static')


def transmla_layer_scratch_bytes(params, q_lora_rank=0):
    return lib().transmla_layer_scratch_bytes(ctypes.byref(params), int(q_lora_rank))


def transmla_layer_decode_step(params, weights, x, page_table, seqlens, cache, workspace, scratch, y, dev_status=None,
                               stream=None):
    """weights: dict of device tensors w_uq, w_qr, w_dkv_kr, w_uk, w_uv, w_o and optionally w_dq (low-rank queries)."""
    w_dq = weights.get('w_dq')
    lw = LayerWeights(w_dq=None if w_dq is None else w_dq.data_ptr(), q_lora_rank=0 if w_dq is None else w_dq.shape[0],
                      w_uq=weights['w_uq'].data_ptr(), w_qr=None if weights.get('w_qr') is None else weights['w_qr'].data_ptr(),
                      w_dkv_kr=weights['w_dkv_kr'].data_ptr(), w_uk=weights['w_uk'].data_ptr(),
                      w_uv=weights['w_uv'].data_ptr(), w_o=weights['w_o'].data_ptr())
    _check(lib().transmla_layer_decode_step(
        ctypes.byref(params), ctypes.byref(lw), _ptr(x), _ptr(page_table), _ptr(seqlens), _ptr(cache), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(scratch), scratch.numel() * scratch.element_size(), _ptr(y),
        _ptr(dev_status), _stream(stream)), 'transmla_layer_decode_step')


def transmla_selftest_bounded_wait(dev_status, cycles_out=None, stream=None):
    _check(lib().transmla_selftest_bounded_wait(_ptr(dev_status), _ptr(cycles_out), _stream(stream)),
           'transmla_selftest_bounded_wait')


FP8_ROW_BYTES = 656


def transmla_latent_append_fp8(params, x, w_dkv_kr, positions, page_table, cache_fp8, scratch, dev_status=None, stream=None):
    _check(lib().transmla_latent_append_fp8(ctypes.byref(params), _ptr(x), _ptr(w_dkv_kr), _ptr(positions), _ptr(page_table),
                                            _ptr(cache_fp8), _ptr(scratch), scratch.numel() * scratch.element_size(),
                                            _ptr(dev_status), _stream(stream)), 'transmla_latent_append_fp8')


def transmla_mla_decode_fp8(params, q_nope, q_pe, w_uk, cache_fp8, page_table, seqlens, workspace, dev_status=None,
                            stream=None):
    _check(lib().transmla_mla_decode_fp8(ctypes.byref(params), _ptr(q_nope), _ptr(q_pe), _ptr(w_uk), _ptr(cache_fp8),
                                         _ptr(page_table), _ptr(seqlens), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
           'transmla_mla_decode_fp8')


def transmla_prefill_scratch_bytes(params):
    return int(lib().transmla_prefill_scratch_bytes(ctypes.byref(params)))


def _nbytes(t):
    return t.numel() * t.element_size()


def transmla_prefill_decompress(params, cache, page_table, seqlens, w_uk, w_uv, scratch, dev_status=None, stream=None):
    _check(lib().transmla_prefill_decompress(ctypes.byref(params), _ptr(cache), _ptr(page_table), _ptr(seqlens), _ptr(w_uk),
                                             _ptr(w_uv), _ptr(scratch), _nbytes(scratch), _ptr(dev_status), _stream(stream)),
           'transmla_prefill_decompress')


def transmla_prefill_attention(params, q_nope, q_pe, cache, scratch, page_table, seqlens, out, lse=None, dev_status=None,
                               stream=None):
    _check(lib().transmla_prefill_attention(ctypes.byref(params), _ptr(q_nope), _ptr(q_pe), _ptr(cache), _ptr(scratch),
                                            _nbytes(scratch), _ptr(page_table), _ptr(seqlens), _ptr(out), _ptr(lse),
                                            _ptr(dev_status), _stream(stream)),
           'transmla_prefill_attention')


def transmla_mla_prefill(params, q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, scratch, out, lse=None,
                         dev_status=None, stream=None):
    _check(lib().transmla_mla_prefill(ctypes.byref(params), _ptr(q_nope), _ptr(q_pe), _ptr(w_uk), _ptr(w_uv), _ptr(cache),
                                      _ptr(page_table), _ptr(seqlens), _ptr(scratch), _nbytes(scratch), _ptr(out), _ptr(lse),
                                      _ptr(dev_status), _stream(stream)),
           'transmla_mla_prefill')


# ---- conversion calls: fp32 device tensors, row-major and contiguous
def transmla_conv_gemm(a, b, c, ta=False, tb=False, alpha=1.0, stream=None):
    """c[M,N] = alpha * op(a) op(b); shapes are taken from the tensors."""
    M, N = c.shape
    K = a.shape[0] if ta else a.shape[1]
    _check(lib().transmla_conv_gemm(int(ta), int(tb), M, N, K, float(alpha), _ptr(a), a.shape[1], _ptr(b), b.shape[1],
                                    _ptr(c), c.shape[1], _stream(stream)), 'transmla_conv_gemm')


def transmla_conv_rorope_covariance(k_act, g, d, fold, scratch, cov, stream=None):
    _check(lib().transmla_conv_rorope_covariance(_ptr(k_act), k_act.shape[0], g, d, fold, _ptr(scratch), _nbytes(scratch),
                                                 _ptr(cov), _stream(stream)), 'transmla_conv_rorope_covariance')


def transmla_conv_rorope_scratch_bytes(n, g, d, fold):
    return int(lib().transmla_conv_rorope_scratch_bytes(n, g, d, fold))


def transmla_conv_sym_eig(a, eigvals, eigvecs, dev_status=None, stream=None):
    batch, m, _ = a.shape
    _check(lib().transmla_conv_sym_eig(_ptr(a), batch, m, _ptr(eigvals), _ptr(eigvecs), _ptr(dev_status), _stream(stream)),
           'transmla_conv_sym_eig')


def transmla_conv_rorope_apply(x, u, g, d, fold, y, stream=None):
    _check(lib().transmla_conv_rorope_apply(_ptr(x), x.shape[1], _ptr(u), g, d, fold, _ptr(y), _stream(stream)),
           'transmla_conv_rorope_apply')


def transmla_conv_alpha(k_nope, v, scratch, alpha_out, stream=None):
    _check(lib().transmla_conv_alpha(_ptr(k_nope), k_nope.shape[0], k_nope.shape[1], _ptr(v), v.shape[1], _ptr(scratch),
                                     _ptr(alpha_out), _stream(stream)), 'transmla_conv_alpha')


def transmla_conv_balance_concat(k_nope, v, alpha, z, stream=None):
    _check(lib().transmla_conv_balance_concat(_ptr(k_nope), k_nope.shape[0], k_nope.shape[1], _ptr(v), v.shape[1], _ptr(alpha),
                                              _ptr(z), _stream(stream)), 'transmla_conv_balance_concat')


def transmla_conv_subspace_scratch_bytes(m, r):
    return int(lib().transmla_conv_subspace_scratch_bytes(m, r))


def transmla_conv_top_subspace(cmat, q, iters, scratch, dev_status=None, stream=None):
    m, r = q.shape
    _check(lib().transmla_conv_top_subspace(_ptr(cmat), m, r, iters, _ptr(q), _ptr(scratch), _nbytes(scratch), _ptr(dev_status),
                                            _stream(stream)), 'transmla_conv_top_subspace')


def transmla_page_claims_at_run_time(params):
    return bool(lib().transmla_page_claims_at_run_time(ctypes.byref(params)))


def transmla_stream_probe(params, cache, page_table, workspace, dev_status=None, stream=None):
    """Streams the pages of the split plan left in `workspace` by a preceding transmla_mla_decode and discards them."""
    _check(lib().transmla_stream_probe(ctypes.byref(params), _ptr(cache), _ptr(page_table), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(dev_status), _stream(stream)),
           'transmla_stream_probe')


def transmla_profile_decode_kernel(start_event, stop_event):
    """torch.cuda.Event objects (timing enabled, already created by a record) or None, None."""
    a = ctypes.c_void_p(0 if start_event is None else start_event.cuda_event)
    b = ctypes.c_void_p(0 if stop_event is None else stop_event.cuda_event)
    lib().transmla_profile_decode_kernel(a, b)


# -------- conveniences built only from the calls above (device-memory plumbing, no arithmetic)
def alloc_workspace(params, device='cuda'):
    lay = transmla_workspace_layout(params)
    return torch.empty(lay.total_bytes, dtype=torch.uint8, device=device), lay


def workspace_views(params, workspace, lay=None):
    """Typed views of the workspace regions (see transmla_workspace_layout_t)."""
    lay = lay or transmla_workspace_layout(params)
    B, SH = params.batch, params.q_len * params.num_heads
    K, r = params.kv_lora_rank + params.qk_rope_dim, params.kv_lora_rank

    def view(off, n, dtype):
        esz = torch.empty((), dtype=dtype).element_size()
        return workspace[off:off + n * esz].view(dtype)
    return {
        'q_hat': view(lay.q_hat_offset, B * SH * K, torch.bfloat16).view(B, params.q_len, params.num_heads, K),
        'cum_pages': view(lay.cum_pages_offset, B + 1, torch.int32),
        'seq_parts': view(lay.cum_pages_offset, 3 * B + 1, torch.int32)[B + 1:].view(B, 2),
        'plan': view(lay.plan_offset, lay.num_partitions * 4, torch.int32).view(lay.num_partitions, 4),
        'partial_o': view(lay.partial_o_offset, lay.num_slots * SH * r, torch.float32).view(lay.num_slots, SH, r),
        'partial_lse': view(lay.partial_lse_offset, lay.num_slots * SH, torch.float32).view(lay.num_slots, SH),
    }
