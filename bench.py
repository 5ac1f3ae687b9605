#!/usr/bin/env python
"""Benchmark of the absorbed-MLA decode step (append + absorb + split-KV decode + combine).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--layer]

One step = one pass of the whole path over one batch: every sequence appends its new token's
latent and decodes over its cached tokens.  The default workload is the LLaMA-2-7B-converted
shape (32 heads, latent 512 + rope 64, nope 128, v 128) at batch 16 x 8192 cached tokens.  With N
GPUs every rank runs its own batch (sequences are independent; no collective on the data path),
so the scaling is weak.  Rank 0 prints one JSON line.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = 'absorbed-MLA decode tokens/s and latent-cache HBM GB/s (% of 8 TB/s) at batch x 8K'
NOMINAL_HBM_GBS = 8000.0
KERNELS_PER_STEP = 3      # prologue (append + absorb + plan), split-KV decode, combine


def workloads():
    from paper_2502_07864_b200 import synth
    w = {}
    for B in (1, 4, 16, 32, 64, 128):
        w[f'llama2-7b-mla_b{B}_8k'] = (synth.LLAMA2_7B, [8192] * B, 3)
    w['llama2-7b-mla_b16_8k'] = (synth.LLAMA2_7B, [8192] * 16, 2)
    w['llama2-7b-mla_ragged_b32'] = (synth.LLAMA2_7B, synth.uniform_seqlens(32, 1024, 32768, 4), 4)
    w['llama2-7b-mla_b4_128k'] = (synth.LLAMA2_7B, [131072] * 4, 4)
    w['qwen2.5-72b-mla_b64_s2'] = (synth.QWEN25_72B, synth.uniform_seqlens(64, 2048, 8192, 5), 5)
    for B in (16, 64, 128):      # the same shape over the FP8 latent cache (656 bytes a token instead of 1152)
        w[f'llama2-7b-mla-fp8_b{B}_8k'] = (synth.LLAMA2_7B, [8192] * B, 6)
    # the conversion of one layer on n = 8192 synthetic calibration tokens, LLaMA-2-7B shape (g = 32 heads of d = 128)
    w['llama2-7b_conversion_n8192'] = (synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096), [8192], 9)
    for S in (128, 512, 2048, 8192):   # prefill in the MHA form: a chunk of S query positions over 8192 cached tokens
        w[f'llama2-7b-mla_prefill_b4_8k_s{S}'] = (synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=S), [8192] * 4, 8)
        if S <= 2048:   # the headline batch; 2.6 GB of decompressed keys and values
            w[f'llama2-7b-mla_prefill_b16_8k_s{S}'] = (synth.MLAShape(H=32, dn=128, dR=64, dv=128, r=512, D=4096, S=S), [8192] * 16, 8)
    return w


def measured_hbm_peak():
    path = os.path.join(ROOT, 'MEASURED_PEAKS.json')
    try:
        return float(json.load(open(path))['hbm_gbs']), 'measured'
    except Exception:
        return 6650.0, 'fallback'


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a GEMM timed alone (the split-KV kernel is timed alone too)."""
    path = os.path.join(ROOT, 'MEASURED_PEAKS.json')
    try:
        return float(json.load(open(path))['bf16_tflops']), 'measured'
    except Exception:
        return 1590.0, 'fallback'


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ('clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,'
              'clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap')

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(['nvidia-smi', f'--query-gpu={self.FIELDS}', '--format=csv,noheader,nounits',
                                          '-i', str(index), '-lms', '20'], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(',')]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {'sm_mhz': None, 'sm_max_mhz': None, 'reasons': ['nvidia-smi unavailable']}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.15] or [r for (_, r) in self.rows[-3:]]
        sm, mx, reasons = [], None, set()
        for r in rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except Exception:
                continue
            for name, v in zip(('hw_slowdown', 'hw_thermal_slowdown', 'sw_thermal_slowdown', 'sw_power_cap'), r[2:6]):
                if v.lower().startswith('active'):
                    reasons.add(name)
        return {'sm_mhz': statistics.median(sm) if sm else None, 'sm_max_mhz': mx, 'reasons': sorted(reasons),
                'samples': len(sm)}


def oracle_sample(shape, seqlens, seed, n_seq):
    """Inputs of the first n_seq sequences of the workload, on the CPU, as float64 numpy."""
    import torch
    from paper_2502_07864_b200 import synth
    case = synth.make_decode_case(shape, seqlens[:n_seq], seed, device='cpu')
    return {k: (v.to(torch.float64).numpy() if v.is_floating_point() else v.numpy()) for k, v in case.items()}


def time_oracle(shape, c, scale):
    from oracle import mla_oracle as orc
    t0 = time.perf_counter()
    orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'], c['seqlens'],
                            scale, page_size=shape.page_size)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p['num_threads'] for p in threadpool_info() if p.get('user_api') == 'blas']
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def cpu_baseline(shape, seqlens, seed, scale, budget_s=15.0):
    """The fp64 oracle, as it stands, on a bounded sample: whole sequences of the workload, all heads."""
    c1 = oracle_sample(shape, seqlens, seed, 1)
    t1 = time_oracle(shape, c1, scale)
    n = int(max(1, min(len(seqlens), budget_s // max(t1, 1e-3))))
    if n > 1:
        c = oracle_sample(shape, seqlens, seed, n)
        t = time_oracle(shape, c, scale)
    else:
        t = t1
    return {'value': n * shape.S / t, 'unit': 'tokens/s', 'cores': blas_threads(), 'kind': 'oracle',
            'sample': f'first {n} of {len(seqlens)} sequences, all {shape.H} heads, all cached tokens; {t:.1f} s'}


def run_reference(args, name, shape, seqlens, seed):
    """The oracle as the reference arm: every step decodes a bounded sample of the workload on the host.

    The sample is the first sequence of the workload, all its cached tokens, and as many heads as fit
    a per-step time budget chosen so that the whole run ends within a few minutes; a step that does
    n of the H heads of one token counts as n/H tokens.
    """
    rank = int(os.environ.get('RANK', '0'))
    if rank != 0:
        return
    from oracle import mla_oracle as orc
    scale = (shape.dn + shape.dR) ** -0.5
    c = oracle_sample(shape, seqlens, seed, 1)

    def run(only):
        t0 = time.perf_counter()
        orc.mla_decode_mha_form(c['q_nope'], c['q_pe'], c['w_uk'], c['w_uv'], c['cache'], c['page_table'],
                                c['seqlens'], scale, page_size=shape.page_size, only=only)
        return time.perf_counter() - t0
    run([(0, 0, 0)])
    t_head = run([(0, 0, 0)])
    budget = min(1.0, 150.0 / max(args.steps + args.warmup, 1))
    n_heads = int(max(1, min(shape.H, budget // max(t_head, 1e-4))))
    only = [(0, s, h) for s in range(shape.S) for h in range(n_heads)]
    for _ in range(args.warmup):
        run(only)
    t = sum(run(only) for _ in range(args.steps))
    tokens_per_step = shape.S * n_heads / shape.H
    value = args.steps * tokens_per_step / t
    sample = f'1 of {len(seqlens)} sequences ({seqlens[0]} cached tokens), {n_heads} of {shape.H} heads per step'
    print(json.dumps({
        'impl': 'reference', 'metric': METRIC, 'value': value, 'unit': 'tokens/s', 'n_gpus': args.gpus,
        'steps': args.steps, 'warmup': args.warmup, 'ms_per_step': 1e3 * t / args.steps, 'higher_is_better': True,
        'scaling': 'weak', 'vs_baseline': None, 'dtype': 'f64', 'data': 'synthetic',
        'config': {'workload': name, 'sample': sample},
        'cpu_baseline': {'value': value, 'unit': 'tokens/s', 'cores': blas_threads(), 'kind': 'oracle', 'sample': sample},
        'e2e': {'value': value, 'unit': 'tokens/s', 'h2d_bytes_per_step': 0, 'd2h_bytes_per_step': 0},
    }))


def kernel_source_hash(fp8=False):
    """Hash of the sources the split-KV kernel is compiled from; ties an ncu capture to the code it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for f in ('decode_fp8.cu' if fp8 else 'decode_sm100.cu', 'common.cuh', 'sm100_ptx.cuh'):
        h.update(open(os.path.join(ROOT, 'paper_2502_07864_b200', 'csrc', f), 'rb').read())
    return h.hexdigest()[:16]


def traffic_from_profile(name):
    """dram__bytes_read.sum + dram__bytes_write.sum of one split-KV launch, from the ncu summary under profiles/ for
    this workload; None when there is none or when the kernel's sources have changed since the capture."""
    fp8 = '-fp8' in name
    kernel = 'decode_fp8' if fp8 else 'decode_sm100'
    path = os.path.join(ROOT, 'profiles', f'{kernel}_{name.replace("-mla", "").replace("-fp8", "")}.md')
    try:
        text = open(path).read()
    except OSError:
        return None
    vals = {}
    for line in text.splitlines():
        if line.startswith('traffic_bytes_per_launch:') or line.startswith('kernel_source_hash:'):
            k, v = line.split(':', 1)
            vals[k] = v.strip()
    if vals.get('kernel_source_hash') != kernel_source_hash(fp8) or 'traffic_bytes_per_launch' not in vals:
        return None
    return float(vals['traffic_bytes_per_launch'])


def run_ours(args, name, shape, seqlens, seed):
    import torch
    import torch.distributed as dist
    from paper_2502_07864_b200 import binding, build, replicas

    rank = int(os.environ.get('RANK', '0'))
    world = int(os.environ.get('WORLD_SIZE', '1'))
    local = int(os.environ.get('LOCAL_RANK', '0'))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group('nccl', device_id=torch.device('cuda', local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.lib()          # raises if the CUDA library is missing: there is no other path

    line = measure(args, name, shape, seqlens, seed, rank, world, local, full=True)
    if rank == 0:
        if world == 1 and args.sweep:
            # the other rows of the target range, each measured the same way (shorter), so that one run shows them all
            line['sweep'] = []
            for other in args.sweep.split(','):
                if other and other != name:
                    sh, sl, sd = workloads()[other]
                    row = measure(args, other, sh, sl, sd, rank, world, local, full=False)
                    keep = ('config', 'ms_per_step', 'value', 'decode_kernel_us', 'cache_gbs_pct_of_8tbs', 'roofline', 'clocks')
                    if 'prefill' in row:   # a prefill row carries its own metric and the two kernels' figures
                        keep += ('metric', 'unit', 'prefill')
                    if 'conversion_ms' in row:
                        keep += ('metric', 'unit', 'conversion_ms')
                    line['sweep'].append({k: row[k] for k in keep})
        if world == 1 and not args.no_cpu_baseline:
            line['cpu_baseline'] = cpu_baseline(shape, seqlens, seed, (shape.dn + shape.dR) ** -0.5)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_prefill(args, name, shape, seqlens, seed, rank, world, local):
    """A prefill workload: one step = decompress the cached tokens (Eq. 8) + causal attention of the chunk (Eq. 9
    left), two launches.  Both are dense contractions: the roofline is the measured bf16 GEMM rate."""
    import torch
    from paper_2502_07864_b200 import binding, replicas, synth
    B, S, H = len(seqlens), shape.S, shape.H
    stream = torch.cuda.current_stream()
    n_copies = 2
    case = synth.make_decode_case(shape, seqlens, seed, device='cuda')
    caches = [case['cache']] + [case['cache'].clone() for _ in range(n_copies - 1)]
    params = binding.make_params(shape, B, case['cache'].shape[0], case['page_table'].shape[1], (shape.dn + shape.dR) ** -0.5)
    scratch = torch.empty(binding.transmla_prefill_scratch_bytes(params) // 2, dtype=torch.bfloat16, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    out = torch.empty(B, S, H, shape.dv, dtype=torch.bfloat16, device='cuda')
    lse = torch.empty(B, S, H, dtype=torch.float32, device='cuda')
    steps = max(3, min(args.steps, 20))

    def step(i):
        binding.transmla_mla_prefill(params, case['q_nope'], case['q_pe'], case['w_uk'], case['w_uv'], caches[i % n_copies],
                                     case['page_table'], case['seqlens'], scratch, out, lse, status, stream)

    for i in range(3):
        step(i)
    replicas.barrier('cuda')
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    t0 = time.perf_counter()
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    replicas.barrier('cuda')
    t1 = time.perf_counter()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None
    parts = {'decompress': [], 'attention': []}
    for i in range(5):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record(stream)
        binding.transmla_prefill_decompress(params, caches[i % n_copies], case['page_table'], case['seqlens'], case['w_uk'],
                                            case['w_uv'], scratch, status, stream)
        ev[1].record(stream)
        binding.transmla_prefill_attention(params, case['q_nope'], case['q_pe'], caches[i % n_copies], scratch,
                                           case['page_table'], case['seqlens'], out, lse, status, stream)
        ev[2].record(stream)
        torch.cuda.synchronize()
        parts['decompress'].append(ev[0].elapsed_time(ev[1]))
        parts['attention'].append(ev[1].elapsed_time(ev[2]))
    assert int(status.item()) == 0
    (ms_total,) = replicas.max_over_ranks([ms_total], device='cuda')
    if rank != 0:
        return None
    dec_ms, att_ms = statistics.median(parts['decompress']), statistics.median(parts['attention'])
    f_dec = 2.0 * shape.r * H * (shape.dn + shape.dv) * sum(seqlens)
    vis = sum(max(0, L - (S - 1 - s)) for L in seqlens for s in range(S))        # visible (query, token) pairs per head
    f_att = 2.0 * (shape.dn + shape.dR + shape.dv) * H * vis
    tpeak, tpeak_kind = measured_tensor_peak()
    top, top_ms, top_f = ('prefill attention', att_ms, f_att) if att_ms >= dec_ms else ('prefill decompress', dec_ms, f_dec)
    ms_step = ms_total / steps
    return {
        'metric': 'MHA-form prefill tokens/s (chunk of S query positions per sequence over the paged latent cache)',
        'value': replicas.whole_job_rate(B * S, steps, ms_total), 'unit': 'tokens/s', 'n_gpus': world, 'steps': steps, 'warmup': 3,
        'ms_per_step': ms_step, 'higher_is_better': True, 'scaling': 'weak', 'vs_baseline': None, 'dtype': 'bf16',
        'data': 'synthetic',
        'config': {'workload': name, 'batch_per_gpu': B, 'q_len': S, 'heads': H, 'latent': shape.r, 'rope': shape.dR,
                   'cached_tokens_per_gpu': sum(seqlens), 'page_size': shape.page_size,
                   'l2': f'inputs larger than L2: decompressed store {scratch.numel() * 2 / 1e6:.0f} MB, cache rotates over '
                         f'{n_copies} copies', 'parallelism': f'replicas x{world}, no data-path collective'},
        'decode_kernel_us': None, 'cache_gbs_pct_of_8tbs': None,
        'prefill': {'decompress_us': dec_ms * 1e3, 'decompress_tflops': f_dec / dec_ms / 1e9,
                    'attention_us': att_ms * 1e3, 'attention_tflops': f_att / att_ms / 1e9,
                    'flops_decompress': f_dec, 'flops_attention': f_att},
        'roofline': {'bound': 'tensor', 'kernel': top, 'achieved': top_f / top_ms / 1e9, 'peak': tpeak, 'unit': 'TFLOP/s',
                     'frac': top_f / top_ms / 1e9 / tpeak, 'peak_kind': f'{tpeak_kind} bf16 GEMM', 'traffic': None,
                     'flops_per_launch': top_f},
        'gpu_launches': 2 * steps, 'clocks': clocks,
    }


def measure_conversion(args, name, shape, seqlens, seed, rank, world, local):
    """The conversion of one layer (Sec. 4.2, 4.3; App. B, C, D) on n synthetic calibration tokens: one step = key
    activations, per-group covariances, their eigenvectors, rotation of W_K, NoPE-key and value activations, alpha,
    the joint second moment, the rank-r subspace (orthogonal iteration) and the rewrite of W_DKV.  fp32 SIMT
    arithmetic: the roofline of its dominant kernel is the fp32 FMA rate."""
    import torch
    from paper_2502_07864_b200 import binding, replicas, synth
    n, D, g, d, r, fold, iters = seqlens[0], shape.D, shape.H, shape.dn, shape.r, 4, 20
    stream = torch.cuda.current_stream()
    case = synth.make_conversion_case(n, D, g, d, seed, device='cuda')
    x, w_k, w_v = case['x'], case['w_k'], case['w_v']
    groups, m, mz = d // 2 // fold, g * fold, (2 * g - 1) * d
    f32 = dict(dtype=torch.float32, device='cuda')
    k_act, v_act, k_nope = torch.empty(n, g * d, **f32), torch.empty(n, g * d, **f32), torch.empty(n, (g - 1) * d, **f32)
    cov, vals, U = torch.empty(groups, m, m, **f32), torch.empty(groups, m, **f32), torch.empty(groups, m, m, **f32)
    seg = torch.empty(binding.transmla_conv_rorope_scratch_bytes(n, g, d, fold) // 4, **f32)
    w_rot, w_dkv = torch.empty_like(w_k), torch.empty(mz, D, **f32)
    alpha, norms = torch.zeros(1, **f32), torch.empty(2 * n, **f32)
    Z, Cm = torch.empty(n, mz, **f32), torch.empty(mz, mz, **f32)
    gen = torch.Generator(device='cuda'); gen.manual_seed(seed)
    q0 = torch.randn(mz, r, generator=gen, device='cuda')
    Q = torch.empty_like(q0)
    ws = torch.empty(binding.transmla_conv_subspace_scratch_bytes(mz, r), dtype=torch.uint8, device='cuda')
    out_dkv = torch.empty(r, D, **f32)
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    ev = {}

    def mark(tag):
        ev.setdefault(tag, []).append(torch.cuda.Event(enable_timing=True))
        ev[tag][-1].record(stream)

    def step():
        mark('start')
        binding.transmla_conv_gemm(x, w_k, k_act, tb=True); mark('k_act')
        binding.transmla_conv_rorope_covariance(k_act, g, d, fold, seg, cov); mark('cov')
        binding.transmla_conv_sym_eig(cov, vals, U, status); mark('eig')
        binding.transmla_conv_rorope_apply(w_k, U, g, d, fold, w_rot); mark('rotate')
        binding.transmla_conv_gemm(x, w_rot[d:], k_nope, tb=True)
        binding.transmla_conv_gemm(x, w_v, v_act, tb=True); mark('nope_v_act')
        binding.transmla_conv_alpha(k_nope, v_act, norms, alpha)
        binding.transmla_conv_balance_concat(k_nope, v_act, alpha, Z); mark('alpha_concat')
        binding.transmla_conv_gemm(Z, Z, Cm, ta=True); mark('second_moment')
        Q.copy_(q0)
        binding.transmla_conv_top_subspace(Cm, Q, iters, ws, status); mark('subspace')
        w_dkv[:(g - 1) * d].copy_(w_rot[d:] / alpha); w_dkv[(g - 1) * d:].copy_(w_v)
        binding.transmla_conv_gemm(Q, w_dkv, out_dkv, ta=True); mark('rewrite')

    steps = max(2, min(args.steps, 3))
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    ev.clear()
    sampler = ClockSampler(local) if rank == 0 else None
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    replicas.barrier('cuda')
    t1 = time.perf_counter()
    clocks = sampler.stop(t0, t1) if sampler else None
    assert int(status.item()) == 0
    tags = ['k_act', 'cov', 'eig', 'rotate', 'nope_v_act', 'alpha_concat', 'second_moment', 'subspace', 'rewrite']
    prev = ['start'] + tags[:-1]
    part_ms = {t: statistics.median(ev[p][i].elapsed_time(ev[t][i]) for i in range(steps)) for p, t in zip(prev, tags)}
    ms_step = statistics.median(ev['start'][i].elapsed_time(ev['rewrite'][i]) for i in range(steps))
    (ms_step,) = replicas.max_over_ranks([ms_step], device='cuda')
    if rank != 0:
        return None
    f_sm = 2.0 * n * mz * mz
    sm_mhz = (clocks or {}).get('sm_mhz') or 1965.0
    peak = 148 * 128 * 2 * 1965.0e6 / 1e12     # fp32 FMA lanes x 2 flop x the maximum SM clock
    return {
        'metric': 'conversion of one layer: calibration tokens/s (RoRoPE + FreqFold + balanced joint PCA, synthetic activations)',
        'value': n * world / (ms_step * 1e-3), 'unit': 'tokens/s', 'n_gpus': world, 'steps': steps, 'warmup': 3,
        'ms_per_step': ms_step, 'higher_is_better': True, 'scaling': 'weak', 'vs_baseline': None, 'dtype': 'f32', 'data': 'synthetic',
        'config': {'workload': name, 'calibration_tokens': n, 'hidden': D, 'kv_heads': g, 'head_dim': d, 'freqfold': fold,
                   'rank': r, 'subspace_rounds': iters, 'l2': 'inputs larger than L2 (activations 2 x 134 MB, second moment 260 MB)',
                   'parallelism': f'replicas x{world}, no data-path collective'},
        'decode_kernel_us': None, 'cache_gbs_pct_of_8tbs': None,
        'conversion_ms': part_ms,
        'roofline': {'bound': 'alu', 'kernel': 'gemm_kernel<float> (second moment Z^T Z)', 'achieved': f_sm / part_ms['second_moment'] / 1e9,
                     'peak': peak, 'unit': 'TFLOP/s', 'frac': f_sm / part_ms['second_moment'] / 1e9 / peak,
                     'peak_kind': 'derived: 148 SMs x 128 fp32 lanes x 2 flop x 1965 MHz', 'traffic': None, 'flops_per_launch': f_sm,
                     'sm_mhz_sampled': sm_mhz},
        # gemm 6, gather 1, Jacobi 1, rotation 1, norms 3, concat 1, and (iters + 3) Cholesky QRs of three launches each
        'gpu_launches': (13 + iters + 3 * (iters + 3)) * steps, 'clocks': clocks,
    }


def measure(args, name, shape, seqlens, seed, rank, world, local, full):
    if '_conversion_' in name:
        return measure_conversion(args, name, shape, seqlens, seed, rank, world, local)
    if '_prefill_' in name:
        return measure_prefill(args, name, shape, seqlens, seed, rank, world, local)
    """One workload: whole-step time over args.steps steps, split-KV kernel time, read-probe ceiling, and (full) the
    host-buffer end-to-end figure and the optional layer step.  Returns the JSON line as a dict (rank 0)."""
    import torch
    from paper_2502_07864_b200 import binding, replicas, synth

    steps = args.steps if full else min(args.steps, 200)
    B, S, H = len(seqlens), shape.S, shape.H
    scale = (shape.dn + shape.dR) ** -0.5
    n_copies = args.cache_copies
    dc = synth.make_decode_case(shape, seqlens, replicas.rank_seed(seed, rank), device='cuda')
    ac = synth.make_append_case(shape, [L - S for L in seqlens], replicas.rank_seed(seed, rank) + 1, device='cuda')
    fp8 = '-fp8' in name
    if fp8:   # the FP8 cache replaces the bf16 one: same page table, rows in the library's 656-byte format
        first = synth.make_fp8_cache(shape, dc['cache'].shape[0], seed + 100, device='cuda')
        dc['cache'] = None
        caches = [first] + [first.clone() for _ in range(n_copies - 1)]
        fp8_scratch = torch.empty(B * S * shape.row, dtype=torch.float32, device='cuda')
        fp8_positions = torch.tensor([L - S for L in seqlens], dtype=torch.int32, device='cuda')
    else:
        caches = [dc['cache']] + [dc['cache'].clone() for _ in range(n_copies - 1)]
    # Weights rotate as well (their copies together exceed L2): in a whole model every other layer's weights pass
    # through L2 between two steps of this layer, so a step must find its own weights in HBM, not in L2.
    n_w = args.weight_copies
    weights = [(ac['w_dkv_kr'], dc['w_uk'], dc['w_uv'])] + [
        (ac['w_dkv_kr'].clone(), dc['w_uk'].clone(), dc['w_uv'].clone()) for _ in range(n_w - 1)]
    weight_bytes = sum(t.numel() * t.element_size() for t in weights[0])
    params = binding.make_params(shape, B, caches[0].shape[0], dc['page_table'].shape[1], scale)
    ws, lay = binding.alloc_workspace(params)
    out = torch.empty(B, S, H, shape.dv, dtype=torch.bfloat16, device='cuda')
    lse = torch.empty(B, S, H, dtype=torch.float32, device='cuda')
    status = torch.zeros(1, dtype=torch.int32, device='cuda')
    stream = torch.cuda.current_stream()

    def step(i, ev=None):
        if ev is not None:
            binding.transmla_profile_decode_kernel(ev[0], ev[1])
        if fp8:   # append, absorb + plan + split-KV decode, combine: five launches
            w_dkv_kr, w_uk, w_uv = weights[i % n_w]
            binding.transmla_latent_append_fp8(params, ac['x'], w_dkv_kr, fp8_positions, dc['page_table'], caches[i % n_copies],
                                               fp8_scratch, status, stream)
            binding.transmla_mla_decode_fp8(params, dc['q_nope'], dc['q_pe'], w_uk, caches[i % n_copies], dc['page_table'],
                                            dc['seqlens'], ws, status, stream)
            binding.transmla_mla_combine(params, ws, w_uv, out, lse, status, stream)
            return
        binding.transmla_decode_step(params, ac['x'], dc['q_nope'], dc['q_pe'], dc['page_table'], dc['seqlens'],
                                     *weights[i % n_w], caches[i % n_copies], ws, out, lse,
                                     status, stream)

    def barrier():
        replicas.barrier('cuda')

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    # The split-KV kernel is timed by events the library records around it, on every 8th step of the timed
    # region only: an event record between two kernels switches off their launch overlap for that step.
    sampled = list(range(0, steps, 8))
    kev = {i: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for i in sampled}
    for a, b_ in kev.values():       # create the underlying CUDA events before handing them to the library
        a.record(stream); b_.record(stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for i in range(steps):
        step(i, kev.get(i))
    e1.record(stream)
    barrier()
    t1 = time.perf_counter()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1) if sampler else None
    kernel_times = [a.elapsed_time(b_) for a, b_ in kev.values()]
    # At least 16 launches of the split-KV kernel are timed whatever --steps is: what the timed region did not give
    # comes from extra steps after it, each with the library's events around its split-KV kernel.
    extra = max(0, 16 - len(kernel_times))
    for i in range(extra):
        ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        ev[0].record(stream); ev[1].record(stream)
        step(steps + i, ev)
        torch.cuda.synchronize()
        kernel_times.append(ev[0].elapsed_time(ev[1]))
    kernel_ms = statistics.mean(kernel_times)
    word = int(status.item())
    assert word == 0, f'device status word {word:#x} after the timed steps'

    # Read-only streaming probe: the same pages through the same grid and TMA ring with nothing computed; its time is
    # the floor under the split-KV kernel for this workload (r = 512, dR = 64 only).
    probe_us = None
    if shape.r == 512 and shape.dR == 64 and not fp8:
        probe = []
        for i in range(3 + 20):
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record(stream)
            binding.transmla_stream_probe(params, caches[i % n_copies], dc['page_table'], ws, status, stream)
            ev[1].record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                probe.append(ev[0].elapsed_time(ev[1]) * 1e3)
        probe_us = statistics.median(probe)

    # end to end through the host-buffer entry point: pinned host inputs, result read back every step
    def end_to_end():
        staging = torch.empty(binding.transmla_step_staging_bytes(params), dtype=torch.uint8, device='cuda')
        pin = lambda t: t.cpu().contiguous().pin_memory()
        h = {k: pin(v) for k, v in (('x', ac['x']), ('q_nope', dc['q_nope']), ('q_pe', dc['q_pe']),
                                    ('page_table', dc['page_table']), ('seqlens', dc['seqlens']))}
        h_out = torch.empty(B, S, H, shape.dv, dtype=torch.bfloat16).pin_memory()
        h_lse = torch.empty(B, S, H, dtype=torch.float32).pin_memory()

        def host_step(i):
            word = binding.transmla_decode_step_host(params, h['x'], h['q_nope'], h['q_pe'], h['page_table'], h['seqlens'],
                                                     *weights[i % n_w], caches[i % n_copies], staging,
                                                     ws, h_out, h_lse, stream)
            assert word == 0, f'device status word {word:#x} in host step {i}'
        for i in range(3):
            host_step(i)
        barrier()
        t2 = time.perf_counter()
        for i in range(steps):
            host_step(i)
        barrier()
        e2e_s = time.perf_counter() - t2
        h2d = sum(v.numel() * v.element_size() for v in h.values())
        d2h = h_out.numel() * 2 + h_lse.numel() * 4 + 4
        return e2e_s, h2d, d2h

    e2e_s, h2d, d2h = end_to_end() if full and not fp8 else (float('nan'), 0, 0)   # skipped for the rows of the sweep

    layer = None
    if args.layer and full:
        # the whole attention layer (queries -> the step above -> W_O) on device buffers; its weights rotate too
        lws = []
        for i in range(args.layer_weight_copies):
            lw = synth.make_layer_weights(shape, seed + 10 + i, q_lora_rank=args.q_lora_rank, device='cuda')
            lw.update(w_dkv_kr=weights[i % n_w][0], w_uk=weights[i % n_w][1], w_uv=weights[i % n_w][2])
            lws.append(lw)
        scratch = torch.empty(binding.transmla_layer_scratch_bytes(params, args.q_lora_rank), dtype=torch.uint8, device='cuda')
        y = torch.empty(B, S, shape.D, dtype=torch.bfloat16, device='cuda')

        def layer_step(i):
            binding.transmla_layer_decode_step(params, lws[i % len(lws)], ac['x'], dc['page_table'], dc['seqlens'],
                                               caches[i % n_copies], ws, scratch, y, status, stream)
        for i in range(max(args.warmup, 3)):
            layer_step(i)
        barrier()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record(stream)
        for i in range(steps):
            layer_step(i)
        l1.record(stream)
        barrier()
        word = int(status.item())
        assert word == 0, f'device status word {word:#x} after the layer steps'
        layer_ms = replicas.max_over_ranks([l0.elapsed_time(l1)], device='cuda')[0] / steps
        lbytes = sum(t.numel() * t.element_size() for t in lws[0].values())
        layer = {'ms_per_step': layer_ms, 'tokens_per_s': B * S * world / (layer_ms * 1e-3), 'weight_bytes': lbytes,
                 'q_lora_rank': args.q_lora_rank, 'launches_per_step': 6 + (1 if args.q_lora_rank else 0),
                 'gbs_weights_plus_cache': (lbytes + sum(seqlens) * shape.row * 2) / (layer_ms * 1e-3) / 1e9}

    ms_total, e2e_ms = replicas.max_over_ranks([ms_total, e2e_s * 1e3], device='cuda')
    if rank != 0:
        return None

    tokens_per_step = B * S * world
    ms_step = ms_total / steps
    cache_bytes = sum(seqlens) * (synth.FP8_ROW_BYTES if fp8 else shape.row * 2)   # live latent rows, read once
    q_hat_bytes = B * S * H * shape.row * 2
    algo_bytes = cache_bytes + q_hat_bytes                           # per split-KV launch
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    peak, peak_kind = measured_hbm_peak()
    # the other roof: 2 * (r + dR) flop for a score and 2 * r for its share of the weighted sum, per query row and token
    flops = 2.0 * (shape.row + shape.r) * H * S * sum(seqlens)
    tpeak, tpeak_kind = measured_tensor_peak()
    tflops = flops / (kernel_ms * 1e-3) / 1e12
    # ncu dram__bytes_read.sum + dram__bytes_write.sum of one split-KV launch of this workload, as recorded in the
    # summary under profiles/ together with a hash of the kernel's sources; null once those have changed
    traffic = traffic_from_profile(name) if world == 1 else None
    claims = 'run-time' if binding.transmla_page_claims_at_run_time(params) else 'planned'
    line = {
        'metric': METRIC, 'value': replicas.whole_job_rate(B * S, steps, ms_total), 'unit': 'tokens/s', 'n_gpus': world,
        'steps': steps, 'warmup': max(args.warmup, 3), 'ms_per_step': ms_step, 'higher_is_better': True,
        'scaling': 'weak', 'vs_baseline': None, 'dtype': 'e4m3 cache, bf16/fp16 operands' if fp8 else 'bf16', 'data': 'synthetic',
        'config': {'workload': name, 'batch_per_gpu': B, 'q_len': S, 'heads': H, 'latent': shape.r, 'rope': shape.dR,
                   'cached_tokens_per_gpu': sum(seqlens), 'page_size': shape.page_size,
                   'num_partitions': lay.num_partitions, 'page_claims': claims,
                   'l2': f'cache rotates over {n_copies} copies ({n_copies * cache_bytes / 1e6:.0f} MB) and the weights '
                         f'over {n_w} copies ({n_w * weight_bytes / 1e6:.0f} MB) between steps',
                   'parallelism': f'replicas x{world}, no data-path collective'},
        'cache_gbs': world * cache_bytes / (ms_step * 1e-3) / 1e9,
        'cache_gbs_pct_of_8tbs': 100.0 * cache_bytes / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        'decode_kernel_us': kernel_ms * 1e3, 'decode_kernel_launches_timed': len(kernel_times),
        'decode_kernel_timing': f'library events around the split-KV kernel: every 8th step of the timed region ({len(kev)}) '
                                f'and {extra} extra steps after it',
        'roofline': {'bound': 'hbm', 'achieved': achieved, 'peak': peak, 'unit': 'GB/s', 'frac': achieved / peak,
                     'peak_kind': f'{peak_kind} copy bandwidth', 'frac_of_8tbs': achieved / NOMINAL_HBM_GBS,
                     'kernel': 'split-KV decode', 'algorithmic_bytes_per_launch': algo_bytes, 'traffic': traffic,
                     'traffic_source': 'ncu capture summarised under profiles/ (null: none for this workload, or the kernel changed since)',
                     'read_probe_us': probe_us,
                     'read_probe_gbs': None if probe_us is None else cache_bytes / probe_us / 1e3,
                     'tensor': {'achieved_tflops': tflops, 'peak_tflops': tpeak, 'peak_kind': f'{tpeak_kind} bf16 GEMM',
                                'frac': tflops / tpeak, 'flops_per_launch': flops}},
        'e2e': {'value': replicas.whole_job_rate(B * S, steps, e2e_ms), 'unit': 'tokens/s',
                'h2d_bytes_per_step': h2d, 'd2h_bytes_per_step': d2h, 'ms_per_step': e2e_ms / steps},
        'gpu_launches': (5 if fp8 else KERNELS_PER_STEP) * steps,
        'clocks': clocks,
    }
    if layer is not None:
        line['layer'] = layer
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument('--gpus', type=int, default=1)
    ap.add_argument('--steps', type=int, default=1000)
    ap.add_argument('--warmup', type=int, default=20)
    ap.add_argument('--impl', default='ours', choices=['ours', 'reference'])
    ap.add_argument('--workload', default='llama2-7b-mla_b16_8k')
    ap.add_argument('--cache-copies', type=int, default=4)
    ap.add_argument('--weight-copies', type=int, default=12)
    ap.add_argument('--no-cpu-baseline', action='store_true')
    ap.add_argument('--layer', action='store_true', help='also time the whole layer step (queries, attention, W_O)')
    ap.add_argument('--q-lora-rank', type=int, default=0, help='low-rank queries for --layer (0: full rank)')
    ap.add_argument('--layer-weight-copies', type=int, default=6)
    ap.add_argument('--sweep', default='llama2-7b-mla_b64_8k,llama2-7b-mla_b128_8k,qwen2.5-72b-mla_b64_s2,llama2-7b-mla-fp8_b64_8k,'
                            'llama2-7b-mla_prefill_b16_8k_s2048',
                    help='comma-separated workloads measured after the main one (1 GPU; empty: none)')
    args = ap.parse_args()
    w = workloads()
    if args.workload not in w:
        sys.exit(f'unknown workload {args.workload}; choose from {sorted(w)}')
    shape, seqlens, seed = w[args.workload]
    if args.impl == 'reference':
        run_reference(args, args.workload, shape, seqlens, seed)
    else:
        run_ours(args, args.workload, shape, seqlens, seed)


if __name__ == '__main__':
    main()
