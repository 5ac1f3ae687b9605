"""The N > 1 path of the benchmark on CPU: two gloo ranks as data-parallel replicas.

No kernel runs here; the test covers what the ranks exchange: distinct seeded batches per rank, the
barrier, the maximum of the per-rank times and the whole-job rate built from it, and that the
reference arm leaves every rank but 0 without work.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world_size, port, out_dir):
    os.environ.update(MASTER_ADDR='127.0.0.1', MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world_size))
    sys.path.insert(0, ROOT)
    from paper_2502_07864_b200 import replicas, synth
    dist.init_process_group('gloo', rank=rank, world_size=world_size)
    assert replicas.world() == (rank, world_size)
    case = synth.make_decode_case(synth.TINY, [17, 64], replicas.rank_seed(1, rank))
    replicas.barrier('cpu')
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    total_ms, e2e_ms = replicas.max_over_ranks([my_ms, 2 * my_ms])
    rate = replicas.whole_job_rate(units_per_rank_per_step=2, steps=5, total_ms=total_ms)
    json.dump({'total_ms': total_ms, 'e2e_ms': e2e_ms, 'rate': rate, 'q0': float(case['q_nope'].float().sum())},
              open(os.path.join(out_dir, f'rank{rank}.json'), 'w'))
    replicas.barrier('cpu')
    dist.destroy_process_group()


def test_two_replicas_share_only_timing(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.load(open(tmp_path / f'rank{r}.json')) for r in (0, 1))
    assert r0['total_ms'] == r1['total_ms'] == 15.0 and r0['e2e_ms'] == 30.0       # the slowest rank decides
    assert abs(r0['rate'] - 2 * 2 * 5 / 15e-3) < 1e-6                              # both ranks' work over that time
    assert r0['q0'] != r1['q0']                                                    # each replica has its own batch


def test_without_a_process_group_it_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_2502_07864_b200 import replicas
    assert replicas.world() == (0, 1)
    assert replicas.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert replicas.whole_job_rate(16, 10, 2.0) == 16 * 10 / 2e-3


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK='1', WORLD_SIZE='2', LOCAL_RANK='1')
    res = subprocess.run([sys.executable, os.path.join(ROOT, 'bench.py'), '--impl', 'reference', '--gpus', '2',
                          '--steps', '1', '--warmup', '0'], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ''
