"""Builds libtransmla.so (sm_100a only) in-tree with nvcc."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, 'csrc')
LIB = os.path.join(HERE, 'libtransmla.so')
SOURCES = ['api.cu', 'small_kernels.cu', 'decode_generic.cu', 'decode_sm100.cu', 'static_workspace.cu', 'selftest.cu', 'linear.cu', 'linear_sm100.cu', 'stream_probe.cu', 'decode_fp8.cu', 'append_fp8.cu', 'prefill_decompress.cu', 'prefill_attention.cu', 'prefill_api.cu', 'conversion.cu', 'conversion_api.cu']


def _stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, 'include', 'transmla.h')]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False):
    """Compile the library if it is missing or older than its sources.  Returns its path."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get('NVCC', '/usr/local/cuda/bin/nvcc')
    cmd = [nvcc, '-gencode', 'arch=compute_100a,code=sm_100a', '-O3', '-std=c++17', '-lineinfo', '-shared',
           '-Xcompiler', '-fPIC', '-I', os.path.join(ROOT, 'include'), '-I', CSRC]
    if verbose:
        cmd += ['-Xptxas', '-v']
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ['-o', LIB + '.tmp']
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError('nvcc failed building libtransmla.so')
    os.replace(LIB + '.tmp', LIB)
    if verbose:
        sys.stderr.write(res.stderr)
    return LIB


if __name__ == '__main__':
    build(force=True, verbose='-v' in sys.argv)
    print(LIB)
