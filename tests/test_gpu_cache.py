"""The cache of generated kernels: handles of the same graph share one loaded kernel, a destroyed
handle gives its kernel back, and with PN_CACHE_DIR set a second process loads the compiled kernel
from disk instead of compiling it."""
import os
import subprocess
import sys
import time

import pytest

import paper_2605_29357_b200 as pn
from pn_workloads import configs as C

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_handles_share_kernels_and_give_them_back():
    w = C.c1(M=8, N=192)                      # a shape no other test uses: its kernel is not loaded yet
    a = pn.Graph(w.desc, 0, 0)
    loaded, used = a.kernel_cache
    b = pn.Graph(w.desc, 0, 0)                # the same source: no second module
    assert b.kernel_cache == (loaded, used)
    b.close()
    assert a.kernel_cache == (loaded, used)   # still held by a
    a.close()
    c = pn.Graph(C.c1(M=8, N=320).desc, 0, 0)
    loaded2, used2 = c.kernel_cache
    assert used2 == used and loaded2 == loaded + 1    # a's kernel is loaded but unused; c's is new
    c.close()


def test_disk_cache_spares_the_second_process_the_compilation(tmp_path):
    code = (
        "import sys, time; sys.path.insert(0, %r)\n"
        "import paper_2605_29357_b200 as pn\n"
        "from pn_workloads import configs as C\n"
        "import torch; torch.cuda.init()\n"
        "pn.Graph(C.c1(M=4, N=64).desc, 0, 0)\n"      # pays the one-time start-up costs
        "w = C.c5(**C.SMALL['c5'])\n"
        "t0 = time.perf_counter(); g = pn.Graph(w.desc, 0, pn.FLAG_UNFUSED); dt = time.perf_counter() - t0\n"
        "print('SECONDS', dt, g.n_kernels)\n" % ROOT)
    env = dict(os.environ, PN_CACHE_DIR=str(tmp_path / "kernels"))
    times = []
    for _ in range(2):
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        line = [ln for ln in r.stdout.splitlines() if ln.startswith("SECONDS")][-1].split()
        times.append(float(line[1]))
    files = os.listdir(tmp_path / "kernels")
    assert files and all(f.endswith("_sm100a.cubin") for f in files)
    assert times[1] < 0.5 * times[0], times   # several NVRTC compilations against reading a few files
