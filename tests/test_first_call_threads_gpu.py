"""Two host threads make their FIRST calls into the library at the same moment (fresh process, so
every per-device table -- device properties, each kernel's shared-memory attribute, the resident
grid size -- is still unset): both must succeed and give the results a single thread gets."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys, threading
import numpy as np, torch
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
from gpu_util import random_bits, to_dev
from paper_2605_09825_b200 import api
api.load_library()
torch.cuda.init(); torch.zeros(1, device="cuda")
rng = np.random.default_rng(5)
X = [to_dev(random_bits(rng, 416, 288)) for _ in range(2)]
W = [to_dev(random_bits(rng, 672, 288)) for _ in range(2)]
streams = [torch.cuda.Stream() for _ in range(2)]
gate = threading.Barrier(2)
out, err = [None, None], [None, None]
def work(i):
    try:
        with torch.cuda.stream(streams[i]):
            gate.wait()
            out[i] = api.linear_fprop(X[i], W[i], api.HADAMARD_DET, api.ROUND_RNE, 3)
            streams[i].synchronize()
    except Exception as exc:
        err[i] = repr(exc)
th = [threading.Thread(target=work, args=(i,)) for i in range(2)]
[t.start() for t in th]; [t.join() for t in th]
assert err == [None, None], err
api.check()
for i in range(2):
    want = api.linear_fprop(X[i], W[i], api.HADAMARD_DET, api.ROUND_RNE, 3)
    api.check()
    assert torch.equal(out[i], want), i
print("threads-ok")
"""


def test_two_threads_first_call():
    res = subprocess.run([sys.executable, "-c", CHILD, ROOT], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "threads-ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
