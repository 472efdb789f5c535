"""The library may be called from any host thread: the first tensor-core launch of a context made
on a thread that has not touched CUDA before (new tensor maps are encoded there) gives the same
result as on the main thread."""
import os
import subprocess
import sys
import threading

import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_first_launch_from_a_worker_thread():
    w = synth.Workload("t", (256, 1024, 1024, 35), S=4, B=128, K=2, rounds=1, precision="bf16", x_dist="normal",
                       lr=0.05, seed=21)
    W, b, data = H.make_problem(w)
    _, Wm, bm, _, lm = H.gpu_round(w, W, b, data, seed=4)          # main thread
    out = {}

    def work():
        try:
            out["r"] = H.gpu_round(w, W, b, data, seed=4)            # new context, new buffers, new thread
        except Exception as e:                                        # surfaces in the main thread below
            out["e"] = e

    t = threading.Thread(target=work)
    t.start()
    t.join()
    assert "e" not in out, out.get("e")
    _, Wt, bt, _, lt = out["r"]
    assert np.array_equal(lt, lm)
    for l in range(len(W)):
        assert np.array_equal(Wt[l], Wm[l]) and np.array_equal(bt[l], bm[l])


_TWO_THREADS = r"""
import sys, threading
import numpy as np
import torch
sys.path.insert(0, sys.argv[1])
from paper_1910_02120_b200 import synth
from tests import helpers as H

# two shapes that use different kernel templates; both threads start at once, each with its own
# context and stream, in a process where no kernel of the library has been launched before
cases = [synth.Workload("a", (256, 1024, 1024, 35), S=4, B=128, K=2, rounds=1, precision="bf16", x_dist="normal",
                        lr=0.05, seed=21),
         synth.Workload("b", (512, 4096, 16), S=8, B=512, K=2, rounds=1, precision="bf16", x_dist="normal",
                        lr=0.05, seed=22)]
probs = [H.make_problem(w) for w in cases]
torch.zeros(1, device="cuda:0")
gate = threading.Barrier(2)
out = [None, None]

def work(i):
    try:
        with torch.cuda.stream(torch.cuda.Stream()):
            gate.wait()
            r = H.gpu_round(cases[i], *probs[i], seed=4)
        out[i] = r
    except Exception as e:
        out[i] = e

ts = [threading.Thread(target=work, args=(i,)) for i in range(2)]
[t.start() for t in ts]
[t.join() for t in ts]
for i in range(2):
    assert not isinstance(out[i], Exception), out[i]
    ref = H.gpu_round(cases[i], *probs[i], seed=4)          # same case again, alone
    assert np.array_equal(out[i][4], ref[4])
    for a, b in zip(out[i][1] + out[i][2], ref[1] + ref[2]):
        assert np.array_equal(a, b)
print("ok")
"""


def test_two_threads_make_the_first_launches_of_a_fresh_process_together():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _TWO_THREADS, root], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]
