"""The library may be called from any host thread: the first tensor-core launch of a context made
on a thread that has not touched CUDA before (new tensor maps are encoded there) gives the same
result as on the main thread."""
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
