"""Host-side logic of bench.py that needs no GPU: the work model behind the roofline numbers,
the replica aggregation over two gloo ranks, and the reference arm's bounded oracle sample."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_1910_02120_b200 import synth  # noqa: E402


def test_work_model_matches_closed_forms():
    # flop count of Sec. 2.3 with the true constants: forward 2B per weight, backward 4B (2B for
    # the first layer, which needs no input gradient); middle layers cost 1/S of the full layer
    w = synth.C3
    wm = bench.work_model(w)
    N0, N1, N2, N3 = w.layer_dims
    S, B, K = w.S, w.B, w.K
    packed = N0 * N1 + N1 * N2 // S + N2 * N3
    assert wm["packed_elems"] == packed
    assert wm["flops"]["fwd"] == 2 * B * packed * K
    assert wm["flops"]["dw_sgd"] == 2 * B * packed * K
    assert wm["flops"]["dx"] == 2 * B * (N1 * N2 // S + N2 * N3) * K
    per_step = sum(wm["flops"].values()) / K
    assert abs(per_step - 2.07e11) / 2.07e11 < 0.01
    assert wm["bytes"]["gather"] == packed * 10 and wm["bytes"]["scatter"] == packed * 8
    assert wm["bytes"]["dw_sgd"] == packed * 10 * K


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    val = bench.job_value(1000, 4, world, ms)
    if rank == 0:
        json.dump({"ms": ms, "value": val}, open(out, "w"))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks(tmp_path):
    out = str(tmp_path / "r.json")
    port = 29500 + os.getpid() % 1000
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 15.0                                  # max over ranks
    assert abs(r["value"] - 2 * 1000 * 4 / 15e-3) < 1e-6    # both replicas' samples over that time


def test_reference_arm_prints_one_json_line():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "C1",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "samples/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["steps"] == 2


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "C1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, env=env)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_recorded_dram_traffic_is_dropped_when_the_kernel_source_changes(tmp_path, monkeypatch):
    """roofline.traffic comes from a tracked ncu record and must read null once the kernel it was
    taken on has been edited."""
    import hashlib
    import json
    import bench
    src = tmp_path / "k.cu"
    src.write_text("kernel v1")
    rec = {"W": {"upd": {"dram_bytes_per_launch": 110.0, "algorithmic_per_launch": 100.0, "unit": "bytes",
                         "source": "k.cu", "source_sha256": hashlib.sha256(b"kernel v1").hexdigest()}}}
    f = tmp_path / "t.json"
    f.write_text(json.dumps(rec))
    monkeypatch.setattr(bench, "TRAFFIC_FILE", str(f))
    monkeypatch.setattr(bench, "CSRC", str(tmp_path))
    assert bench.measured_traffic("W", "upd", 200.0) == 220.0          # scaled by the launch's algorithmic work
    assert bench.measured_traffic("W", "other", 200.0) is None
    assert bench.measured_traffic("V", "upd", 200.0) is None
    src.write_text("kernel v2")
    assert bench.measured_traffic("W", "upd", 200.0) is None
