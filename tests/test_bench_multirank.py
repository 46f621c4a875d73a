"""The N > 1 path of bench.py on CPU: two gloo ranks, independent replicas, max-over-ranks timing."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%d" %% int(os.environ["PORT"]),
                            rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
    rank = dist.get_rank()
    mine = 0.010 if rank == 0 else 0.025            # rank 1 is the slow replica
    slowest = bench.max_over_ranks(mine, device="cpu")
    value = bench.whole_job_value(32768, dist.get_world_size(), slowest)
    print(json.dumps({"rank": rank, "slowest": slowest, "value": value}))
    dist.barrier()
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_agree_on_the_slowest_replica(tmp_path):
    import json
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert abs(o["slowest"] - 0.025) < 1e-12                 # both ranks see the max
        assert abs(o["value"] - 2 * 32768 / 0.025) < 1e-6        # whole-job tokens/s of two replicas


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, device="cpu") == 0.5
    assert bench.whole_job_value(100, 1, 0.5) == 200.0


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_ncu_traffic_is_tied_to_kernel_source_and_shape(monkeypatch):
    """The stored DRAM-traffic figures are reported only for the kernel source and per-layer shape they were
    measured on; anything else must give null rather than a stale number."""
    import bench
    from paper_2412_14838_b200 import synth
    w = synth.WORKLOADS["mistral32k"]
    got = bench.ncu_traffic(w, w.L // 4 + 1)
    if got is not None:                       # the source is the measured one
        assert got["cold_bytes_per_launch"] >= got["live_bytes_per_launch"] >= 4 * w.k_bytes_per_layer()
    assert bench.ncu_traffic(w, w.L + 1) is None          # another grouping of the layers
    assert bench.ncu_traffic(w) is None
    assert bench.ncu_traffic(synth.WORKLOADS["tiny"], 2) is None
    monkeypatch.setitem(bench.NCU_TRAFFIC, "kernel_sha256", "0" * 64)
    assert bench.ncu_traffic(w, w.L // 4 + 1) is None
