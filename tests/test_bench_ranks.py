"""The N > 1 path of bench.py on CPU: N independent replicas, no data-path collective; the only
exchange is the final aggregation (slowest rank's time, summed units), run here as two gloo ranks."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1))
print(json.dumps(dict(rank=rank, ms=ms, units=units)))
dist.destroy_process_group()
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_max_time_and_summed_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = [json.loads(p.communicate(timeout=120)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    for o in outs:
        assert o["ms"] == 15.0 and o["units"] == 300.0       # max over ranks, sum over ranks


def test_single_process_aggregation_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.5, 7) == (3.5, 7.0)


def test_reference_arm_other_ranks_do_no_work():
    """Under torchrun only rank 0 runs the oracle; the other ranks exit 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_byte_model_counts_the_rows_of_every_variant():
    """Algorithmic KV bytes follow the rows alive per layer: one chain at one layer, one layer per
    prediction step, a chain under every node."""
    sys.path.insert(0, ROOT)
    import bench
    import synth_inputs as si
    s = si.CONFIGS["c2"]
    kv_row = 2 * 2 * s.n_kv
    try:
        bench.INSERT_LAYERS, bench.CHAINS = None, False
        base = bench.algorithmic_bytes(s, 512)
        assert base["kv_write"] == kv_row * (s.l * s.T + (s.L - s.l) * (s.T + s.k))
        bench.INSERT_LAYERS = [15, 20, 25]
        per_step = bench.algorithmic_bytes(s, 512)
        rows = sum(s.T + sum(1 for t in (15, 20, 25) if t <= j) for j in range(s.L))
        assert per_step["kv_write"] == kv_row * rows and per_step["weights"] == base["weights"]
        bench.INSERT_LAYERS, bench.CHAINS = None, True
        chains = bench.algorithmic_bytes(s, 512)
        assert chains["kv_write"] == kv_row * (s.l * s.T + (s.L - s.l) * s.T * (1 + s.k))
    finally:
        bench.INSERT_LAYERS, bench.CHAINS = None, False


def test_reference_arm_rejects_bad_insert_layers():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                        "--insert-layers", "1,0,1"], capture_output=True, text=True, timeout=120)
    assert r.returncode != 0 and "non-decreasing" in (r.stderr + r.stdout)
