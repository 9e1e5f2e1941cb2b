"""The N > 1 path of the benchmark on CPU: two gloo ranks, no GPU.

The compress / decompress pair has no exchange step (samples are independent), so N GPUs run N replicas and
the only cross-rank code is the aggregation of the timing: time = max over ranks, bytes = sum over ranks."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["DIV_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
    rank = dist.get_rank()
    ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), dist, None)
    solo_ms, solo_units = bench.aggregate_over_ranks(3.0, 7.0, None, None)
    print(json.dumps({"rank": rank, "ms": ms, "units": units, "solo": [solo_ms, solo_units]}))
    dist.destroy_process_group()
""")


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_aggregate_max_time_and_summed_bytes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   DIV_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        r = json.loads(out.strip().splitlines()[-1])
        assert r["ms"] == 15.0                 # the slower rank
        assert r["units"] == 3000.0            # both ranks' bytes
        assert r["solo"] == [3.0, 7.0]         # one rank: untouched


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
