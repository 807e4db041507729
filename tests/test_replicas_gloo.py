"""World-size-2 CPU test (gloo) of the multi-process path of bench.py: replicas only, no data-path collective.

Each rank times its own replica; the job's time is the maximum over ranks and the reported value is the sum of
the tokens all ranks decoded divided by that time.  The reference arm runs on rank 0 alone.
"""
import json
import os
import socket
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = textwrap.dedent("""
    import json, os, sys
    import torch, torch.distributed as dist
    sys.path.insert(0, os.environ["KL_ROOT"])
    import bench
    rank = int(os.environ["RANK"])
    dist.init_process_group("gloo")
    bench._DIST["on"] = True
    bench.barrier()
    local_ms = 10.0 + 5.0 * rank               # rank 1 is the slow replica
    value, ms = bench.replica_throughput(steps=8, batch=1, world=dist.get_world_size(), ms_local=local_ms)
    bench.barrier()
    print(json.dumps({"rank": rank, "value": value, "ms": ms, "max_only": bench.max_over_ranks(float(rank))}))
    dist.destroy_process_group()
""")


def test_two_replicas_report_whole_job_throughput_over_the_slowest_rank(tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), KL_ROOT=str(ROOT), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 15.0                         # the slowest replica's time, on every rank
        assert abs(o["value"] - 2 * 8 / 15.0e-3) < 1e-6  # tokens of BOTH replicas over that time
        assert o["max_only"] == 1.0


def test_single_process_path_needs_no_process_group():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench._DIST["on"] is False
    value, ms = bench.replica_throughput(steps=4, batch=1, world=1, ms_local=8.0)
    assert ms == 8.0 and abs(value - 500.0) < 1e-9


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", CUDA_VISIBLE_DEVICES="")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "1", "--workload", "tiny_b1_ctx128"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    assert res.stdout.strip() == ""


def test_reference_arm_prints_one_line_on_rank_zero():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", CUDA_VISIBLE_DEVICES="")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--workload", "tiny_b1_ctx128"], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
