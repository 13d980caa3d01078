"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path does not shard (replicas
only), so what runs across ranks is the max-over-ranks step time and the reference arm's rule
that only rank 0 works and prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["TWN_ROOT"])
import torch.distributed as dist
import bench
rank, local, world = bench.dist_env()
dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{os.environ['MASTER_PORT']}", rank=rank, world_size=world)
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, dist, "cpu")
assert ms == 15.0, ms
# whole-job value for replicas: units of all ranks over the slowest rank's time
value = world * 64 / (ms * 1e-3)
if rank == 0:
    print("VALUE", value)
dist.destroy_process_group()
"""


def _free_port():
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    port = str(_free_port())
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port, TWN_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "VALUE 8533.3" in outs[0][0]
    assert "VALUE" not in outs[1][0]


def test_reference_arm_only_rank0_prints():
    outs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2")
        p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                            "lenet5_fwd", "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env,
                           capture_output=True, text=True, timeout=300)
        assert p.returncode == 0, p.stderr
        outs.append(p.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
    assert outs[1] == ""
