"""Host logic of the multi-GPU bench (replicas only): two gloo ranks on CPU.

The path has no exchange step, so N GPUs run N independent replicas; what the ranks share is only the timing
rule (barrier, then the maximum over ranks) and who prints. These tests cover that rule and the rule that the
oracle arm runs on rank 0 alone.
"""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
mine = [10.0 + 5.0 * rank, 100.0 - 20.0 * rank]          # rank 1 is slower on the first, faster on the second
got = bench.max_over_ranks(mine, world, "cpu")
dist.barrier()
print(json.dumps({"rank": rank, "max": got, "rate": bench.whole_job_rate(2.0e12, got[0], world)}))
dist.destroy_process_group()
"""


def _spawn(code, extra_args=(), world=2, port=29611):
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", code, ROOT, *extra_args], env=env, cwd=ROOT,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_whole_job_rate_gloo_world2():
    outs = _spawn(WORKER)
    for out in outs:
        rec = json.loads(out.strip().splitlines()[-1])
        assert rec["max"] == [15.0, 100.0]                    # slowest rank wins, per entry
        # two replicas, 2e12 ops each, 15 ms per step -> 2 * 2e12 / 0.015 s = 266.67 TOPS for the whole job
        assert rec["rate"] == pytest.approx(2 * 2.0e12 / 0.015 / 1e12)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]
    assert bench.whole_job_rate(1.0e12, 1.0, 1) == pytest.approx(1000.0)


REF_WORKER = r"""
import os, sys, types
sys.path.insert(0, sys.argv[1])
import bench
calls = []
def fake_sample(rows=2048, attn_rows=2048, hs=32):
    calls.append(rows)
    return 0.5, "fake sample"
bench.oracle_step_sample = fake_sample
bench.run_reference(types.SimpleNamespace(steps=2, warmup=1))
print("CALLS", len(calls))
"""


def test_reference_arm_runs_on_rank0_only():
    outs = _spawn(REF_WORKER, port=29612)
    lines0 = outs[0].strip().splitlines()
    lines1 = outs[1].strip().splitlines()
    assert lines1 == ["CALLS 0"]                              # rank 1 does no work and prints no line
    rec = json.loads(lines0[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2
    assert rec["e2e"] == {"value": rec["value"], "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["value"] == rec["value"]
    assert lines0[-1] == "CALLS 3"                            # one warm-up and two timed samples


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself():
    """`bench.py --gpus 2` started plainly (no WORLD_SIZE) re-runs itself as two ranks of one node; shown here with
    the oracle arm, which needs no GPU: one JSON line, from rank 0, that says n_gpus = 2."""
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.rank_launch_command(2, ["--gpus", "2"])
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-2:] == ["--gpus", "2"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--steps", "1", "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["extrapolated"] is True
    assert rec["measured_wall_seconds"] > 0
