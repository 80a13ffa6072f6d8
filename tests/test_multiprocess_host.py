"""The N > 1 side of the benchmark on CPU: two processes over gloo.

The decode step needs no exchange between sequences, so N GPUs run N independent replicas; what the
ranks share is the plumbing around the timed region: the barrier, the slowest rank's time, the
whole-job rate, and that only rank 0 reports.  This runs that plumbing (bench.Ranks) without a GPU.
"""
from __future__ import annotations

import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys, time
sys.path.insert(0, {root!r})
import bench
ranks = bench.Ranks("gloo", device="cpu")
ranks.barrier()
mine = 1.0 if ranks.rank == 0 else 3.0            # this rank's "time" in ms
slowest = ranks.max_over_ranks(mine)
if ranks.rank == 1:
    time.sleep(0.3)                               # the barrier must hold rank 0 back
t0 = time.perf_counter()
ranks.barrier()
waited = time.perf_counter() - t0
out = dict(rank=ranks.rank, world=ranks.world, root=ranks.is_root, slowest=slowest,
           rate=ranks.whole_job_rate(10, slowest), waited=waited)
ranks.close()
print("RESULT " + json.dumps(out), flush=True)
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code: str, world: int, extra_env=None, args=()):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), RANK=str(rank),
                   LOCAL_RANK=str(rank), **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, "-c", code, *args], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=240)
        assert p.returncode == 0, se[-2000:]
        outs.append(so)
    return outs


def test_two_ranks_share_barrier_slowest_time_and_rate():
    outs = _spawn(WORKER.format(root=ROOT), 2)
    res = [json.loads(line[len("RESULT "):]) for o in outs for line in o.splitlines() if line.startswith("RESULT ")]
    assert sorted(r["rank"] for r in res) == [0, 1] and all(r["world"] == 2 for r in res)
    assert [r["root"] for r in sorted(res, key=lambda r: r["rank"])] == [True, False]
    for r in res:
        assert r["slowest"] == 3.0                       # the maximum over ranks, on every rank
        assert abs(r["rate"] - 2 * 10 / 3e-3) < 1e-6     # both replicas' steps over the slowest rank's time
    r0 = next(r for r in res if r["rank"] == 0)
    assert r0["waited"] > 0.2                            # rank 0 waited at the barrier for rank 1


def test_single_process_needs_no_process_group():
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    code = (f"import sys; sys.path.insert(0, {ROOT!r}); import bench; r = bench.Ranks('gloo', device='cpu'); r.barrier(); "
            "assert r.world == 1 and r.is_root and r.max_over_ranks(2.5) == 2.5 and r.whole_job_rate(5, 1.0) == 5000.0; "
            "r.close(); print('ok')")
    p = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and "ok" in p.stdout, p.stderr[-2000:]


def test_reference_arm_runs_on_rank_0_only():
    """Under a 2-process launch the oracle arm works on rank 0 alone; the other rank leaves with status 0
    and prints nothing."""
    code = (f"import sys; sys.path.insert(0, {ROOT!r}); import bench; "
            "sys.argv = ['bench.py', '--impl', 'reference', '--workload', 'tiny', '--steps', '1', '--warmup', '0', '--gpus', '2']; "
            "bench.main()")
    outs = _spawn(code, 2)
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1].strip() == ""
