"""The benchmark's N > 1 logic on CPU ranks: two `gloo` processes run the replica plumbing (barrier, max over
ranks, whole-job rate), and the reference arm's rank-0-only rule is checked with a second rank that must stay silent."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_RANK_PROG = r"""
import json, os, sys, time
sys.path.insert(0, %r)
import bench
rep = bench.Replicas("gloo")
assert rep.world == 2 and rep.rank == int(os.environ["RANK"])
# the slower rank decides the time of the whole job
ms = [12.5, 40.0][rep.rank]
t0 = time.monotonic()
if rep.rank == 1:
    time.sleep(0.5)
rep.barrier()
waited = time.monotonic() - t0
worst = rep.max_over_ranks(ms)
rate = rep.whole_job_rate(100, worst)
rep.barrier()
rep.close()
print(json.dumps({"rank": rep.rank, "worst": worst, "rate": rate, "waited": waited}))
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _env(rank, world, port):
    e = dict(os.environ)
    e.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
             OMP_NUM_THREADS="1")
    return e


def test_two_gloo_ranks_barrier_max_and_sum():
    port = _free_port()
    procs = [subprocess.Popen([sys.executable, "-c", _RANK_PROG % ROOT], env=_env(r, 2, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["worst"] == 40.0                       # the max over ranks, on every rank
        assert abs(o["rate"] - 2 * 100 / 0.040) < 1e-9  # both replicas' units over the slower rank's time
    assert outs[0]["waited"] >= 0.4                     # rank 0 did wait at the barrier for rank 1


def test_single_process_needs_no_process_group():
    import bench

    env_keep = {k: os.environ.pop(k, None) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    try:
        rep = bench.Replicas("gloo")
        assert rep.world == 1 and rep.dist is None
        rep.barrier()
        assert rep.max_over_ranks(3.25) == 3.25
        assert rep.whole_job_rate(10, 1000.0) == 10.0
        rep.close()
    finally:
        for k, v in env_keep.items():
            if v is not None:
                os.environ[k] = v


def test_reference_arm_runs_on_rank_zero_only():
    """Under a 2-rank launch the second rank of `--impl reference` prints nothing and exits 0 without work."""
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
                        "--warmup", "1"], env=_env(1, 2, _free_port()), capture_output=True, text=True, timeout=120)
    assert p.returncode == 0, p.stderr[-2000:]
    assert p.stdout.strip() == ""


def test_reference_arm_line_on_rank_zero():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "1", "--steps", "3",
                        "--warmup", "1", "--layers", "1"], env=_env(0, 1, _free_port()), capture_output=True, text=True,
                       timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "treekv_decode_steps_per_s" and line["unit"] == "steps/s"
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["higher_is_better"] is True and line["config"]["workload"] == "cfg4"
