"""The multi-process plumbing of bench.py (replicas, no data-path collective) on CPU: two gloo ranks."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    import bench
    r = bench.Ranks("gloo", "cpu")
    r.barrier()
    slow = r.max_over_ranks(10.0 + 5.0 * r.rank)          # rank 1 is the slow one
    value = r.job_value(units_per_rank_step=1000.0, steps=4, ms=10.0 + 5.0 * r.rank)
    r.barrier()
    print(json.dumps({"rank": r.rank, "world": r.world, "seed": r.seed(2), "slow": slow, "value": value}))
    r.close()
""") % ROOT


def test_two_ranks_agree_on_the_slowest_time_and_use_their_own_seeds(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert [o["world"] for o in outs] == [2, 2]
    assert outs[0]["seed"] == 2 and outs[1]["seed"] == 1002          # every replica draws its own inputs
    assert outs[0]["slow"] == outs[1]["slow"] == 15.0                 # max over ranks, known to both
    # whole-job value: both ranks' units over the slowest rank's time
    assert outs[0]["value"] == outs[1]["value"] == 1000.0 * 2 * 4 / 15e-3


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    env = {k: os.environ.pop(k) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK") if k in os.environ}
    try:
        r = bench.Ranks("gloo", "cpu")
        assert (r.rank, r.world) == (0, 1) and r.dist is None
        assert r.max_over_ranks(3.5) == 3.5 and r.seed(7) == 7
        r.barrier()
        r.close()
    finally:
        os.environ.update(env)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""         # the other ranks exit without work
