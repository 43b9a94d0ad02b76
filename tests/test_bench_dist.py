"""The N > 1 plumbing of bench.py (barrier, max-over-ranks time, summed units) on two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, {root!r})
    import bench
    rank, local, world = bench.init_dist("gloo")
    assert world == 2 and rank == int(os.environ["RANK"])
    bench.barrier(world)
    # rank 0 was "faster": the job time is the slower rank's, the work is the sum
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1), world)
    bench.barrier(world)
    print(json.dumps({{"rank": rank, "ms": ms, "units": units}}))
""")


def test_two_rank_aggregation_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = 29000 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        outs.append(out.strip().splitlines()[-1])
    import json
    for line in outs:
        d = json.loads(line)
        assert d["ms"] == 15.0 and d["units"] == 300.0


def test_reference_arm_skips_nonzero_ranks():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
