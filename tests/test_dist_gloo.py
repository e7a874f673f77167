"""The N > 1 host logic of the benchmark on CPU: two gloo ranks, no GPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2606_11718_b200 import dist
    g = dist.Group("gloo")
    assert g.world == 2
    g.barrier()
    # rank 1 is the slow one: 4 ms per step vs 2 ms; each rank processes 10 units per step
    ups, ms = dist.job_throughput(10.0, 2.0 * (g.rank + 1), g)
    items = dist.shard(list(range(7)), g.rank, g.world)
    g.barrier()
    if g.rank == 0:
        print(json.dumps({"ups": ups, "ms": ms, "items": items}))
    else:
        assert items == [3, 4, 5, 6]
    g.close()
""") % ROOT


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_max_time_and_aggregate():
    port = free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["ms"] == 4.0                               # the slowest rank sets the time
    assert abs(res["ups"] - 20.0 / 4e-3) < 1e-6           # all ranks' units over that time
    assert res["items"] == [0, 1, 2]


def test_single_process_is_a_noop_group():
    sys.path.insert(0, ROOT)
    from paper_2606_11718_b200 import dist
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    g = dist.Group("gloo")
    assert (g.rank, g.world) == (0, 1)
    assert g.max_over_ranks(3.5) == 3.5 and g.sum_over_ranks(2.0) == 2.0
    assert dist.job_throughput(8.0, 2.0, g) == (4000.0, 2.0)
    assert dist.shard([1, 2, 3], 0, 1) == [1, 2, 3]
    g.close()


def test_reference_arm_rank1_prints_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


SPAWNED = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2606_11718_b200 import dist
    g = dist.Group("gloo")
    ups, ms = dist.job_throughput(5.0, 1.0 + g.rank, g)
    if g.rank == 0:
        print(json.dumps({"n_gpus": g.world, "ups": ups, "ms": ms, "local": g.local}), flush=True)
    g.close()
""") % ROOT


def test_spawn_helper_runs_two_gloo_ranks():
    """The helper behind `bench.py --gpus N` when no launcher set the environment: N children, rank 0 prints one line."""
    driver = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        from paper_2606_11718_b200 import dist
        sys.exit(dist.spawn_ranks(2, [sys.executable, "-c", %r], timeout=120))
    """) % (ROOT, SPAWNED)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT", "MASTER_ADDR")}
    out = subprocess.run([sys.executable, "-c", driver], env=env, capture_output=True, text=True, timeout=180)
    assert out.returncode == 0, out.stderr
    import json
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    res = json.loads(lines[0])
    assert res == {"n_gpus": 2, "ups": 10.0 / 2e-3, "ms": 2.0, "local": 0}


def test_spawn_helper_reports_a_failing_rank():
    sys.path.insert(0, ROOT)
    from paper_2606_11718_b200 import dist
    code = "import os, sys, time\nsys.exit(3) if os.environ['RANK'] == '1' else time.sleep(30)"
    assert dist.spawn_ranks(2, [sys.executable, "-c", code], timeout=60) == 3
