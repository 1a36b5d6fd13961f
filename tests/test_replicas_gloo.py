"""The N > 1 path of the benchmark on CPU: two gloo ranks run the same timing aggregation the GPU job uses
(barrier, max over ranks, whole-job throughput) and draw different batches from the same network."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import numpy as np
    from paper_1602_02830_b200 import replicas, workloads as wl
    world, rank, local = replicas.world()
    replicas.init("gloo")
    replicas.barrier()
    # every rank draws the same network and its own batch
    case = wl.mlp_case(batch=4, sizes=(16, 8, 4), seed=1)
    X = case["X"] if rank == 0 else wl.u8(np.random.default_rng(replicas.rank_seed(1, rank)), (4, 16))
    my_ms = [10.0 + 5.0 * rank, 2.0 - rank]          # rank 1 is slower on the first, faster on the second
    mx = replicas.max_over_ranks(my_ms)
    out = {"rank": rank, "world": world, "max": mx, "w0": int(case["weights"][0].sum()), "x": int(X.sum()),
           "thr": replicas.job_throughput(100.0, mx[0], world)}
    print("RESULT " + json.dumps(out), flush=True)
    replicas.finish()
""") % ROOT


def test_two_gloo_ranks_aggregate_like_the_bench(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    results = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        import json
        line = [l for l in out.splitlines() if l.startswith("RESULT ")][0]
        results.append(json.loads(line[7:]))
    r0, r1 = sorted(results, key=lambda r: r["rank"])
    assert r0["world"] == r1["world"] == 2
    assert r0["max"] == r1["max"] == [15.0, 2.0]                 # slowest rank per entry
    assert r0["w0"] == r1["w0"]                                  # same weights on every replica
    assert r0["x"] != r1["x"]                                    # different batches
    assert abs(r0["thr"] - 2 * 100.0 / 0.015) < 1e-6             # whole-job units/s over the max time


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_1602_02830_b200 import replicas
    assert replicas.world() == (1, 0, 0) or "WORLD_SIZE" in os.environ
    assert replicas.max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert replicas.job_throughput(10000, 0.5, 1) == 2.0e7
