"""N > 1 is "replicas only": two CPU ranks over gloo exercise the timing plumbing bench.py uses
(barrier, max over ranks, whole-job aggregate) and the rule that only rank 0 of the reference
arm works and prints.  No data-path collective exists, so none is tested.
"""
import json
import os
import socket
import subprocess
import sys
import textwrap

REPO = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(world, argv_of_rank, timeout=300):
    port = _free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=REPO)
        procs.append(subprocess.Popen(argv_of_rank(r), env=env, cwd=REPO, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            o, e = p.communicate(timeout=timeout)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        outs.append((p.returncode, o, e))
    return outs


RANK_BODY = textwrap.dedent("""
    import json, time
    import numpy as np
    import oracle
    from paper_2607_10389_b200.replicas import Replicas

    g = Replicas("gloo", None)
    # each rank is a replica with a cache of its own: nothing is exchanged but timings
    rng = np.random.default_rng(100 + g.rank)
    cache = rng.integers(0, 256, 4 * 65536 + 1000 * g.rank, dtype=np.uint8)
    g.barrier()
    t = time.perf_counter()
    wire, crc, res = oracle.encode(cache, 65536)
    out, _, r = oracle.decode_verify(wire, cache.size, 65536)
    mine = (time.perf_counter() - t) * 1e3 + 1000.0 * g.rank      # rank 1 is made the slow one
    g.barrier()
    slowest = g.max_over_ranks(mine)
    print(json.dumps({"rank": g.rank, "world": g.world, "mine": mine, "slowest": slowest,
                      "agg": g.aggregate_gbs(10**9, 500.0), "ok": bool(res.status == 0 and r.status == 0
                      and np.array_equal(out, cache)), "crc0": int(crc[0])}))
    g.close()
""")


def test_two_gloo_ranks_agree_on_the_slowest_time():
    outs = _launch(2, lambda r: [sys.executable, "-c", RANK_BODY])
    recs = []
    for code, o, e in outs:
        assert code == 0, e[-2000:]
        recs.append(json.loads(o.strip().splitlines()[-1]))
    recs.sort(key=lambda d: d["rank"])
    assert [d["rank"] for d in recs] == [0, 1] and all(d["world"] == 2 for d in recs)
    assert all(d["ok"] for d in recs)
    assert recs[0]["crc0"] != recs[1]["crc0"]                 # the replicas really differ
    assert recs[1]["mine"] > recs[0]["mine"]
    # both ranks report the slow rank's figure, and the aggregate counts both replicas
    assert recs[0]["slowest"] == recs[1]["slowest"] == recs[1]["mine"]
    assert recs[0]["agg"] == 2 * 1e9 / 0.5 / 1e9


def test_single_process_needs_no_group():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    env["PYTHONPATH"] = REPO
    code = ("from paper_2607_10389_b200.replicas import Replicas\n"
            "g = Replicas('gloo', None); g.barrier()\n"
            "assert (g.rank, g.world) == (0, 1) and g.max_over_ranks(3.5) == 3.5\n"
            "assert g.aggregate_gbs(2 * 10**9, 1000.0) == 2.0; g.close()\n")
    assert subprocess.run([sys.executable, "-c", code], env=env, cwd=REPO).returncode == 0


def test_reference_arm_runs_on_rank_zero_only():
    argv = [sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
            "--workload", "tiny"]
    outs = _launch(2, lambda r: argv)
    (c0, o0, e0), (c1, o1, e1) = outs
    assert c0 == 0 and c1 == 0, (e0[-1000:], e1[-1000:])
    assert o1.strip() == ""
    line = json.loads(o0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
