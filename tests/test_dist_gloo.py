"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch (no data-path
collective), agree on barrier, max-over-ranks timing and the aggregate throughput, and compile
identical plans for identical inputs."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, ROOT_PLACEHOLDER)
    import numpy as np
    from paper_2607_24260_b200 import dist as kdist, kap, synth
    g = kdist.Group("gloo", device="cpu")
    assert g.world == 2
    # every rank draws its own batch (weak scaling): different seeds, same shapes
    w = synth.config2(g.rank, batch=2, L=2048, layers=1)
    plan = kap.compile_workload(w)
    g.barrier()
    local_time = 1.0 + g.rank                      # pretend rank 1 is slower
    t = g.max_float(local_time)
    total = kdist.aggregate_throughput(float(w.batch), local_time, g)
    lo, hi = kdist.shard_units(7, g.rank, g.world)
    # same inputs on both ranks give bit-identical plans
    same = kap.compile_workload(synth.config2(0, batch=2, L=2048, layers=1))
    digest = int(np.sum(same["plan_logical_pages"].astype(np.int64) * 31 % 1000003))
    agree = g.max_float(digest) == g.sum_float(digest) / 2
    print(json.dumps(dict(rank=g.rank, t=t, total=total, shard=[lo, hi], agree=agree,
                          pages=int(plan["plan_indptr"][-1]))))
    g.close()
""").replace("ROOT_PLACEHOLDER", repr(ROOT))


def test_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    import json
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["t"] == outs[1]["t"] == 2.0                 # max over ranks
    assert outs[0]["total"] == outs[1]["total"] == 4 / 2.0     # all units / slowest time
    assert outs[0]["shard"] == [0, 4] and outs[1]["shard"] == [4, 7]
    assert outs[0]["agree"] and outs[1]["agree"]
    assert outs[0]["pages"] > 0 and outs[1]["pages"] > 0
