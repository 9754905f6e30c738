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


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2` without torchrun starts two ranks itself (torch.distributed.run,
    rendezvous on 127.0.0.1).  On a CPU machine the host leg of the path (--impl host-plan: plan
    compilation only, gloo) runs through exactly the launch, sharding, barrier and
    max-over-ranks code the GPU arm uses."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "host-plan",
                          "--config", "c2", "--steps", "4", "--warmup", "3"], env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                     # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "host-plan" and line["scaling"] == "weak"
    assert line["config"]["sequences_per_rank"] == 8           # shard_units: one batch of 8 per rank
    # all ranks' units / the slowest rank's time
    assert abs(line["value"] - 2 * 8 * 4 / (line["ms_per_step"] * 4e-3)) < 1e-6 * line["value"]
