"""The N > 1 path of bench.py on CPU: two gloo ranks on 127.0.0.1 check the sharding (every rank its own batch
of the same shape), the max-over-ranks reduction and the whole-job value; no GPU and no kernel is involved."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    from paper_2609_38166_b200 import synth
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench.shard_workload(synth.config("gdn_b256"), rank)
    tok = synth.token_inputs(wl.with_(batch=2), 0)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist)             # rank 1 is the slow one
    out = {"rank": rank, "seed": wl.seed, "batch": wl.batch, "ms": ms, "q0": int(tok["q"].ravel()[0]),
           "value": bench.whole_job_value(wl.batch * wl.heads_v, world, 100, ms)}
    dist.barrier()
    dist.destroy_process_group()
    print(json.dumps(out))
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_shard_and_reduce():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        stdout, _ = p.communicate(timeout=120)
        assert p.returncode == 0
        outs.append(json.loads(stdout.strip().splitlines()[-1]))
    a, b = sorted(outs, key=lambda o: o["rank"])
    assert a["seed"] != b["seed"] and a["batch"] == b["batch"] == 256       # same shape, different data
    assert a["q0"] != b["q0"]
    assert a["ms"] == b["ms"] == 15.0                                        # the slowest rank's time
    import bench
    assert a["value"] == b["value"] == bench.whole_job_value(256 * 32, 2, 100, 15.0)
    assert abs(a["value"] - 2 * bench.whole_job_value(256 * 32, 1, 100, 15.0)) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
