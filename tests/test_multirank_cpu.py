"""World-size-2 run (gloo, CPU) of the multi-rank plumbing that `bench.py --gpus N` uses.

The path does not shard: every rank streams its own replica, and the ranks meet only at the
barriers around the timed region and in the two reductions that build the reported line
(max of the per-rank times, sum of the per-rank rates).  This test runs exactly those helpers
in two processes and checks that the replicas' inputs are distinct.
"""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent(
    """
    import hashlib, json, sys
    sys.path.insert(0, %r)
    import torch
    import torch.distributed as dist
    import bench
    from paper_2412_04757_b200 import inputs

    rank, local, world = bench.dist_setup(2)
    assert world == 2 and dist.get_backend() == "gloo"
    dev = torch.device("cpu")
    bench.barrier(world)
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, dev)          # slowest rank decides the time
    rate = bench.sum_over_ranks(512 / (ms * 1e-3), world, dev)        # whole-job rate at that time
    cfg = inputs.config(0)
    st = inputs.SyntheticStream(cfg, seq=rank * cfg.n_seqs)           # the replica this rank would stream
    q, k, v = st.tokens(0, cfg.chunk)
    h = hashlib.sha256(inputs.bf16_bits(k).tobytes()).hexdigest()
    hs = [None, None]
    dist.all_gather_object(hs, h)
    bench.barrier(world)
    if rank == 0:
        print(json.dumps({"ms": ms, "rate": rate, "distinct": hs[0] != hs[1]}))
    dist.destroy_process_group()
    """
) % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_reductions_and_distinct_replicas(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se[-2000:]
    import json

    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ms"] == 20.0                                    # max over ranks
    assert abs(line["rate"] - 2 * 512 / 20e-3) < 1e-6            # both ranks' tokens over the slowest time
    assert line["distinct"]


def test_reference_arm_runs_on_rank_zero_only():
    """Under a multi-rank launch only rank 0 times the oracle; the other ranks leave without work."""
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--config", "0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    assert r.stdout.strip() == ""
