"""Host-side checks of bench.py: the multi-rank timing reduction over gloo
(world size 2, CPU) and the oracle-timing leg on the tiny workload."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r measured (10 + r) ms of device time and (20 - r) ms end to end
    total_ms, e2e_ms = bench.max_over_ranks([10.0 + rank, 20.0 - rank], dist, "cpu")
    value = bench.aggregate_value(1000, world, 4, total_ms)
    out.put((rank, total_ms, e2e_ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_timings_reduce_to_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total_ms, e2e_ms, value in got:
        assert total_ms == 11.0 and e2e_ms == 20.0          # max over ranks, on every rank
        assert abs(value - 1000 * 2 * 4 / 11e-3) < 1e-6      # whole job: both replicas' tokens


def test_oracle_timing_leg_on_the_tiny_workload():
    import bench
    r = bench.oracle_sample("tiny", 2000, n_heads_sample=4, decode_steps=2)
    assert r["kind"] == "oracle" and r["unit"] == "tokens/s" and r["value"] > 0 and r["cores"] >= 1
    assert "gate" in r["sample"]


def test_gpus_flag_turns_into_one_process_per_gpu():
    """`bench.py --gpus N` started by hand (no WORLD_SIZE in the environment) re-launches itself as N
    replicas on this node, rendezvous on 127.0.0.1, with its own arguments passed through."""
    import bench
    cmd = bench.replica_command(4, ["--gpus", "4", "--steps", "5"], 29611)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert "--nproc-per-node=4" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29611"
    assert cmd[-5].endswith("bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "5"]
