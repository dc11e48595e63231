"""The N > 1 launch path of bench.py on CPU: two gloo ranks.

The path shards with no exchange step: every rank runs its own independent sequence and the
only communication is a barrier and a MAX over ranks of the timed duration.  This test runs
that plumbing (rendezvous on 127.0.0.1, per-rank seeds, barrier, max-reduce, whole-job
aggregate) with two CPU processes; the kernels themselves need a GPU and are covered by the
-m gpu tests.
"""

import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    import bench
    from paper_2606_13392_b200.inputs import CONFIGS, make_prefill_inputs

    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = CONFIGS["c1"]
    # every rank draws its own sequence (the rule bench.py uses)
    mycfg = cfg.scaled(seed=bench.rank_seed(cfg.seed, rank))
    x = make_prefill_inputs(mycfg, "cpu")
    checksum = float(x["q"].float().sum())
    # stand-in for the timed region: rank r "takes" (r + 1) * 10 ms per step
    ms_step, value = bench.aggregate(10.0 * (rank + 1) * 4, steps=4, units=cfg.T, world=world,
                                     device=torch.device("cpu"), dist=dist)
    sums = [None] * world
    dist.all_gather_object(sums, checksum)
    if rank == 0:
        torch.save({"ms_step": ms_step, "value": value, "sums": sums}, os.path.join(out_dir, "r0.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_weak_scaling_plumbing(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = torch.load(os.path.join(str(tmp_path), "r0.pt"))
    # the slowest rank (20 ms per step) sets the step time; value is the whole-job aggregate
    assert abs(res["ms_step"] - 20.0) < 1e-9
    assert abs(res["value"] - world * 2048 / 20e-3) < 1e-6
    # the two ranks worked on different sequences
    assert res["sums"][0] != res["sums"][1]


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--workload", "c1"])
    bench.main()  # rank 1: exits without work and prints nothing
    assert capsys.readouterr().out.strip() == ""
