"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on CPU with gloo, world size 2."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2401_15077_b200 import replicas, workloads as W
    # every rank draws its own batch of the same workload
    cfg = W.scaled(W.CONFIGS["tiny"], batch=2, prefix=(8, 40))
    sizes, parent = W.make_trees(cfg, salt=replicas.rank_salt(rank))
    lens = W.make_attn_inputs(cfg, salt=replicas.rank_salt(rank)).seq_lens
    replicas.barrier()
    elapsed_ms = 10.0 * (rank + 1)             # rank 1 is the slow replica
    value = replicas.whole_job_steps_per_s(elapsed_ms, steps=5)
    slowest = replicas.max_over_ranks(elapsed_ms)
    gathered = [None] * world
    dist.all_gather_object(gathered, (parent.tolist(), lens.tolist()))
    out[rank] = (value, slowest, gathered[0] != gathered[1])
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        value, slowest, differ = res[rank]
        assert slowest == 20.0
        assert abs(value - 2 * 5 / 0.020) < 1e-9      # both ranks' steps over the slowest rank's time
        assert differ                                  # the ranks really verified different batches


def test_single_process_needs_no_group():
    from paper_2401_15077_b200 import replicas
    assert not replicas.is_distributed()
    replicas.barrier()
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_steps_per_s(100.0, 10) == 100.0
