"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own stream and
table state (weak scaling, no data-path collective); job figures are MAX of the ranks'
times and SUM of their work."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from oracle import mono_oracle as mo
    from paper_2209_07663_b200 import workload as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = bench.rank_config(wl.scaled(wl.CONFIGS["tiny"], n_examples=64, steps=2), rank)
        stream = wl.Stream(cfg)
        table = mo.OracleTable(cfg.capacity, cfg.dim, cfg.filter_threshold, cfg.ttl, seed=cfg.seed)
        n_ids = 0
        for t in range(cfg.steps):          # the rank's own shard of the job: independent table, own batches
            s = stream.step(t)
            table.apply_grads(s.ids, s.offsets, s.grad_pooled, t)
            n_ids += s.ids.size
        first_ids = stream.step(0).ids[:64]
        (t_max, e_max), (w_sum, _) = bench.aggregate_over_ranks([10.0 + 5.0 * rank, 1.0 + rank], [float(n_ids), 0.0])
        np.save(os.path.join(out_dir, f"rank{rank}.npy"),
                np.array([t_max, e_max, w_sum, float(n_ids), float(first_ids[0] % (1 << 52))]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_the_stream_and_aggregate(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"rank{r}.npy") for r in range(world))
    assert r0[0] == r1[0] == 15.0 and r0[1] == r1[1] == 2.0           # MAX over ranks of each timed region
    assert r0[2] == r1[2] == r0[3] + r1[3]                            # SUM of the ranks' work
    assert r0[4] != r1[4]                                             # different seeds: different ID streams


def test_aggregation_without_a_process_group_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks([3.0, 4.0], [5.0, 6.0]) == ([3.0, 4.0], [5.0, 6.0])
    import paper_2209_07663_b200.workload as wl
    assert bench.rank_config(wl.CONFIGS["tiny"], 0).seed != bench.rank_config(wl.CONFIGS["tiny"], 1).seed
