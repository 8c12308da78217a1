"""World-size-2 run on CPU (gloo): request sharding, the independence of shards that "replicas only" relies on,
and the timing reduction bench.py uses."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2002_02645_b200 import sharding


def test_shard_bounds_partition():
    for total in (0, 1, 7, 1024, 1025):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_bounds(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_bounds(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import fi_oracle as fo
    from paper_2002_02645_b200 import datagen as dg
    fo.set_threads(1)
    w = dg.config2(seed=0, shrink=64)           # 4 stages, 16 requests, 156 entries
    taus = [2e-3, 4e-3, 8e-3, 1.6e-2]
    b0 = w.stages[0].queries.shape[0]
    lo, hi = sharding.shard_bounds(b0, world, rank)
    r = fo.cascade([s.queries[lo:hi] for s in w.stages], [s.cache_vecs for s in w.stages],
                   [s.cache_labels for s in w.stages], taus, k=w.k)
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, r.final_label, r.exit_stage))
    ms, units = sharding.reduce_timing(10.0 * (rank + 1), hi - lo)
    dist.barrier()
    if rank == 0:
        full = fo.cascade([s.queries for s in w.stages], [s.cache_vecs for s in w.stages],
                          [s.cache_labels for s in w.stages], taus, k=w.k)
        label = np.concatenate([g[2] for g in sorted(gathered)])
        stage = np.concatenate([g[3] for g in sorted(gathered)])
        ok = np.array_equal(label, full.final_label) and np.array_equal(stage, full.exit_stage) \
            and ms == 10.0 * world and units == b0 and len(set(full.exit_stage.tolist())) >= 3
        with open(os.path.join(out_dir, "result"), "w") as f:
            f.write("ok" if ok else f"bad {label} {full.final_label} {stage} {full.exit_stage} {ms} {units}")
    dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    from oracle import fi_oracle as fo
    fo.build()
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "result").read_text() == "ok"
