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


def _row_shard_worker(rank, world, port, out_dir):
    """Cache rows split over two ranks: each rank looks the whole batch up in its rows (oracle), the neighbour tuples
    travel through the one all-gather the GPU path uses, and the merge of what arrived equals the unsharded answer."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import fi_oracle as fo
    from paper_2002_02645_b200 import datagen as dg
    fo.set_threads(1)
    st = dg.single_layer(name="t", n_cache=333, n_query=24, dim=64, num_classes=5, dtype="f32", sigma=0.5, k=4,
                         seed=31).stages[0]
    cuts = [sharding.shard_bounds(333, world, r) for r in range(world)]
    lo, hi = cuts[rank]
    mine = fo.lookup(st.queries, st.cache_vecs[lo:hi], st.cache_labels[lo:hi], k=4, tau=0.46)
    tensors = [torch.from_numpy(mine.nd.astype(np.float32)),
               torch.from_numpy((mine.ni + lo).astype(np.int32)),
               torch.from_numpy(st.cache_labels[lo:hi][mine.ni].astype(np.int32)),
               torch.ones(mine.ni.shape, dtype=torch.float32)]
    d, gi, lab, wgt = sharding.gather_shard_tuples(tensors)
    ok = d.shape == (world, 24, 4) and d.dtype == torch.float32 and gi.dtype == torch.int32
    ok = ok and torch.equal(d[rank], tensors[0]) and torch.equal(gi[rank], tensors[1])
    # every rank holds every shard's tuples now; rebuild per-shard results from them and merge
    parts = []
    for r, (a, b) in enumerate(cuts):
        nd = d[r].numpy().astype(np.float64)
        parts.append(fo.LookupResult(None, None, None, nd, gi[r].numpy().astype(np.int64) - a, None))
        ok = ok and np.array_equal(lab[r].numpy(), st.cache_labels[gi[r].numpy()])
    merged = fo.merge_shards(parts, [a for a, _ in cuts], [st.cache_labels[a:b] for a, b in cuts], k=4, tau=0.46)
    whole = fo.lookup(st.queries, st.cache_vecs, st.cache_labels, k=4, tau=0.46)
    ok = ok and np.array_equal(merged.ni, whole.ni) and np.array_equal(merged.label, whole.label) \
        and np.array_equal(merged.hit, whole.hit) and 0 < whole.hit.sum() < 24
    with open(os.path.join(out_dir, f"result{rank}"), "w") as f:
        f.write("ok" if ok else "bad")
    dist.barrier()
    dist.destroy_process_group()


def test_row_sharding_two_ranks_gloo(tmp_path):
    from oracle import fi_oracle as fo
    fo.build()
    port = _free_port()
    mp.spawn(_row_shard_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "result0").read_text() == "ok" and (tmp_path / "result1").read_text() == "ok"


def _bench(*argv, timeout=600):
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    proc = subprocess.run([sys.executable, os.path.join(root, "bench.py"), *argv], stdout=subprocess.PIPE,
                          stderr=subprocess.PIPE, text=True, timeout=timeout, env=env, cwd=root)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [l for l in proc.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, proc.stdout          # rank 0 alone prints, and exactly one line
    return json.loads(lines[0])


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` without a launcher around it starts two ranks itself; they form a process group (gloo here,
    NCCL on GPUs), meet at the barrier, and the timing reduction takes the slowest rank's time and everybody's work."""
    line = _bench("--gpus", "2", "--workload", "launch-check")
    assert line["n_gpus"] == 2 and line["requested"] == 2
    assert line["max_ms"] == 2.0 and line["units"] == 20.0 and line["backend"] == "gloo"


def test_bench_reference_arm_under_two_ranks_prints_one_line():
    line = _bench("--gpus", "2", "--impl", "reference", "--workload", "cfg2-small", "--steps", "1", "--warmup", "0",
                  "--cpu-sample", "2")
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
